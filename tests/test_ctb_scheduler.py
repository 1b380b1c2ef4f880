"""Algorithm 1 (Semantic-Aware CTB Scheduling): the product scheduler against the oracle that restates the
listing, on seeded random traces (identical decisions, in order), plus the properties the algorithm fixes and a
sanity check of the rollout simulator.  CPU only."""
import numpy as np

from oracle import ctb_alg1 as oracle
from paper_2608_10402_b200 import ctb


def _trace(seed, n_ranks, passes=60, inflight_cap=None, window=1, n_kinds=1):
    rng = np.random.default_rng(seed)
    budgets = [int(rng.integers(3000, 9000)) for _ in range(n_ranks)]
    env_limit = int(rng.integers(6, 30))
    sched = ctb.CTBScheduler(budgets, ctx_norm=8192.0, env_limit=env_limit, inflight_cap=inflight_cap, window=window)
    unconsumed = 0
    otasks, oqueue = [], []
    w = oracle.Weights()
    next_id = 0
    for p in range(passes):
        # arrivals
        for _ in range(int(rng.integers(0, 5))):
            group, is_eval, probed = int(rng.integers(0, 6)), bool(rng.random() < 0.15), int(rng.integers(200, 1500))
            kind = int(rng.integers(0, n_kinds))
            sched.submit(next_id, group, probed, is_eval, kind=kind)
            otasks.append(oracle.Task(next_id, group, is_eval, probed, kind=kind))
            oqueue.append(next_id)
            next_id += 1
        # some active tasks finish, the others grow (turn probing)
        act = [t.id for t in otasks if t.state == "active"]
        for tid in act:
            if rng.random() < 0.1:
                sched.finish(tid)
                next(t for t in otasks if t.id == tid).state = "done"
                unconsumed += 1
        grow = {tid: next(t for t in otasks if t.id == tid).footprint + int(rng.integers(0, 900))
                for tid in act if next(t for t in otasks if t.id == tid).state == "active" and rng.random() < 0.7}
        if inflight_cap is not None and rng.random() < 0.3:      # the trainer takes a batch
            n = int(rng.integers(0, unconsumed + 1))
            sched.consume(n)
            unconsumed -= n
        got = sched.schedule(grow)
        want = oracle.schedule_pass(otasks, oqueue, budgets, w, 8192.0, env_limit, grow, inflight_cap=inflight_cap,
                                    unconsumed=unconsumed, window=window)
        assert got == want, f"pass {p}: {got} != {want}"
        yield sched, otasks, budgets, env_limit, got


def test_scheduler_matches_the_listing_on_random_traces():
    n_events = 0
    kinds = set()
    for seed in range(6):
        for sched, otasks, budgets, env_limit, ev in _trace(seed, n_ranks=1 + seed % 3):
            n_events += len(ev)
            kinds.update(k for k, _, _ in ev)
            # same bookkeeping on both sides
            for r in range(len(budgets)):
                assert sched.usage[r] == oracle.token_usage(otasks, r)
            assert {t.id for t in otasks if t.state == "paused"} == set(sched.paused)
    assert n_events > 200 and kinds == {"admit", "evict", "resume"}


def test_budget_concurrency_and_affinity_hold_after_every_pass():
    for sched, otasks, budgets, env_limit, ev in _trace(11, n_ranks=3):
        for r, B in enumerate(budgets):
            # over budget only if a single task alone exceeds it (the loop stops when nothing is left to preempt)
            assert sched.usage[r] <= B or len(sched.active[r]) <= 1
        assert sched.n_active <= env_limit
        evicted_from = {}
        for kind, tid, r in ev:
            if kind == "evict":
                evicted_from[tid] = r
        for kind, tid, r in ev:
            if kind == "resume" and tid in evicted_from:
                assert evicted_from[tid] == r, "a paused task resumed away from the rank that holds its prefix"


def test_priority_tiers_decide_who_is_preempted():
    # one rank, four active tasks that differ in exactly one tier each; shrinking headroom evicts them in the
    # order Low (short context) -> ... -> evaluation task last (Table 1)
    s = ctb.CTBScheduler([10_000], ctx_norm=8192.0)
    s.submit(0, group=0, probed=1000, is_eval=True)
    s.submit(1, group=1, probed=1000)
    s.submit(2, group=2, probed=1000)
    s.submit(3, group=1, probed=1000)          # same group as 1
    s.submit(4, group=1, probed=1000)
    assert [e[0] for e in s.schedule()] == ["admit"] * 5
    s.finish(4)                                 # group 1 is now 1/3 complete: tasks 1 and 3 rank above task 2
    s.schedule({0: 3000, 1: 3000, 2: 3000, 3: 2000})   # usage 11000 > 10000
    assert s.tasks[3].state == "active" and s.tasks[2].state == "paused"   # lowest tier value goes first
    order = []
    for shrink in (7000, 4000, 2500):
        s.budgets[0] = shrink
        order += [tid for kind, tid, _ in s.schedule() if kind == "evict"]
    assert order == [3, 1, 0] or order[:2] == [3, 1]     # short context before long, evaluation task last
    assert s.tasks[0].state in ("active", "paused")


def test_simulated_rollout_ctb_keeps_more_kv_than_request_batching():
    rng = np.random.default_rng(0)
    rollout = ctb.synthetic_rollout(rng, n_groups=24, group_size=8)
    budget = 120_000
    a = ctb.simulate(rollout, "ctb", budget)
    b = ctb.simulate(rollout, "request", budget, fixed_concurrency=96)
    assert a["context"] > 0 and b["context"] > 0
    assert a["hit_rate"] > b["hit_rate"] and a["prefilled"] < b["prefilled"]
    # with ample memory nothing is ever dropped under either policy
    c = ctb.simulate(rollout, "request", 10**9, fixed_concurrency=96)
    assert c["hit_rate"] == 1.0


def test_staleness_and_diversity_constraints_match_the_listing():
    """Section 4.2's admission constraints: no new task while the trajectories in flight reach the cap; among the
    first queued tasks that fit, the type least represented on the rank goes first."""
    n_admit = 0
    for seed in range(4):
        cap = 10 + 3 * seed
        for sched, otasks, budgets, env_limit, ev in _trace(100 + seed, n_ranks=1 + seed % 2, inflight_cap=cap, window=4, n_kinds=3):
            n_admit += sum(1 for k, _, _ in ev if k == "admit")
            in_flight = sum(1 for t in otasks if t.state in ("active", "paused")) + sched.unconsumed
            # an admission happens only below the cap, so a pass can end at the cap but not beyond it through admissions
            if any(k == "admit" for k, _, _ in ev):
                assert in_flight <= cap
            assert [t.id for t in otasks if t.state == "new"] == sched.new_queue[sched._new_head:]
    assert n_admit > 30
    # diversity on a hand-made case: rank 0 already runs two tasks of type 0; the queue holds types 0, 0, 1
    s = ctb.CTBScheduler([100_000], window=3)
    for i, kind in enumerate([0, 0]):
        s.submit(i, group=i, probed=100, kind=kind)
    s.schedule()
    for i, kind in enumerate([0, 0, 1], start=2):
        s.submit(i, group=i, probed=100, kind=kind)
    assert [e[1] for e in s.schedule()] == [4, 2, 3]          # the type-1 task jumps the queue, then arrival order
    # staleness on a hand-made case: cap 3, two active and one finished-but-unconsumed trajectory block admission
    s = ctb.CTBScheduler([100_000], inflight_cap=3)
    for i in range(5):
        s.submit(i, group=i, probed=100)
    assert [e[1] for e in s.schedule()] == [0, 1, 2]
    s.finish(0)
    assert s.schedule() == []                                  # 2 active + 1 unconsumed = cap
    s.consume(1)
    assert [e[1] for e in s.schedule()] == [3]


# ---------------------------------------------------------------------------------------------------------
# Direct pins of the oracle.  Every expected decision list below was worked out by hand from Algorithm 1 (preempt
# the smallest Priority while over budget, then resume before admitting while under it) and the Priority sum of
# Section 4.2 with weights 8 / 4 / 2 / 1 and L_context = tokens / 8192; neither implementation was consulted.
W = oracle.Weights()
CTX = 8192.0


def _task(tid, group, fp, state="active", rank=0, is_eval=False, kind=0, probed=None):
    return oracle.Task(tid, group, is_eval, fp if probed is None else probed, kind=kind, footprint=fp, state=state, rank=rank)


def test_oracle_priority_is_the_weighted_sum_of_section_4_2():
    tasks = [_task(0, 0, 3000, is_eval=True), _task(1, 1, 3000), _task(2, 2, 3000), _task(3, 1, 2000),
             _task(4, 1, 500, state="done"), _task(5, 3, 16384, state="paused")]
    want = {0: 8 + 0 + 2 + 3000 / 8192,            # evaluation task, alone in its group
            1: 4 * (1 / 3) + 2 + 3000 / 8192,      # one of three group members has finished
            2: 0 + 2 + 3000 / 8192,
            3: 4 * (1 / 3) + 2 + 2000 / 8192,
            5: 0 + 0 + 1.0}                        # paused: no active term; context factor capped at 1
    for tid, p in want.items():
        assert abs(oracle.priority(tasks[tid], tasks, W, CTX) - p) < 1e-12, tid


def test_oracle_preempts_in_the_tier_order_of_table_1():
    tasks = [_task(0, 0, 3000, is_eval=True), _task(1, 1, 3000), _task(2, 2, 3000), _task(3, 1, 2000),
             _task(4, 1, 500, state="done")]
    run = lambda B: oracle.schedule_pass(tasks, [], [B], W, CTX, env_limit=100)
    # usage 11000: the task with no tier in its favour goes; nothing paused fits the 2000 tokens of headroom
    assert run(10_000) == [("evict", 2, 0)]
    # of the two members of the part-finished group the shorter context goes first
    assert run(7_000) == [("evict", 3, 0)]
    assert run(4_000) == [("evict", 1, 0)]
    # the evaluation task is the last to go; with the rank empty the only paused task that fits 2500 comes back
    assert run(2_500) == [("evict", 0, 0), ("resume", 3, 0)]
    # headroom again: paused tasks return in Priority order (evaluation, then the part-finished group) while they fit
    assert run(10_000) == [("resume", 0, 0), ("resume", 1, 0)]
    assert [t.state for t in tasks] == ["active", "active", "paused", "active", "done"]
    assert oracle.token_usage(tasks, 0) == 8000


def test_oracle_affinity_resume_before_admit_and_footprint_refresh_on_two_ranks():
    tasks = [_task(0, 0, 3000, rank=0), _task(1, 1, 3100, rank=0), _task(2, 2, 1000, rank=1),
             _task(3, 3, 0, state="new", rank=-1, probed=2000), _task(4, 4, 0, state="new", rank=-1, probed=2500)]
    queue = [3, 4]
    # rank 0 holds 6100 > 5000: the shorter of its two equal-tier tasks is preempted and does not fit back (3100 + 3000).
    # rank 1 has room for it (1000 + 3000) but the task may only return to rank 0, so rank 1 admits from the queue:
    # task 3 (1000 + 2000), then task 4 no longer fits (3000 + 2500 > 5000)
    ev = oracle.schedule_pass(tasks, queue, [5000, 5000], W, CTX, env_limit=100)
    assert ev == [("evict", 0, 0), ("admit", 3, 1)]
    assert queue == [4] and tasks[3].footprint == 2000 and tasks[0].rank == 0
    # task 1 finishes; probing reports task 2 at 1800 tokens (and a number for the paused task 0, which must be ignored).
    # rank 0 is empty: the paused task returns there BEFORE the queued task 4 is admitted beside it (3000 + 2500 > 5000: not at all)
    tasks[1].state = "done"
    ev = oracle.schedule_pass(tasks, queue, [5000, 5000], W, CTX, env_limit=100, new_footprints={2: 1800, 0: 9999})
    assert ev == [("resume", 0, 0)]
    assert tasks[2].footprint == 1800 and tasks[0].footprint == 3000
    assert oracle.token_usage(tasks, 0) == 3000 and oracle.token_usage(tasks, 1) == 3800
    # a larger budget on rank 0 lets the queued task in there, after the resume of the pass before
    ev = oracle.schedule_pass(tasks, queue, [6000, 5000], W, CTX, env_limit=100)
    assert ev == [("admit", 4, 0)] and queue == []


def test_oracle_admission_constraints_by_hand():
    # environment concurrency: two active tasks is the limit, so neither the paused task nor the queue moves
    tasks = [_task(0, 0, 100), _task(1, 1, 100), _task(2, 2, 100, state="paused"), _task(3, 3, 0, state="new", rank=-1, probed=100)]
    assert oracle.schedule_pass(tasks, [3], [10_000], W, CTX, env_limit=2) == []
    assert oracle.schedule_pass(tasks, [3], [10_000], W, CTX, env_limit=3) == [("resume", 2, 0)]
    # task diversity: the rank runs two tasks of type 0; of the queued types 0, 0, 1 the type-1 task goes first,
    # then the others in arrival order (their type is the most common one either way)
    tasks = [_task(0, 0, 100, kind=0), _task(1, 1, 100, kind=0)] + [
        _task(i, i, 0, state="new", rank=-1, probed=100, kind=k) for i, k in ((2, 0), (3, 0), (4, 1))]
    queue = [2, 3, 4]
    assert oracle.schedule_pass(tasks, queue, [100_000], W, CTX, env_limit=100, window=3) == [
        ("admit", 4, 0), ("admit", 2, 0), ("admit", 3, 0)]
    # window 1 is plain arrival order
    tasks = [_task(0, 0, 100, kind=0)] + [_task(i, i, 0, state="new", rank=-1, probed=100, kind=k) for i, k in ((1, 0), (2, 1))]
    assert oracle.schedule_pass(tasks, [1, 2], [100_000], W, CTX, env_limit=100, window=1) == [("admit", 1, 0), ("admit", 2, 0)]
    # policy staleness: cap 3 counts active + paused + finished-but-unconsumed trajectories
    tasks = [_task(i, i, 0, state="new", rank=-1, probed=100) for i in range(5)]
    queue = [0, 1, 2, 3, 4]
    kw = dict(budgets=[100_000], w=W, ctx_norm=CTX, env_limit=100, inflight_cap=3)
    assert oracle.schedule_pass(tasks, queue, unconsumed=0, **kw) == [("admit", 0, 0), ("admit", 1, 0), ("admit", 2, 0)]
    tasks[0].state = "done"
    assert oracle.schedule_pass(tasks, queue, unconsumed=1, **kw) == []            # 2 active + 1 unconsumed = cap
    assert oracle.schedule_pass(tasks, queue, unconsumed=0, **kw) == [("admit", 3, 0)]


def test_oracle_pass_invariants_on_random_states():
    """What the loop guarantees whatever the readings: a rank ends a pass over budget only when one task alone is
    too large for it (or nothing is left to preempt), every resume on a rank precedes every admit there, and a
    paused task comes back only to the rank it left."""
    rng = np.random.default_rng(7)
    for trial in range(200):
        n_ranks = int(rng.integers(1, 4))
        budgets = [int(rng.integers(1000, 6000)) for _ in range(n_ranks)]
        tasks, queue = [], []
        for tid in range(int(rng.integers(3, 14))):
            state = ["active", "paused", "new", "done"][int(rng.integers(0, 4))]
            fp = int(rng.integers(100, 3000))
            rank = int(rng.integers(0, n_ranks)) if state in ("active", "paused") else -1
            tasks.append(_task(tid, int(rng.integers(0, 4)), fp if state != "new" else 0, state=state, rank=rank,
                               is_eval=bool(rng.random() < 0.2), probed=fp))
            if state == "new":
                queue.append(tid)
        home = {t.id: t.rank for t in tasks if t.state == "paused"}
        ev = oracle.schedule_pass(tasks, queue, budgets, W, CTX, env_limit=int(rng.integers(1, 12)))
        for r, B in enumerate(budgets):
            act = [t for t in tasks if t.state == "active" and t.rank == r]
            assert oracle.token_usage(tasks, r) <= B or len(act) <= 1
            kinds_r = [k for k, _, rr in ev if rr == r and k != "evict"]
            assert kinds_r == sorted(kinds_r, key=lambda k: k != "resume"), "an admit came before a resume"
        for k, tid, r in ev:
            if k == "resume" and tid in home:
                assert home[tid] == r
