"""Oracle for the paper's Algorithm 1, "Semantic-Aware CTB Scheduling" (test infrastructure only).

One scheduling pass in the algorithm's own order of steps and with its names.  First the token footprints of
the active tasks are refreshed from turn probing.  Then every rank r is visited in turn: as long as
TokenUsage(r) is above the budget B_r, the active task of r with the smallest Priority is preempted; after that,
as long as TokenUsage(r) is below B_r, the rank is filled - a paused task that fits goes first (the one with the
largest Priority, subject to group affinity), a new task is admitted by its probed footprint only when no paused
task can be resumed and the admission constraints hold, and the fill loop ends when neither is possible.
Priority is the weighted sum of Section 4.2,

    P(t) = w1 * I_eval + w2 * G_completion + w3 * I_active + w4 * L_context .

Readings where the paper is silent:
  * weights: the paper gives none; the caller passes them (the tests use 8, 4, 2, 1, which gives the strict
    tiers of Table 1 because every factor lies in [0, 1]);
  * L_context is the task's current token length divided by `ctx_norm`, capped at 1;
  * G_completion = finished / total members of the task's GRPO group;
  * a task "fits" when TokenUsage(r) + footprint(t) <= B_r;
  * group affinity: a paused task may resume only on the rank it was preempted from (where its group's shared
    prefix lives); a task that never ran has no affinity;
  * the admission constraints of Section 4.1.  Environment concurrency: the number of active tasks stays below
    `env_limit`, for resumes and admissions alike.  Policy staleness: no new task is admitted while the
    trajectories in flight - active, paused, and finished but not yet taken by the trainer (`unconsumed`, kept by
    the caller) - have reached `inflight_cap`.  Task diversity: among the first `window` queued tasks whose
    probed footprint fits, the one whose type has the fewest active tasks on this rank is admitted, ties in
    arrival order; window = 1 is plain arrival order;
  * ties in Priority go to the smaller task id;
  * a preempted task loses its KV state (Table 1 counts the prefill it will have to repeat as the cost of
    evicting a long context), so its footprint no longer counts against any rank.

Everything is plain Python over lists, recomputed from scratch at every use: no heaps, no running sums.
Pinned in tests/test_ctb_scheduler.py by hand-derived decision lists (tier order, affinity over two ranks,
resume before admit, the three admission constraints) and by the invariants the loop guarantees.
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass
class Task:
    id: int
    group: int
    is_eval: bool
    probed: int                 # footprint estimated by the group's probing task (first turn)
    kind: int = 0               # task type (environment), for the diversity constraint
    footprint: int = 0          # current token length (updated at the start of every interaction turn)
    state: str = "new"          # new | active | paused | done
    rank: int = -1              # rank it runs on (active) / was preempted from (paused)


@dataclass
class Weights:
    eval: float = 8.0
    group: float = 4.0
    active: float = 2.0
    ctx: float = 1.0


def priority(t: Task, tasks, w: Weights, ctx_norm: float) -> float:
    members = [u for u in tasks if u.group == t.group]
    g_completion = sum(1 for u in members if u.state == "done") / len(members)
    return (w.eval * (1.0 if t.is_eval else 0.0) + w.group * g_completion
            + w.active * (1.0 if t.state == "active" else 0.0) + w.ctx * min(1.0, t.footprint / ctx_norm))


def token_usage(tasks, r: int) -> int:
    return sum(t.footprint for t in tasks if t.state == "active" and t.rank == r)


def schedule_pass(tasks, new_queue, budgets, w: Weights, ctx_norm: float, env_limit: int, new_footprints=None,
                  inflight_cap=None, unconsumed: int = 0, window: int = 1):
    """One pass of Algorithm 1 over all ranks.

    tasks: list of Task (all of them); new_queue: list of task ids in arrival order (state "new");
    budgets: B_r per rank; new_footprints: {task id: tokens} from turn probing.
    Mutates tasks / new_queue and returns the list of decisions, in order:
    ("evict", task, rank) | ("resume", task, rank) | ("admit", task, rank)."""
    by_id = {t.id: t for t in tasks}
    events = []
    # refresh the footprints of the active tasks (turn probing)
    for tid, tokens in (new_footprints or {}).items():
        if by_id[tid].state == "active":
            by_id[tid].footprint = int(tokens)
    for r, B in enumerate(budgets):
        # over budget: preempt the active task of this rank with the smallest Priority, one at a time
        while token_usage(tasks, r) > B:
            act = [t for t in tasks if t.state == "active" and t.rank == r]
            if not act:
                break
            t_evict = min(act, key=lambda t: (priority(t, tasks, w, ctx_norm), t.id))
            t_evict.state = "paused"
            events.append(("evict", t_evict.id, r))
        # headroom: resume before admitting, stop when neither is possible
        while token_usage(tasks, r) < B:
            usage = token_usage(tasks, r)
            paused_fit = [t for t in tasks if t.state == "paused" and t.rank in (-1, r) and usage + t.footprint <= B]
            n_active = sum(1 for t in tasks if t.state == "active")
            if paused_fit and n_active < env_limit:
                t_res = max(paused_fit, key=lambda t: (priority(t, tasks, w, ctx_norm), -t.id))
                t_res.state = "active"
                t_res.rank = r
                events.append(("resume", t_res.id, r))
            else:
                # no paused task can run here: a new task, if the admission constraints allow one
                in_flight = sum(1 for t in tasks if t.state in ("active", "paused")) + unconsumed
                fits = [tid for tid in new_queue[:window] if usage + by_id[tid].probed <= B]
                if fits and n_active < env_limit and (inflight_cap is None or in_flight < inflight_cap):
                    def same_kind_active(tid):
                        return sum(1 for t in tasks if t.state == "active" and t.rank == r and t.kind == by_id[tid].kind)
                    pick = min(fits, key=lambda tid: (same_kind_active(tid), new_queue.index(tid)))
                    new_queue.remove(pick)
                    t_new = by_id[pick]
                    t_new.state = "active"
                    t_new.rank = r
                    t_new.footprint = t_new.probed
                    events.append(("admit", t_new.id, r))
                else:
                    break
    return events
