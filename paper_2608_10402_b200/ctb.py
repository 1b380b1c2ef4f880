"""Host-side Continuous Task Batching: the scheduler of the paper's Algorithm 1 and a small rollout simulator.

`CTBScheduler` keeps, per rollout rank, a token budget and the footprints of the tasks admitted to it, and in
every pass (a) refreshes the footprints of active tasks, (b) preempts the lowest-priority active tasks of a rank
that is over budget, (c) fills headroom by resuming the highest-priority paused task that fits on the rank it
was preempted from, else by admitting the next new task by its probed footprint (Section 4.1, Section 4.2,
Algorithm 1).  Priority is P(t) = w1*I_eval + w2*G_completion + w3*I_active + w4*L_context (Section 4.2).
The paper gives no weights; the defaults (8, 4, 2, 1) make the four terms strict tiers as in its Table 1.

The scheduler talks to a KV backend through three callbacks, which is where the GPU library comes in:
admit(task, rank), preempt(task, rank) (the task's KV state is dropped: tide_kv_release) and resume(task, rank)
(the task must be prefilled again).  Tasks that merely wait for their environment stay active and keep their KV
state — that is the point of task-level batching.

`simulate` replays a synthetic multi-turn rollout (turn counts, observation sizes and environment latencies
drawn from the ranges the paper reports for its workloads) under CTB and under request-level batching with a
fixed concurrency and LRU eviction of idle requests, and reports the KV cache hit rate: the share of context
tokens that did not have to be prefilled again when a turn started.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class CTBTask:
    id: int
    group: int
    is_eval: bool
    probed: int
    kind: int = 0
    footprint: int = 0
    state: str = "new"      # new | active | paused | done
    rank: int = -1


class CTBScheduler:
    def __init__(self, budgets, weights=(8.0, 4.0, 2.0, 1.0), ctx_norm=8192.0, env_limit=1 << 30,
                 on_admit=None, on_preempt=None, on_resume=None, inflight_cap=None, window=1):
        self.budgets = [int(b) for b in budgets]
        self.w_eval, self.w_group, self.w_active, self.w_ctx = (float(x) for x in weights)
        self.ctx_norm = float(ctx_norm)
        self.env_limit = int(env_limit)
        self.tasks = {}                                   # id -> CTBTask
        self.new_queue = []                               # ids, arrival order (consumed from the front)
        self._new_head = 0
        self.active = [dict() for _ in self.budgets]      # per rank: id -> task
        self.paused = {}                                  # id -> task
        self.usage = [0 for _ in self.budgets]            # per rank: sum of active footprints
        self.group_total = {}
        self.group_done = {}
        self.n_active = 0
        # admission constraints of Section 4.2: policy staleness (no new task while active + paused + finished but
        # unconsumed trajectories reach inflight_cap) and task diversity (among the first `window` queued tasks
        # that fit, the type with the fewest active tasks on the rank goes first)
        self.inflight_cap = inflight_cap
        self.window = int(window)
        self.unconsumed = 0
        self.kind_active = [dict() for _ in self.budgets]   # per rank: task type -> active tasks
        self.on_admit, self.on_preempt, self.on_resume = on_admit, on_preempt, on_resume

    # ---- task life cycle ---------------------------------------------------------------------------------
    def submit(self, task_id, group, probed, is_eval=False, kind=0):
        t = CTBTask(int(task_id), int(group), bool(is_eval), int(probed), int(kind))
        self.tasks[t.id] = t
        self.new_queue.append(t.id)
        self.group_total[t.group] = self.group_total.get(t.group, 0) + 1
        self.group_done.setdefault(t.group, 0)
        return t

    def finish(self, task_id):
        t = self.tasks[task_id]
        if t.state == "active":
            del self.active[t.rank][t.id]
            self.usage[t.rank] -= t.footprint
            self.n_active -= 1
            self.kind_active[t.rank][t.kind] -= 1
        elif t.state == "paused":
            del self.paused[t.id]
        t.state = "done"
        self.group_done[t.group] += 1
        self.unconsumed += 1

    def consume(self, n):
        """The trainer took n finished trajectories."""
        self.unconsumed = max(0, self.unconsumed - int(n))

    def priority(self, t: CTBTask) -> float:
        return (self.w_eval * (1.0 if t.is_eval else 0.0)
                + self.w_group * (self.group_done[t.group] / self.group_total[t.group])
                + self.w_active * (1.0 if t.state == "active" else 0.0)
                + self.w_ctx * min(1.0, t.footprint / self.ctx_norm))

    # ---- one pass of Algorithm 1 -------------------------------------------------------------------------
    def schedule(self, new_footprints=None):
        events = []
        for tid, tokens in (new_footprints or {}).items():
            t = self.tasks[tid]
            if t.state == "active":
                self.usage[t.rank] += int(tokens) - t.footprint
                t.footprint = int(tokens)
        for r, B in enumerate(self.budgets):
            act = self.active[r]
            while self.usage[r] > B and act:
                victim = min(act.values(), key=lambda t: (self.priority(t), t.id))
                del act[victim.id]
                self.usage[r] -= victim.footprint
                self.n_active -= 1
                self.kind_active[r][victim.kind] -= 1
                victim.state = "paused"
                self.paused[victim.id] = victim
                events.append(("evict", victim.id, r))
                if self.on_preempt:
                    self.on_preempt(victim, r)
            while self.usage[r] < B:
                room = B - self.usage[r]
                best = None
                if self.n_active < self.env_limit:
                    for t in self.paused.values():
                        if t.rank in (-1, r) and t.footprint <= room:
                            key = (self.priority(t), -t.id)
                            if best is None or key > best[0]:
                                best = (key, t)
                if best is not None:
                    t = best[1]
                    del self.paused[t.id]
                    self._activate(t, r)
                    events.append(("resume", t.id, r))
                    if self.on_resume:
                        self.on_resume(t, r)
                else:
                    pick = self._pick_new(r, room)
                    if pick is None:
                        break
                    t = self.tasks[pick]
                    if pick == self.new_queue[self._new_head]:
                        self._new_head += 1
                    else:
                        self.new_queue.remove(pick)
                    t.footprint = t.probed
                    self._activate(t, r)
                    events.append(("admit", t.id, r))
                    if self.on_admit:
                        self.on_admit(t, r)
        return events

    def _pick_new(self, r, room):
        """The queued task to admit on rank r, or None: constraints of Section 4.2."""
        if self._new_head >= len(self.new_queue) or self.n_active >= self.env_limit:
            return None
        if self.inflight_cap is not None and self.n_active + len(self.paused) + self.unconsumed >= self.inflight_cap:
            return None
        best = None
        for pos in range(self._new_head, min(len(self.new_queue), self._new_head + self.window)):
            tid = self.new_queue[pos]
            t = self.tasks[tid]
            if t.probed <= room:
                key = (self.kind_active[r].get(t.kind, 0), pos)
                if best is None or key < best[0]:
                    best = (key, tid)
        return None if best is None else best[1]

    def _activate(self, t, r):
        t.state = "active"
        t.rank = r
        self.active[r][t.id] = t
        self.usage[r] += t.footprint
        self.n_active += 1
        self.kind_active[r][t.kind] = self.kind_active[r].get(t.kind, 0) + 1

    def pending_new(self):
        return len(self.new_queue) - self._new_head


# ---------------------------------------------------------------------------------------------------------
def synthetic_rollout(rng, n_groups=40, group_size=8, max_turns=20, ctx_cap=8192):
    """Per task: prompt tokens (shared by its group), and per turn (action tokens, observation tokens,
    environment latency in engine steps).  Ranges follow the text workloads of the paper's Appendix C
    (at most 20 turns and 8192 context tokens; a few thousand tokens per trajectory)."""
    tasks = []
    for g in range(n_groups):
        prompt = int(rng.integers(300, 900))
        for _ in range(group_size):
            turns = int(rng.integers(3, max_turns + 1))
            plan, total = [], prompt
            for _t in range(turns):
                act, obs, lat = int(rng.integers(20, 120)), int(rng.integers(50, 600)), int(rng.integers(1, 30))
                if total + act + obs > ctx_cap:
                    break
                plan.append((act, obs, lat))
                total += act + obs
            tasks.append({"group": g, "prompt": prompt, "turns": plan})
    return tasks


def simulate(rollout, policy, budget_tokens, fixed_concurrency=None, weights=(8.0, 4.0, 2.0, 1.0)):
    """Engine-step simulation on one rank.  Returns {"hit_rate", "prefilled", "context", "steps"}.

    policy "ctb": tasks are admitted / preempted / resumed by CTBScheduler against `budget_tokens`; a task that
    waits for its environment stays resident.  policy "request": request-level batching with at most
    `fixed_concurrency` tasks in flight; every turn is a new request whose prefix is reused only if it is still
    cached; idle prefixes are evicted least-recently-used when memory is needed (they are not pinned)."""
    n = len(rollout)
    ctx = [0] * n                  # tokens of the trajectory so far
    resident = [0] * n             # how many of them are still cached
    turn = [0] * n
    new_obs = [0] * n              # observation tokens of the turn that is about to start (new work, not a miss)
    wake = {}                      # task -> step at which its environment answers
    context_tokens = prefilled = 0
    step = 0
    if policy == "ctb":
        def drop(t, r):
            resident[t.id] = 0
        sched = CTBScheduler([budget_tokens], weights=weights, on_preempt=drop)
        for i, t in enumerate(rollout):
            sched.submit(i, t["group"], probed=t["prompt"] + 200)
        started = set()
        while sched.pending_new() or sched.n_active or sched.paused:
            sched.schedule({i: ctx[i] for i in list(sched.active[0])})
            progressed = False
            for i in list(sched.active[0]):
                if wake.get(i, 0) > step:
                    continue                                  # waiting for the environment, KV stays resident
                progressed = True
                t = rollout[i]
                if i not in started:
                    started.add(i)
                    ctx[i] = t["prompt"]
                else:
                    preserved = ctx[i] - new_obs[i]            # what the task had when it paused for its environment
                    context_tokens += preserved
                    prefilled += preserved - min(resident[i], preserved)   # whatever was dropped is prefilled again
                resident[i] = ctx[i]
                if turn[i] >= len(t["turns"]):
                    sched.finish(i)
                    resident[i] = 0
                    continue
                act, obs, lat = t["turns"][turn[i]]
                turn[i] += 1
                ctx[i] += act + obs
                new_obs[i] = obs
                resident[i] = ctx[i] - obs                     # the observation arrives (and is appended) at wake-up
                wake[i] = step + lat
            step += 1
            if not progressed and not sched.active[0] and not sched.pending_new() and sched.paused:
                sched.schedule()
        return {"hit_rate": 1.0 - prefilled / max(1, context_tokens), "prefilled": prefilled,
                "context": context_tokens, "steps": step}
    # ---- request-level batching, fixed concurrency, LRU cache of idle prefixes ----
    assert fixed_concurrency
    queue = list(range(n))
    inflight = set()
    last_used = {}
    started = set()
    while queue or inflight:
        while queue and len(inflight) < fixed_concurrency:
            inflight.add(queue.pop(0))
        for i in sorted(inflight):
            if wake.get(i, 0) > step:
                continue
            t = rollout[i]
            if i not in started:
                started.add(i)
                ctx[i] = t["prompt"]
            else:
                preserved = ctx[i] - new_obs[i]
                context_tokens += preserved
                prefilled += preserved - min(resident[i], preserved)
            resident[i] = ctx[i]
            last_used[i] = step
            if turn[i] >= len(t["turns"]):
                inflight.discard(i)
                resident[i] = 0
                continue
            act, obs, lat = t["turns"][turn[i]]
            turn[i] += 1
            ctx[i] += act + obs
            new_obs[i] = obs
            resident[i] = ctx[i] - obs
            wake[i] = step + lat
            # memory pressure: requests that are running now are safe, idle prefixes go first (LRU)
            while sum(resident) > budget_tokens:
                idle = [j for j in inflight if wake.get(j, 0) > step and resident[j] > 0 and j != i]
                if not idle:
                    break
                victim = min(idle, key=lambda j: (last_used.get(j, -1), j))
                resident[victim] = 0
        step += 1
    return {"hit_rate": 1.0 - prefilled / max(1, context_tokens), "prefilled": prefilled,
            "context": context_tokens, "steps": step}
