"""Oracle for the paper's Algorithm 1, "Semantic-Aware CTB Scheduling" (test infrastructure only).

One scheduling pass, written in the order and notation of the listing: update the token footprints of the
active tasks; then for each rank r, while TokenUsage(r) exceeds the budget B_r preempt the active task of r with
the lowest Priority; while TokenUsage(r) is below B_r resume the paused task with the highest Priority that fits
(enforcing group affinity), otherwise admit a new task by its probed footprint if it satisfies the constraints,
otherwise stop.  Priority is the unnumbered equation of Section 4.2,

    P(t) = w1 * I_eval + w2 * G_completion + w3 * I_active + w4 * L_context .

Readings where the paper is silent (the same ones the product scheduler takes):
  * weights: the paper gives none; the caller passes them (the tests use 8, 4, 2, 1, which reproduces the strict
    tiers of Table 1 because every factor lies in [0, 1]);
  * L_context is the task's current token length divided by `ctx_norm` (so that it lies in [0, 1]);
  * G_completion = finished / total of the task's GRPO group;
  * "fits in B_r": TokenUsage(r) + footprint(t) <= B_r;
  * "enforcing group affinity": a paused task may resume only on the rank it was preempted from (where its
    group's shared prefix lives); a task that never ran has no affinity;
  * new tasks: "admit if it satisfies the constraints" (Section 4.2 lists policy staleness, task diversity and
    environment concurrency).  Environment concurrency: the number of active tasks stays below `env_limit`.
    Policy staleness ("throttles dispatch when Rollout is likely to generate more data than Trainer can consume
    within the staleness bound"): no new task is admitted while the trajectories in flight - active, paused, and
    finished but not yet consumed by the trainer (`unconsumed`, kept by the caller) - reach `inflight_cap`.
    Task diversity ("penalizes assigning too many identical task types to the same batch"): among the first
    `window` queued tasks whose probed footprint fits, the one whose type has the fewest active tasks on this
    rank is admitted, ties in arrival order; window = 1 is plain arrival order;
  * ties in Priority go to the smaller task id;
  * a preempted task loses its KV state (Table 1: evicting long contexts costs a redundant prefill), so its
    footprint no longer counts against any rank.

Everything is plain Python over lists: no heaps, no incremental sums.
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
    """One iteration of the outer loop of Algorithm 1.

    tasks: list of Task (all of them); new_queue: list of task ids in arrival order (state "new");
    budgets: B_r per rank; new_footprints: {task id: tokens} from turn probing.
    Mutates tasks / new_queue and returns the list of decisions, in order:
    ("evict", task, rank) | ("resume", task, rank) | ("admit", task, rank)."""
    by_id = {t.id: t for t in tasks}
    events = []
    # line 2: update token footprint for t in T_act via turn probing
    for tid, tokens in (new_footprints or {}).items():
        if by_id[tid].state == "active":
            by_id[tid].footprint = int(tokens)
    # line 3: for each rank r
    for r, B in enumerate(budgets):
        # lines 4-7: while TokenUsage(r) > B_r: preempt argmin Priority over the active tasks of r
        while token_usage(tasks, r) > B:
            act = [t for t in tasks if t.state == "active" and t.rank == r]
            if not act:
                break
            t_evict = min(act, key=lambda t: (priority(t, tasks, w, ctx_norm), t.id))
            t_evict.state = "paused"
            events.append(("evict", t_evict.id, r))
        # lines 8-18: while TokenUsage(r) < B_r
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
                # line 13: admit a new task if it satisfies the constraints
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
