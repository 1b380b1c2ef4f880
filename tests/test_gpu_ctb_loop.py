"""The scheduler of Algorithm 1 driving the GPU library on one rank with a tight token budget: tasks that wait
for their environment keep their KV state and resume by appending (tide_kv_append), tasks the scheduler preempts
lose it (tide_kv_release) and are prefilled again when they resume.  Either way the attention output of a turn
must equal attention over the task's whole token history computed from scratch by the float64 oracle — the
CTB invariant (recomputing the history is pure redundancy) observed at system level."""
import math

import numpy as np
import pytest

from oracle import attention as oa
from paper_2608_10402_b200 import ctb, inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

HQ, HKV, D, S = 28, 4, 128, 16


def test_scheduler_drives_the_cache_and_results_do_not_depend_on_residency():
    import torch
    from paper_2608_10402_b200 import tide

    rng = np.random.default_rng(42)
    n_tasks, scale = 12, 1.0 / math.sqrt(D)
    # per task: the whole trajectory's K/V/Q bits are fixed up front, so a re-prefill replays identical tokens
    plans = []
    for i in range(n_tasks):
        turns = [(int(rng.integers(2, 6)), int(rng.integers(30, 160)), int(rng.integers(1, 6))) for _ in range(int(rng.integers(2, 5)))]
        total = 120 + sum(a + o for a, o, _ in turns)
        plans.append({"prompt": 120, "turns": turns,
                      "k": inputs.normal_bf16(rng, (total, HKV, D)), "v": inputs.normal_bf16(rng, (total, HKV, D)),
                      "q": inputs.normal_bf16(rng, (total, HQ, D))})
    kv = tide.TideKV(HQ, HKV, D, S, 400, n_tasks, 64, n_tasks, 2048, free_order=rng.permutation(400))
    resident = [False] * n_tasks
    stats = {"appended": 0, "reprefilled": 0, "evictions": 0}

    def on_preempt(t, r):
        if resident[t.id]:
            kv.release(t.id)
            resident[t.id] = False
        stats["evictions"] += 1

    sched = ctb.CTBScheduler([1500], ctx_norm=1024.0, on_preempt=on_preempt)     # room for ~4 trajectories
    for i in range(n_tasks):
        sched.submit(i, group=i // 4, probed=150)
    ctx, done_ctx, turn, wake, step = [0] * n_tasks, [0] * n_tasks, [0] * n_tasks, {}, 0
    while sched.pending_new() or sched.n_active or sched.paused:
        sched.schedule({i: max(ctx[i], 1) for i in list(sched.active[0])})
        rows, qs, checks, ids, cnts, ks, vs = [], [], [], [], [], [], []
        for i in sorted(sched.active[0]):
            if wake.get(i, 0) > step:
                continue
            p = plans[i]
            if turn[i] > len(p["turns"]):
                continue
            # tokens the task has produced / received so far
            target = p["prompt"] + sum(a + o for a, o, _ in p["turns"][:turn[i]])
            if not resident[i]:
                kv.alloc(i)
                resident[i] = True
                lo = 0                                        # nothing preserved: prefill the whole history again
                stats["reprefilled"] += done_ctx[i]
            else:
                lo = done_ctx[i]                              # preserved state: append only what is new
                stats["appended"] += target - lo
            ids.append(i); cnts.append(target - lo)
            ks.append(p["k"][lo:target]); vs.append(p["v"][lo:target]); qs.append(p["q"][lo:target])
            rows.append((i, target - lo, target))
            checks.append((i, lo, target))
            ctx[i] = done_ctx[i] = target
        if rows:
            indptr = np.concatenate([[0], np.cumsum(cnts)]).astype(np.int32)
            kv.append(ids, indptr, H.to_dev(np.concatenate(ks), torch), H.to_dev(np.concatenate(vs), torch))
            T = int(indptr[-1])
            out = torch.zeros((T, HQ, D), dtype=torch.int16, device="cuda")
            lse = torch.zeros((T, HQ), dtype=torch.float32, device="cuda")
            kv.attend(rows, H.to_dev(np.concatenate(qs), torch), scale, out, lse)
            assert kv.status() == tide.OK
            got_o, got_l = H.from_dev(out), lse.cpu().numpy()
            for (i, lo, target), a, b in zip(checks, indptr[:-1], indptr[1:]):
                p = plans[i]
                ref_o, ref_l = oa.attend_contiguous(p["q"][lo:target], p["k"][:target], p["v"][:target], scale)
                H.check_outputs(got_o[a:b], got_l[a:b], ref_o, ref_l, f"task {i} step {step}")
        for (i, lo, target) in checks:
            p = plans[i]
            if turn[i] == len(p["turns"]):
                sched.finish(i)
                kv.release(i)
                resident[i] = False
                turn[i] += 1
            else:
                wake[i] = step + p["turns"][turn[i]][2]
                turn[i] += 1
        step += 1
        assert step < 2000
    assert stats["evictions"] > 0 and stats["reprefilled"] > 0 and stats["appended"] > 0, stats
    assert kv.usage() == (0, 400)
    kv.close()
