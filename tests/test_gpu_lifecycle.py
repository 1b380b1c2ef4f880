"""Multi-turn rollout replay on the GPU against the oracle: the lifecycle a CTB rank drives around the hot path
(paper Section 3.2 / Section 4 / Section 5.2 / Appendix C.2): admit a task and prefill its prompt from scratch
(a row with no preserved prefix), decode, pause for the environment, resume with observation tokens, prune old
observations with a sliding window, release finished groups, and flush everything at a weight synchronisation
before the next training step.  After every call the bookkeeping is compared bit for bit and every attention
result is compared with the float64 oracle."""
import math

import numpy as np
import pytest

from oracle import cbuild
from oracle.paged_kv import PagedKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

HQ, HKV, D, S = 28, 4, 128, 16
MAX_TASKS, MAX_PAGES, NUM_PAGES = 24, 160, 900


def test_multi_turn_replay_with_prune_release_and_reset():
    import torch
    from paper_2608_10402_b200 import tide

    rng = np.random.default_rng(2024)
    scale = 1.0 / math.sqrt(D)
    order = rng.permutation(NUM_PAGES).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, NUM_PAGES, MAX_TASKS, MAX_PAGES, MAX_TASKS, 4096, free_order=order)
    orc = PagedKVOracle(NUM_PAGES, S, HKV, D, MAX_TASKS, MAX_PAGES, free_order=order)

    def same_state(tasks):
        for t in tasks:
            assert kv.task_len(t) == orc.task_len(t)
            assert np.array_equal(kv.page_table(t), orc.page_table(t)), f"page table of task {t}"
        assert kv.usage() == (orc.used_tokens(), orc.free_pages())

    def same_bits(t):
        gk, gv = kv.read(t)
        ok, ov = orc.read(t)
        assert np.array_equal(H.from_dev(gk), ok) and np.array_equal(H.from_dev(gv), ov), f"cache bits of task {t}"

    def step(active, n_new):
        """append n_new[t] tokens to every active task and attend; checked against the oracle"""
        ids = list(active)
        cnt = [int(n_new[t]) for t in ids]
        indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
        total = int(indptr[-1])
        nk, nv = inputs.normal_bf16(rng, (total, HKV, D)), inputs.normal_bf16(rng, (total, HKV, D))
        q = inputs.normal_bf16(rng, (total, HQ, D))
        kv.append(ids, indptr, H.to_dev(nk, torch), H.to_dev(nv, torch))
        orc.append(ids, indptr, nk, nv)
        rows = [(t, c, orc.task_len(t)) for t, c in zip(ids, cnt)]
        out = torch.zeros((total, HQ, D), dtype=torch.int16, device="cuda")
        lse = torch.zeros((total, HQ), dtype=torch.float32, device="cuda")
        kv.attend(rows, H.to_dev(q, torch), scale, out, lse)
        assert kv.status() == tide.OK
        ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
        H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, "replay step")
        same_state(ids)

    for training_step in range(2):
        # ---- admission: every task prefills its prompt from scratch (q_len = ctx_len, no preserved prefix) ----
        tasks = list(range(8 * training_step, 8 * training_step + 8))
        for t in tasks:
            kv.alloc(t, 64)
            orc.alloc(t, 64)
        step(tasks, {t: int(rng.integers(40, 300)) for t in tasks})
        active = set(tasks)
        for turn in range(4):
            # a few decode steps (the action), every active task appends one token per step
            for _ in range(3):
                step(sorted(active), {t: 1 for t in active})
            # the environment answers for most tasks; the rest stay paused with their KV resident
            resumed = sorted(t for t in active if rng.random() < 0.75)
            if resumed:
                obs = {t: int(rng.integers(20, 400)) for t in resumed}   # mixes decode-style, tile and tcgen05 paths
                step(resumed, obs)
            # sliding window: drop an old observation from the middle of two trajectories
            for t in sorted(active)[:2]:
                L = orc.task_len(t)
                keep, tail = int(rng.integers(10, L // 3)), int(rng.integers(L // 3, L - 5))
                kv.prune(t, keep, tail)
                orc.prune(t, keep, tail)
                same_state([t])
                same_bits(t)
            # one trajectory of the group finishes and leaves
            if turn == 2:
                done = sorted(active)[-2:]
                kv.release_many(done)
                orc.release_many(done)
                active -= set(done)
                same_state(sorted(active))
        # a pruned task still attends correctly (its moved tail is what the oracle holds)
        step(sorted(active), {t: 5 for t in active})
        for t in sorted(active)[:3]:
            same_bits(t)
        # ---- weight synchronisation: all rollout KV is invalid ----
        new_order = rng.permutation(NUM_PAGES).astype(np.int32)
        kv.reset(new_order)
        orc.reset(new_order)
        assert kv.usage() == (0, NUM_PAGES)
        with pytest.raises(tide.TideError) as e:
            kv.task_len(tasks[0])
        assert e.value.code == tide.ERR_UNKNOWN_TASK
    kv.close()
