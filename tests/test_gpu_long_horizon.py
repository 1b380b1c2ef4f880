"""Long-horizon stress (configs[4]): a pool that holds the KV of ALL resident tasks, most of them paused, with
pages freed and re-used between steps (tide_kv_release, then appends of newly admitted tasks).

The pool is sized by TIDE_STRESS_POOL_GB (default 16 so that the routine run stays short; the workload is quoted
at ~150 GB, which the same test runs when the variable says so).  A resident population is drawn from the
Pareto(1.5) length law until ~90 % of the pages are in use; every step batches 256 residents (230 decode rows,
26 resume rows appending 500..4000 tokens), then releases 10 % of the batch and admits as many new tasks.
Checked against the oracle on every step: page tables, lengths, free-page count (bit-exact, oracle run without
values), cache bits of sampled paused and active residents (values are a reproducible integer hash), and
attention outputs of sampled rows."""
import json
import math
import os
import time

import numpy as np
import pytest

from oracle import cbuild
from oracle.paged_kv import PagedKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

HQ, HKV, D, S = 28, 4, 128, 32
XM, CAP = 1024, 128 * 1024
STEPS = 8


def _hash_kv_np(task, start, count):
    return (inputs.hashed_bf16_bits(task, start, count, HKV, D, 0), inputs.hashed_bf16_bits(task, start, count, HKV, D, 1))


def _hash_kv_dev(torch, task, start, count):
    return (inputs.hashed_bf16_bits_torch(torch, task, start, count, HKV, D, 0),
            inputs.hashed_bf16_bits_torch(torch, task, start, count, HKV, D, 1))


def test_long_horizon_release_and_reuse():
    import torch
    from paper_2608_10402_b200 import tide

    pool_gb = float(os.environ.get("TIDE_STRESS_POOL_GB", "16"))
    free_b, _ = torch.cuda.mem_get_info()
    page_bytes = HKV * 2 * D * S * 2
    num_pages = int(min(pool_gb * 1e9, 0.85 * free_b - 6e9) // page_bytes)
    assert num_pages > 4096
    rng = np.random.default_rng(1005)
    # ---- resident population: Pareto lengths until ~90 % of the pages are used ----
    lens = []
    used = 0
    while True:
        L = int(np.clip(round(XM * (1.0 - rng.random()) ** (-1.0 / 1.5)), XM, CAP))
        if not lens:
            L = CAP                                            # always exercise the longest context
        pages = -(-L // S)
        if used + pages > 0.9 * num_pages:
            break
        lens.append(L)
        used += pages
    n_res = len(lens)
    assert n_res >= 256, "pool too small for a 256-row batch"
    max_tasks = n_res + STEPS * 32 + 8
    max_pages_per_task = -(-(CAP + 4000 + STEPS) // S) + 1
    max_batch_tokens = 230 + 26 * 4000
    free_order = rng.permutation(num_pages).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, num_pages, max_tasks, max_pages_per_task, 256, max_batch_tokens, free_order=free_order)
    orc = PagedKVOracle(num_pages, S, HKV, D, max_tasks, max_pages_per_task, free_order=free_order, store_values=False)

    def admit(task, L):
        kv.alloc(task, L)
        orc.alloc(task, L)
        k, v = _hash_kv_dev(torch, task, 0, L)
        kv.append([task], [0, L], k, v)
        orc.append([task], [0, L])

    t0 = time.time()
    length = {}
    for t, L in enumerate(lens):
        admit(t, L)
        length[t] = L
    torch.cuda.synchronize()
    fill_s = time.time() - t0
    next_task = n_res
    scale = 1.0 / math.sqrt(D)
    report = {"pool_gb": num_pages * page_bytes / 1e9, "num_pages": num_pages, "residents": n_res, "fill_seconds": fill_s, "steps": []}

    def check_bits(task):
        gk, gv = kv.read(task)
        ek, ev = _hash_kv_np(task, 0, length[task])
        assert np.array_equal(H.from_dev(gk), ek) and np.array_equal(H.from_dev(gv), ev), f"cache bits of task {task}"

    for step in range(STEPS):
        live = np.array(sorted(length))
        batch = rng.choice(live, size=256, replace=False)
        n_new = np.concatenate([np.ones(230, np.int64), rng.integers(500, 4001, size=26)])
        n_new = n_new[rng.permutation(256)]
        # a row must keep its table within bounds
        n_new = np.array([min(int(n), max_pages_per_task * S - length[int(t)]) for t, n in zip(batch, n_new)])
        indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
        total = int(indptr[-1])
        nk = torch.empty((total, HKV, D), dtype=torch.int16, device="cuda")
        nv = torch.empty_like(nk)
        for j, (t, n) in enumerate(zip(batch, n_new)):
            a, b = _hash_kv_dev(torch, int(t), length[int(t)], int(n))
            nk[indptr[j]:indptr[j + 1]], nv[indptr[j]:indptr[j + 1]] = a, b
        q_bits = inputs.normal_bf16(rng, (total, HQ, D))
        q = H.to_dev(q_bits, torch)
        out = torch.zeros((total, HQ, D), dtype=torch.int16, device="cuda")
        lse = torch.zeros((total, HQ), dtype=torch.float32, device="cuda")
        rows = [(int(t), int(n), length[int(t)] + int(n)) for t, n in zip(batch, n_new)]
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        kv.append([int(t) for t in batch], indptr, nk, nv)
        kv.attend(rows, q, scale, out, lse)
        e1.record()
        torch.cuda.synchronize()
        assert kv.status() == tide.OK
        orc.append([int(t) for t in batch], indptr)
        for t, n in zip(batch, n_new):
            length[int(t)] += int(n)
        # ---- bookkeeping, bit-exact, for every row of the batch ----
        for t in batch:
            assert kv.task_len(int(t)) == orc.task_len(int(t))
            assert np.array_equal(kv.page_table(int(t)), orc.page_table(int(t)))
        assert kv.usage() == (orc.used_tokens(), orc.free_pages())
        # ---- cache bits of a few paused residents and a few rows of the batch ----
        paused = np.setdiff1d(live, batch)
        for t in list(rng.choice(paused, size=3, replace=False)) + list(batch[:2]):
            if length[int(t)] <= 40000:
                check_bits(int(t))
        # ---- attention of sampled rows against the float64 oracle ----
        picks = [j for j in range(256) if n_new[j] == 1][:3] + [j for j in range(256) if n_new[j] > 1][:1]
        small_pages = sum(-(-rows[j][2] // S) for j in picks) + 2
        val = PagedKVOracle(small_pages, S, HKV, D, len(picks), max_pages_per_task)
        srows, sq, items, idx = [], [], [], []
        for r, j in enumerate(picks):
            t, n, L = rows[j]
            k, v = _hash_kv_np(t, 0, L)
            val.alloc(r)
            val.append([r], [0, L], k, v)
            srows.append((r, n, L))
            sq.append(q_bits[indptr[j]:indptr[j + 1]])
            qs = [0] if n == 1 else sorted({0, n - 1, n // 2, int(rng.integers(0, n))})
            items.extend((r, i) for i in qs)
            idx.extend(int(indptr[j]) + i for i in qs)
        ref_o, ref_l = cbuild.attend_paged(val, srows, np.concatenate(sq), scale, items=items)
        got_o, got_l = H.from_dev(out), lse.cpu().numpy()
        stats = H.check_outputs(got_o[idx], got_l[idx], ref_o, ref_l, f"long-horizon step {step}")
        dec_bytes = HKV * D * 4 * sum(r[2] for r in rows if r[1] == 1)
        pairs = sum(r[1] * (r[2] - r[1]) + r[1] * (r[1] + 1) // 2 for r in rows if r[1] > 1)
        report["steps"].append({"ms": e0.elapsed_time(e1), "new_tokens": total, "decode_kv_gb": dec_bytes / 1e9,
                                "resume_tflop": 4 * D * HQ * pairs / 1e12, "free_pages": kv.usage()[1], **stats})
        # ---- release 10 % of the batch, admit as many new tasks: their pages are re-used at once ----
        leaving = rng.choice(batch, size=26, replace=False)
        freed = set()
        for t in leaving:
            freed.update(int(p) for p in orc.page_table(int(t)))
            kv.release(int(t))
            orc.release(int(t))
            del length[int(t)]
        reused = 0
        for _ in range(26):
            L = int(np.clip(round(XM * (1.0 - rng.random()) ** (-1.0 / 1.5)), XM, CAP))
            if -(-L // S) > orc.free_pages():
                continue
            admit(next_task, L)
            length[next_task] = L
            assert np.array_equal(kv.page_table(next_task), orc.page_table(next_task))
            reused += len(freed & set(int(p) for p in orc.page_table(next_task)))
            next_task += 1
        assert reused > 0, "released pages were not handed out again"
        assert kv.usage() == (orc.used_tokens(), orc.free_pages())
    out_dir = os.environ.get("TIDE_REPORT_DIR", "")
    if out_dir and os.path.isdir(out_dir):
        with open(os.path.join(out_dir, f"long_horizon_{int(report['pool_gb'])}gb.json"), "w") as f:
            json.dump(report, f, indent=1)
    print(json.dumps({k: v for k, v in report.items() if k != "steps"}), [round(s["ms"], 3) for s in report["steps"]])
    kv.close()
