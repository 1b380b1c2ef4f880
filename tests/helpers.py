"""Shared helpers of the parity tests: drive the oracle and the CUDA library with the same bits."""
from __future__ import annotations

import numpy as np

from oracle import attention as oa
from oracle import cbuild
from oracle.paged_kv import PagedKVOracle

ATOL, RTOL, LSE_TOL, REL_FRO_MAX = 1e-2, 1e-2, 1e-3, 5e-3


def oracle_fill(w, kv_bits):
    """Oracle cache after every task's prefix was appended (one call per task, batch order) and then the
    step's new tokens were appended in ONE call."""
    c = PagedKVOracle(w.num_pages, w.S, w.Hkv, w.D, w.max_tasks, w.max_pages_per_task, free_order=w.free_order)
    for b in range(w.B):
        c.alloc(int(w.task[b]))
    for b in range(w.B):
        p = int(w.prefix[b])
        c.append([int(w.task[b])], [0, p], kv_bits[b][0][:p], kv_bits[b][1][:p])
    indptr = np.concatenate([[0], np.cumsum(w.n_new)])
    nk = np.concatenate([kv_bits[b][0][int(w.prefix[b]):] for b in range(w.B)])
    nv = np.concatenate([kv_bits[b][1][int(w.prefix[b]):] for b in range(w.B)])
    c.append([int(t) for t in w.task], indptr, nk, nv)
    return c, indptr, nk, nv


def to_dev(bits, torch):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()


def from_dev(t):
    return t.cpu().numpy().view(np.uint16)


def gpu_fill(w, kv_bits, nk, nv, indptr, tide, torch, max_batch_tokens=None, tune=()):
    """The same sequence of calls on the CUDA library."""
    total_q = int(w.n_new.sum())
    kv = tide.TideKV(w.Hq, w.Hkv, w.D, w.S, w.num_pages, w.max_tasks, w.max_pages_per_task,
                     max_batch_rows=max(w.B, 1), max_batch_tokens=max_batch_tokens or max(total_q, 1),
                     free_order=w.free_order)
    for knob, value in tune:
        kv.tune(knob, value)
    for b in range(w.B):
        kv.alloc(int(w.task[b]))
    for b in range(w.B):
        p = int(w.prefix[b])
        kv.append([int(w.task[b])], [0, p], to_dev(kv_bits[b][0][:p], torch), to_dev(kv_bits[b][1][:p], torch))
    kv.append([int(t) for t in w.task], indptr, to_dev(nk, torch), to_dev(nv, torch))
    return kv


def compare_bookkeeping(w, c, kv):
    for b in range(w.B):
        t = int(w.task[b])
        assert kv.task_len(t) == c.task_len(t)
        assert np.array_equal(kv.page_table(t), c.page_table(t)), f"page table of task {t}"
    used, free = kv.usage()
    assert used == c.used_tokens() and free == c.free_pages()


def compare_cache(w, c, kv, tasks=None):
    for b in (range(w.B) if tasks is None else tasks):
        t = int(w.task[b])
        gk, gv = kv.read(t)
        ok, ov = c.read(t)
        assert np.array_equal(from_dev(gk), ok), f"K bits of task {t}"
        assert np.array_equal(from_dev(gv), ov), f"V bits of task {t}"


def check_outputs(got_bits, got_lse, ref_o, ref_lse, what=""):
    """Elementwise |gpu - oracle| <= 1e-2 + 1e-2 |oracle|, LSE within 1e-3, relative Frobenius error <= 5e-3."""
    got = oa.bf16_bits_to_f64(got_bits)
    err = np.abs(got - ref_o)
    bound = ATOL + RTOL * np.abs(ref_o)
    worst = float((err / bound).max()) if err.size else 0.0
    rel_fro = float(np.linalg.norm(got - ref_o) / max(np.linalg.norm(ref_o), 1e-300)) if err.size else 0.0
    lse_err = float(np.abs(got_lse.astype(np.float64) - ref_lse).max()) if ref_lse.size else 0.0
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert worst <= 1.0, f"{what}: worst error/tolerance {worst:.3f}, max abs err {err.max():.3e}"
    assert lse_err <= LSE_TOL, f"{what}: LSE error {lse_err:.3e}"
    assert rel_fro <= REL_FRO_MAX, f"{what}: relative Frobenius error {rel_fro:.3e}"
    return {"worst_ratio": worst, "max_abs": float(err.max()) if err.size else 0.0, "rel_fro": rel_fro, "lse_err": lse_err}


def oracle_attend(c, w, q_bits, items=None):
    return cbuild.attend_paged(c, w.rows(), q_bits, w.scale, items=items)


def sample_items(w, rng, per_row=6):
    """A stratified sample of (row, query index): first / last of the chunk, page boundaries, the image/text
    boundary and a few random positions; every decode row's single query."""
    items = []
    for b in range(w.B):
        n, p = int(w.n_new[b]), int(w.prefix[b])
        if n == 1:
            items.append((b, 0))
            continue
        picks = {0, n - 1, n // 2}
        first_page_edge = (-p) % w.S                      # query whose position is slot 0 of a page
        if first_page_edge < n:
            picks.add(first_page_edge)
            if first_page_edge > 0:
                picks.add(first_page_edge - 1)
        ni = int(w.n_image[b])
        if 0 < ni < n:
            picks.update({ni - 1, ni})
        picks.update(int(x) for x in rng.integers(0, n, size=per_row))
        items.extend((b, i) for i in sorted(picks))
    return items
