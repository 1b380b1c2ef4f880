"""Pins for the oracle's attention (numpy float64 and plain C), CPU only.

Each test checks the oracle against something other than itself: scalar brute
force, closed forms, invariants the method fixes (paged = contiguous, page
permutation, resume-from-cache = recompute-from-scratch, split-merge =
unsplit), or a library softmax restricted to a special case.
"""
import math

import numpy as np
import pytest
import torch

from oracle import attention as oa
from oracle import cbuild
from oracle.paged_kv import PagedKVOracle
from paper_2608_10402_b200 import inputs


def bits(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rand_bits(rng, shape, sigma=1.0):
    return inputs.normal_bf16(rng, shape, sigma)


def test_bf16_widening_is_exact():
    for val, pattern in [(1.0, 0x3F80), (-2.0, 0xC000), (0.5, 0x3F00), (0.0, 0x0000), (1.5, 0x3FC0)]:
        assert oa.bf16_bits_to_f64(np.array([pattern], np.uint16))[0] == val
    allb = np.arange(65536, dtype=np.uint16)
    ref = torch.from_numpy(allb.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    got = oa.bf16_bits_to_f64(allb)
    ok = np.isfinite(ref)
    assert np.array_equal(got[ok], ref[ok])


def test_worked_example_closed_form():
    # D=2, scale=1, prefix 1, chunk 2, one head; every input exact in bf16.
    q = bits([[[1, 0]], [[1, 0]]])                      # [n=2, Hq=1, D=2]
    k = bits([[[0, 0]], [[1, 0]], [[2, 0]]])            # logits 0, 1, 2
    v = bits([[[1, 0]], [[0, 1]], [[1, 1]]])
    o, lse = oa.attend_contiguous(q, k, v, 1.0)
    e = math.e
    w0 = np.array([1, e]) / (1 + e)
    w1 = np.array([1, e, e * e]) / (1 + e + e * e)
    assert np.allclose(o[0, 0], [w0[0], w0[1]], atol=1e-14)               # keys 0..1 only
    assert np.allclose(o[1, 0], [w1[0] + w1[2], w1[1] + w1[2]], atol=1e-14)
    assert abs(lse[0, 0] - math.log(1 + e)) < 1e-14
    assert abs(lse[1, 0] - math.log(1 + e + e * e)) < 1e-14
    # printed to six places for a reader: 0.268941 / 0.731059 ; 0.755272 / 0.909969 ; 1.313262 ; 2.407606
    assert np.allclose(o[0, 0], [0.268941, 0.731059], atol=1e-6)
    assert np.allclose(o[1, 0], [0.755272, 0.909969], atol=1e-6)
    assert abs(lse[0, 0] - 1.313262) < 1e-6 and abs(lse[1, 0] - 2.407606) < 1e-6


@pytest.mark.parametrize("n,L,Hq,Hkv,D", [(1, 5, 2, 1, 4), (3, 7, 4, 2, 4), (4, 4, 6, 2, 3), (2, 8, 3, 3, 2)])
def test_bruteforce_on_tiny_inputs(n, L, Hq, Hkv, D):
    rng = np.random.default_rng(n * 100 + L)
    q, k, v = rand_bits(rng, (n, Hq, D)), rand_bits(rng, (L, Hkv, D)), rand_bits(rng, (L, Hkv, D))
    o, lse = oa.attend_contiguous(q, k, v, 0.37)
    bo, bl = oa.attend_bruteforce(oa.bf16_bits_to_f64(q), oa.bf16_bits_to_f64(k), oa.bf16_bits_to_f64(v), 0.37)
    assert np.allclose(o, np.array(bo), rtol=0, atol=1e-13)
    assert np.allclose(lse, np.array(bl), rtol=0, atol=1e-13)


def test_gqa_head_mapping_consecutive_heads_share_a_kv_head():
    # V of KV head g is the constant g+1, so query head h must return (h // G) + 1.
    rng = np.random.default_rng(0)
    Hq, Hkv, D, L = 6, 3, 4, 9
    q, k = rand_bits(rng, (2, Hq, D)), rand_bits(rng, (L, Hkv, D))
    v = bits(np.broadcast_to(np.arange(1, Hkv + 1, dtype=np.float32)[None, :, None], (L, Hkv, D)))
    o, _ = oa.attend_contiguous(q, k, v, 0.5)
    for h in range(Hq):
        assert np.allclose(o[:, h, :], h // 2 + 1, atol=1e-14)


def test_zero_query_gives_log_count_and_running_mean():
    # Q = 0: every visible key weighs the same, so LSE = ln(#visible) and O = mean of visible V.
    rng = np.random.default_rng(1)
    n, L, D = 5, 12, 4
    p = L - n
    q = np.zeros((n, 2, D), np.uint16)
    k, v = rand_bits(rng, (L, 1, D)), rand_bits(rng, (L, 1, D))
    o, lse = oa.attend_contiguous(q, k, v, 0.7)
    vf = oa.bf16_bits_to_f64(v)[:, 0, :]
    for i in range(n):
        assert abs(lse[i, 0] - math.log(p + i + 1)) < 1e-14
        assert np.allclose(o[i, 1], vf[: p + i + 1].mean(axis=0), atol=1e-14)


def test_single_key_duplicate_keys_and_needle():
    rng = np.random.default_rng(2)
    D = 8
    q, k, v = rand_bits(rng, (1, 1, D)), rand_bits(rng, (6, 1, D)), rand_bits(rng, (6, 1, D))
    # single key: O = V_0, LSE = s_0
    o, lse = oa.attend_contiguous(q, k[:1], v[:1], 0.25)
    s0 = 0.25 * float(oa.bf16_bits_to_f64(q)[0, 0] @ oa.bf16_bits_to_f64(k)[0, 0])
    assert np.allclose(o[0, 0], oa.bf16_bits_to_f64(v)[0, 0], atol=1e-15) and abs(lse[0, 0] - s0) < 1e-15
    # duplicating every key: same O, LSE + ln 2
    o1, l1 = oa.attend_contiguous(q, k, v, 0.25)
    o2, l2 = oa.attend_contiguous(q, np.concatenate([k, k]), np.concatenate([v, v]), 0.25)
    assert np.allclose(o1, o2, atol=1e-14) and abs(l2[0, 0] - l1[0, 0] - math.log(2)) < 1e-14
    # permuting the keys of a decode row: same result
    perm = rng.permutation(6)
    o3, l3 = oa.attend_contiguous(q, k[perm], v[perm], 0.25)
    assert np.allclose(o1, o3, atol=1e-14) and abs(l3[0, 0] - l1[0, 0]) < 1e-14
    # one dominant key (logit gap >= 40): O ~ V_j
    qn = bits(np.full((1, 1, D), 4.0))
    kn = np.zeros((20, 1, D), np.uint16)
    kn[13] = bits(np.full((1, D), 4.0))          # logit 4*4*8 = 128 against 0
    vn = rand_bits(rng, (20, 1, D))
    o4, _ = oa.attend_contiguous(qn, kn, vn, 1.0)
    assert np.allclose(o4[0, 0], oa.bf16_bits_to_f64(vn)[13, 0], atol=1e-12)


def test_constant_v_rows_return_that_constant():
    rng = np.random.default_rng(3)
    q, k = rand_bits(rng, (3, 4, 8)), rand_bits(rng, (10, 2, 8))
    v = bits(np.full((10, 2, 8), -1.25))
    o, _ = oa.attend_contiguous(q, k, v, 0.3)
    assert np.allclose(o, -1.25, atol=1e-14)


def test_against_library_softmax_with_explicit_mask():
    # second opinion from a library routine: torch float64 softmax over an explicitly built mask
    rng = np.random.default_rng(4)
    n, L, Hq, Hkv, D = 6, 19, 4, 2, 8
    q, k, v = rand_bits(rng, (n, Hq, D)), rand_bits(rng, (L, Hkv, D)), rand_bits(rng, (L, Hkv, D))
    o, lse = oa.attend_contiguous(q, k, v, 0.2)
    tq = torch.from_numpy(oa.bf16_bits_to_f64(q)).permute(1, 0, 2)                       # [Hq, n, D]
    tk = torch.from_numpy(oa.bf16_bits_to_f64(k)).permute(1, 0, 2).repeat_interleave(2, 0)  # [Hq, L, D]
    tv = torch.from_numpy(oa.bf16_bits_to_f64(v)).permute(1, 0, 2).repeat_interleave(2, 0)
    mask = torch.full((n, L), float("-inf"), dtype=torch.float64)
    for i in range(n):
        mask[i, : L - n + i + 1] = 0.0
    logits = 0.2 * tq @ tk.transpose(1, 2) + mask
    ref_o = (torch.softmax(logits, dim=-1) @ tv).permute(1, 0, 2).numpy()
    ref_l = torch.logsumexp(logits, dim=-1).permute(1, 0).numpy()
    assert np.allclose(o, ref_o, atol=1e-13) and np.allclose(lse, ref_l, atol=1e-13)


def _fill_cache(w, free_order=None, chunks=None):
    """Build a PagedKVOracle holding every task of workload w (prefix and appended chunk)."""
    c = PagedKVOracle(w.num_pages, w.S, w.Hkv, w.D, w.max_tasks, w.max_pages_per_task,
                      free_order=w.free_order if free_order is None else free_order)
    kv = [w.task_kv(b) for b in range(w.B)]
    for b in range(w.B):
        c.alloc(int(w.task[b]))
    # preserved prefixes first (turn by turn if chunks is given), then ONE append call with every row's new tokens
    for b in range(w.B):
        p = int(w.prefix[b])
        cuts = [0, p] if chunks is None else sorted({0, p, *[x for x in chunks if x < p]})
        for a, z in zip(cuts[:-1], cuts[1:]):
            c.append([int(w.task[b])], [0, z - a], kv[b][0][a:z], kv[b][1][a:z])
    indptr = np.concatenate([[0], np.cumsum(w.n_new)])
    nk = np.concatenate([kv[b][0][int(w.prefix[b]):] for b in range(w.B)])
    nv = np.concatenate([kv[b][1][int(w.prefix[b]):] for b in range(w.B)])
    c.append([int(t) for t in w.task], indptr, nk, nv)
    return c, kv


def test_paged_equals_contiguous_and_page_permutation_invariance():
    w = inputs.make_workload(1, len_div=4)
    c, kv = _fill_cache(w)
    q = np.concatenate([w.task_q(b) for b in range(w.B)])
    o, lse = oa.attend(c, w.rows(), q, w.scale)
    off = 0
    for b in range(w.B):
        n = int(w.n_new[b])
        ro, rl = oa.attend_contiguous(q[off:off + n], kv[b][0], kv[b][1], w.scale)
        assert np.array_equal(o[off:off + n], ro) and np.array_equal(lse[off:off + n], rl)
        off += n
    other = np.random.default_rng(99).permutation(w.num_pages)
    c2, _ = _fill_cache(w, free_order=other, chunks=[5, 16, 17, 40])
    assert any(list(c.page_table(t)) != list(c2.page_table(t)) for t in range(w.B))
    o2, lse2 = oa.attend(c2, w.rows(), q, w.scale)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)


def test_ctb_invariant_resume_equals_recompute_from_scratch():
    # The resumed chunk's outputs, computed from the preserved cache, equal the last n rows of a
    # from-scratch causal pass over the whole sequence (q_len = ctx_len): recomputation is pure redundancy.
    w = inputs.make_workload(1, len_div=4)
    c, kv = _fill_cache(w)
    for b in range(w.B):
        n, L = int(w.n_new[b]), int(w.ctx[b])
        qf = w.task_q_full(b)
        o_res, l_res = oa.attend(c, [w.rows()[b]], qf[L - n:], w.scale)
        o_all, l_all = oa.attend(c, [(int(w.task[b]), L, L)], qf, w.scale)
        assert np.allclose(o_res, o_all[L - n:], atol=1e-15) and np.allclose(l_res, l_all[L - n:], atol=1e-15)
        # and the first rows of the full pass are what an earlier, shorter resume would have produced
        o_pre, _ = oa.attend_contiguous(qf[: L - n], kv[b][0][: L - n], kv[b][1][: L - n], w.scale)
        assert np.allclose(o_pre, o_all[: L - n], atol=1e-15)


def test_split_merge_equals_unsplit():
    rng = np.random.default_rng(6)
    L, D = 50, 8
    q = oa.bf16_bits_to_f64(rand_bits(rng, (D,)))
    k = oa.bf16_bits_to_f64(rand_bits(rng, (L, D)))
    v = oa.bf16_bits_to_f64(rand_bits(rng, (L, D)))
    full_o, full_l = oa.attend_subset(q, k, v, 0.4, np.arange(L))
    for trial in range(20):
        cuts = np.sort(rng.integers(0, L + 1, size=rng.integers(1, 6)))
        bounds = np.concatenate([[0], cuts, [L]])                       # may contain empty and single-key splits
        perm = rng.permutation(L)
        parts = [oa.attend_subset(q, k, v, 0.4, perm[a:z]) for a, z in zip(bounds[:-1], bounds[1:])]
        mo, ml = oa.merge([p[0] for p in parts], [p[1] for p in parts])
        assert np.allclose(mo, full_o, atol=1e-12) and abs(ml - full_l) < 1e-12
    eo, el = oa.merge([np.zeros(D)], [-np.inf])
    assert el == -np.inf and np.all(eo == 0)


def test_merge_closed_form_two_equal_parts():
    # two subsets with equal LSE: O is the plain average, LSE rises by ln 2
    o, l = oa.merge([[1.0, 3.0], [3.0, 5.0]], [0.7, 0.7])
    assert np.allclose(o, [2.0, 4.0]) and abs(l - (0.7 + math.log(2))) < 1e-15


def test_c_oracle_matches_numpy_oracle_and_samples_items():
    w = inputs.make_workload(1, len_div=2)
    c, _ = _fill_cache(w)
    q = np.concatenate([w.task_q(b) for b in range(w.B)])
    o, lse = oa.attend(c, w.rows(), q, w.scale)
    co, cl = cbuild.attend_paged(c, w.rows(), q, w.scale)
    assert np.allclose(o, co, rtol=0, atol=1e-12) and np.allclose(lse, cl, rtol=0, atol=1e-12)
    # sampled items: (row, query index)
    res = [b for b in range(w.B) if w.n_new[b] > 1]
    items = [(res[0], 0), (res[0], int(w.n_new[res[0]]) - 1), (res[1], 3)]
    so, sl = cbuild.attend_paged(c, w.rows(), q, w.scale, items=items)
    qoff = np.concatenate([[0], np.cumsum(w.n_new)])
    for k, (b, i) in enumerate(items):
        assert np.array_equal(so[k], co[qoff[b] + i]) and np.array_equal(sl[k], cl[qoff[b] + i])


def test_c_oracle_bruteforce_and_zero_query_closed_form():
    # the C oracle pinned on its own: scalar brute force and LSE = ln(count) for Q = 0
    rng = np.random.default_rng(8)
    c = PagedKVOracle(8, 4, 2, 4, 2, 8, free_order=rng.permutation(8))
    c.alloc(0)
    k, v = rand_bits(rng, (11, 2, 4)), rand_bits(rng, (11, 2, 4))
    c.append([0], [0, 11], k, v)
    q = rand_bits(rng, (3, 4, 4))
    co, cl = cbuild.attend_paged(c, [(0, 3, 11)], q, 0.6)
    bo, bl = oa.attend_bruteforce(oa.bf16_bits_to_f64(q), oa.bf16_bits_to_f64(k), oa.bf16_bits_to_f64(v), 0.6)
    assert np.allclose(co, np.array(bo), atol=1e-13) and np.allclose(cl, np.array(bl), atol=1e-13)
    zo, zl = cbuild.attend_paged(c, [(0, 3, 10)], np.zeros_like(q), 0.6)
    for i in range(3):
        assert abs(zl[i, 0] - math.log(8 + i)) < 1e-14
        assert np.allclose(zo[i, 3], oa.bf16_bits_to_f64(v)[: 8 + i, 1].mean(axis=0), atol=1e-14)
