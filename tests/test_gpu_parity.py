"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle, element by element, on the
same seeded bits.  Page tables, lengths and cache contents bit-exact; attention within
|gpu - oracle| <= 1e-2 + 1e-2 |oracle| and LSE within 1e-3 (bf16 inputs, fp32 accumulation)."""
import math

import numpy as np
import pytest

from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2608_10402_b200 import tide
    assert torch.cuda.is_available()
    return tide, torch


def run_workload(w, tide, torch, full_oracle=True, seed=0, tune=()):
    kv_bits = [w.task_kv(b) for b in range(w.B)]
    q_bits = np.concatenate([w.task_q(b) for b in range(w.B)])
    c, indptr, nk, nv = H.oracle_fill(w, kv_bits)
    kv = H.gpu_fill(w, kv_bits, nk, nv, indptr, tide, torch, tune=tune)
    H.compare_bookkeeping(w, c, kv)
    H.compare_cache(w, c, kv)
    total_q = q_bits.shape[0]
    out = torch.zeros((total_q, w.Hq, w.D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((total_q, w.Hq), dtype=torch.float32, device="cuda")
    kv.attend(w.rows(), H.to_dev(q_bits, torch), w.scale, out, lse)
    assert kv.status() == tide.OK
    got_o, got_l = H.from_dev(out), lse.cpu().numpy()
    if full_oracle:
        ref_o, ref_l = H.oracle_attend(c, w, q_bits)
        stats = H.check_outputs(got_o, got_l, ref_o, ref_l, w.name)
    else:
        items = H.sample_items(w, np.random.default_rng(seed))
        ref_o, ref_l = H.oracle_attend(c, w, q_bits, items=items)
        qoff = np.concatenate([[0], np.cumsum(w.n_new)])
        idx = np.array([qoff[b] + i for b, i in items])
        stats = H.check_outputs(got_o[idx], got_l[idx], ref_o, ref_l, w.name + " (sampled)")
    kv.close()
    return stats


def test_config1_tiny_ctb_step(env):
    tide, torch = env
    run_workload(inputs.make_workload(1), tide, torch)


@pytest.mark.parametrize("index,n_tasks,len_div", [(2, 12, 8), (3, 12, 8), (4, 6, 16), (5, 16, 16)])
def test_reduced_configs_full_oracle(env, index, n_tasks, len_div):
    tide, torch = env
    run_workload(inputs.make_workload(index, n_tasks=n_tasks, len_div=len_div), tide, torch)


@pytest.mark.parametrize("index,n_tasks,len_div", [(3, 12, 8), (4, 6, 16), (5, 16, 16)])
def test_the_64_key_tcgen05_kernel_matches_too(env, index, n_tasks, len_div):
    # the append-prefill kernel with 64-key tiles (Q in TMEM) stays selectable next to the default 128-key one
    tide, torch = env
    run_workload(inputs.make_workload(index, n_tasks=n_tasks, len_div=len_div), tide, torch, tune=[(tide.TUNE_UMMA_TILE_KEYS, 64)])


def test_small_batches_with_uploaded_descriptors_match_too(env):
    # by default a small append and a small decode-only batch carry their descriptors in the launch's parameters; with
    # that turned off they are uploaded like those of large batches, and the results must be the same
    tide, torch = env
    run_workload(inputs.make_workload(2, n_tasks=12, len_div=8), tide, torch, tune=[(tide.TUNE_INLINE_DESCRIPTORS, 0)])
    run_workload(inputs.make_workload(1), tide, torch, tune=[(tide.TUNE_INLINE_DESCRIPTORS, 0)])


def test_planning_uploads_through_the_copy_engine_match_too(env):
    # by default the small planning uploads are done by a kernel that reads the mapped staging slot; the copy-engine
    # path stays selectable and must give the same pages, cache bits and outputs
    tide, torch = env
    run_workload(inputs.make_workload(3, n_tasks=12, len_div=8), tide, torch, tune=[(tide.TUNE_UPLOAD_BY_KERNEL, 0)])


def _single_row_case(tide, torch, Hq, Hkv, D, S, n, L, q_bits, k_bits, v_bits, scale, free_seed=0):
    pages = (L + S - 1) // S + 3
    kv = tide.TideKV(Hq, Hkv, D, S, pages, 2, pages, 4, max(n, 4),
                     free_order=np.random.default_rng(free_seed).permutation(pages))
    kv.alloc(0)
    kv.append([0], [0, L], H.to_dev(k_bits, torch), H.to_dev(v_bits, torch))
    out = torch.zeros((n, Hq, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((n, Hq), dtype=torch.float32, device="cuda")
    kv.attend([(0, n, L)], H.to_dev(q_bits, torch), scale, out, lse)
    assert kv.status() == tide.OK
    res = H.oa.bf16_bits_to_f64(H.from_dev(out)), lse.cpu().numpy().astype(np.float64)
    kv.close()
    return res


@pytest.mark.parametrize("n,L", [(1, 777), (5, 300), (40, 1000), (70, 70)])
def test_zero_query_counts_visible_keys(env, n, L):
    # Q = 0 => LSE = ln(#visible keys) and O = running mean of V: any off-by-one in the causal alignment,
    # the split ranges or the ragged tail shows up here with O(1) outputs.
    tide, torch = env
    rng = np.random.default_rng(L)
    Hq, Hkv, D, S = 8, 2, 64, 16
    k, v = inputs.normal_bf16(rng, (L, Hkv, D)), inputs.normal_bf16(rng, (L, Hkv, D))
    o, lse = _single_row_case(tide, torch, Hq, Hkv, D, S, n, L, np.zeros((n, Hq, D), np.uint16), k, v, 0.125)
    vf = H.oa.bf16_bits_to_f64(v)
    for i in range(n):
        vis = L - n + i + 1
        assert np.abs(lse[i] - math.log(vis)).max() < 1e-3
        for h in range(Hq):
            assert np.abs(o[i, h] - vf[:vis, h // 4].mean(axis=0)).max() < 1e-2


def test_needle_key_checks_slot_order_and_heads(env):
    # one dominant key per KV head (logit gap >> 40): O must equal that key's V row (O(1) values).
    tide, torch = env
    rng = np.random.default_rng(7)
    Hq, Hkv, D, S, L = 28, 4, 128, 16, 2500
    k = np.zeros((L, Hkv, D), np.uint16)
    v = inputs.normal_bf16(rng, (L, Hkv, D))
    q = inputs.f32_to_bf16_bits(np.full((1, Hq, D), 2.0, np.float32))
    needles = [3, 1029, 2047, 2499]
    for g, j in enumerate(needles):
        k[j, g] = inputs.f32_to_bf16_bits(np.full(D, 2.0, np.float32))     # logit 2*2*128*scale = 45.3
    o, _ = _single_row_case(tide, torch, Hq, Hkv, D, S, 1, L, q, k, v, 1.0 / math.sqrt(D))
    vf = H.oa.bf16_bits_to_f64(v)
    for h in range(Hq):
        g = h // 7
        assert np.abs(o[0, h] - vf[needles[g], g]).max() < 2e-2


def test_constant_v_returns_that_constant(env):
    tide, torch = env
    rng = np.random.default_rng(9)
    Hq, Hkv, D, S, n, L = 32, 8, 128, 32, 33, 600
    k = inputs.normal_bf16(rng, (L, Hkv, D))
    v = inputs.f32_to_bf16_bits(np.full((L, Hkv, D), -1.25, np.float32))
    q = inputs.normal_bf16(rng, (n, Hq, D))
    o, _ = _single_row_case(tide, torch, Hq, Hkv, D, S, n, L, q, k, v, 0.1)
    assert np.abs(o + 1.25).max() < 1e-2


def test_ctb_invariant_on_gpu_resume_equals_recompute(env):
    # resumed chunk from the preserved cache == last n rows of a from-scratch causal pass (q_len = ctx_len)
    tide, torch = env
    w = inputs.make_workload(1, len_div=2)
    kv_bits = [w.task_kv(b) for b in range(w.B)]
    c, indptr, nk, nv = H.oracle_fill(w, kv_bits)
    total = int(w.ctx.sum())
    kv = H.gpu_fill(w, kv_bits, nk, nv, indptr, tide, torch, max_batch_tokens=total)
    for b in range(w.B):
        n, L, t = int(w.n_new[b]), int(w.ctx[b]), int(w.task[b])
        qf = w.task_q_full(b)
        o_all = torch.zeros((L, w.Hq, w.D), dtype=torch.int16, device="cuda")
        l_all = torch.zeros((L, w.Hq), dtype=torch.float32, device="cuda")
        kv.attend([(t, L, L)], H.to_dev(qf, torch), w.scale, o_all, l_all)
        o_res = torch.zeros((n, w.Hq, w.D), dtype=torch.int16, device="cuda")
        l_res = torch.zeros((n, w.Hq), dtype=torch.float32, device="cuda")
        kv.attend([(t, n, L)], H.to_dev(qf[L - n:], torch), w.scale, o_res, l_res)
        # both passes against the oracle's from-scratch pass first: the resumed rows must equal ITS last n rows
        ref_o, ref_l = H.cbuild.attend_paged(c, [(t, L, L)], qf, w.scale)
        H.check_outputs(H.from_dev(o_all), l_all.cpu().numpy(), ref_o, ref_l, "from-scratch pass")
        H.check_outputs(H.from_dev(o_res), l_res.cpu().numpy(), ref_o[L - n:], ref_l[L - n:], "resumed chunk vs from-scratch oracle")
        # and, as a second check, against each other
        a = H.oa.bf16_bits_to_f64(H.from_dev(o_all))[L - n:]
        r = H.oa.bf16_bits_to_f64(H.from_dev(o_res))
        assert np.abs(a - r).max() <= 2e-2 and np.abs(l_all.cpu().numpy()[L - n:] - l_res.cpu().numpy()).max() < 1e-3
    assert kv.status() == tide.OK
    kv.close()


def test_error_paths_change_nothing(env):
    tide, torch = env
    kv = tide.TideKV(8, 2, 64, 16, 3, 3, 2, 4, 64)
    z = torch.zeros((64, 2, 64), dtype=torch.int16, device="cuda")
    kv.alloc(0)
    kv.alloc(1)
    kv.append([0], [0, 3], z, z)

    def snapshot():
        return (kv.usage(), [(t, kv.task_len(t), tuple(kv.page_table(t))) for t in (0, 1)])

    def fails(code, fn):
        before = snapshot()
        with pytest.raises(tide.TideError) as e:
            fn()
        assert e.value.code == code, (e.value.code, code)
        assert snapshot() == before

    q = torch.zeros((4, 8, 64), dtype=torch.int16, device="cuda")
    o = torch.zeros_like(q)
    fails(tide.ERR_INVALID_ARG, lambda: kv.alloc(3))
    fails(tide.ERR_TASK_EXISTS, lambda: kv.alloc(0))
    fails(tide.ERR_NO_PAGES, lambda: kv.alloc(2, 33))
    fails(tide.ERR_UNKNOWN_TASK, lambda: kv.append([2], [0, 1], z, z))
    fails(tide.ERR_DUPLICATE_TASK, lambda: kv.append([0, 0], [0, 1, 2], z, z))
    fails(tide.ERR_INVALID_ARG, lambda: kv.append([0, 1], [0, 2, 1], z, z))
    fails(tide.ERR_TABLE_FULL, lambda: kv.append([0], [0, 30], z, z))
    fails(tide.ERR_NO_PAGES, lambda: kv.append([0, 1], [0, 14, 46], z, z))
    fails(tide.ERR_UNKNOWN_TASK, lambda: kv.release(2))
    fails(tide.ERR_INVALID_ARG, lambda: kv.truncate(0, 4))
    fails(tide.ERR_CTX_RANGE, lambda: kv.attend([(0, 1, 4)], q, 1.0, o))
    fails(tide.ERR_CTX_RANGE, lambda: kv.attend([(0, 0, 2)], q, 1.0, o))
    fails(tide.ERR_CTX_RANGE, lambda: kv.attend([(0, 3, 2)], q, 1.0, o))
    fails(tide.ERR_UNKNOWN_TASK, lambda: kv.attend([(2, 1, 1)], q, 1.0, o))
    fails(tide.ERR_WORKSPACE, lambda: kv.attend([(0, 1, 3)] * 5, q, 1.0, o))
    kv.append([1], [0, 0], z, z)      # zero-length append: no-op
    assert kv.task_len(1) == 0
    kv.close()


def test_append_leaves_neighbouring_slots_untouched(env):
    # canary: the scatter may only touch the 16-byte chunks of the slots it was asked to fill
    tide, torch = env
    rng = np.random.default_rng(21)
    Hq, Hkv, D, S = 8, 2, 64, 16
    kv = tide.TideKV(Hq, Hkv, D, S, 8, 2, 8, 2, 16)
    kv.pool.fill_(0x5A)
    a = inputs.normal_bf16(rng, (48, Hkv, D))
    b = inputs.normal_bf16(rng, (5, Hkv, D))
    kv.alloc(0)
    kv.append([0], [0, 48], H.to_dev(a, torch), H.to_dev(a[::-1].copy(), torch))
    kv.truncate(0, 20)
    torch.cuda.synchronize()
    before = kv.pool.clone()
    kv.append([0], [0, 5], H.to_dev(b, torch), H.to_dev(b[::-1].copy(), torch))      # positions 20..24
    torch.cuda.synchronize()
    changed = (kv.pool != before).view(-1)
    n = changed.numel() // 16 * 16
    chunks = changed[:n].view(-1, 16).any(dim=1).sum().item()
    assert 0 < chunks <= 5 * Hkv * (D // 8) * 2
    k, v = kv.read(0)
    assert np.array_equal(H.from_dev(k)[:20], a[:20]) and np.array_equal(H.from_dev(k)[20:], b)
    assert np.array_equal(H.from_dev(v)[:20], a[::-1][:20]) and np.array_equal(H.from_dev(v)[20:], b[::-1])
    kv.close()


@pytest.mark.parametrize("groups, zero_copy", [(0, 1), (0, 0), (3, 1), (8, 1)])
def test_step_host_matches_append_then_attend(env, groups, zero_copy):
    # groups > 0 forces the step to be cut into that many row groups whose copies and kernels overlap (what large
    # steps do by themselves); pages, cache bits and outputs must not depend on the cut.  A small step in one group
    # is by default not copied at all (the kernels address the pinned host buffers); zero_copy = 0 takes the copies.
    tide, torch = env
    w = inputs.make_workload(1)
    kv_bits = [w.task_kv(b) for b in range(w.B)]
    q_bits = np.concatenate([w.task_q(b) for b in range(w.B)])
    c, indptr, nk, nv = H.oracle_fill(w, kv_bits)
    total_q = int(w.n_new.sum())
    kv = tide.TideKV(w.Hq, w.Hkv, w.D, w.S, w.num_pages, w.max_tasks, w.max_pages_per_task, w.B, total_q,
                     free_order=w.free_order)
    kv.tune(tide.TUNE_HOST_STEP_CHUNKS, groups)
    kv.tune(tide.TUNE_HOST_ZERO_COPY, zero_copy)
    for b in range(w.B):
        kv.alloc(int(w.task[b]))
    for b in range(w.B):
        p = int(w.prefix[b])
        kv.append([int(w.task[b])], [0, p], H.to_dev(kv_bits[b][0][:p], torch), H.to_dev(kv_bits[b][1][:p], torch))
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
    hk, hv, hq = pin(nk), pin(nv), pin(q_bits)
    hout = torch.zeros((total_q, w.Hq, w.D), dtype=torch.int16).pin_memory()
    hlse = torch.zeros((total_q, w.Hq), dtype=torch.float32).pin_memory()
    kv.step_host(w.rows(), hk, hv, hq, w.scale, hout, hlse)
    assert kv.status() == tide.OK
    H.compare_bookkeeping(w, c, kv)
    H.compare_cache(w, c, kv)
    ref_o, ref_l = H.oracle_attend(c, w, q_bits)
    H.check_outputs(hout.numpy().view(np.uint16), hlse.numpy(), ref_o, ref_l, "step_host")
    kv.close()


def test_outputs_are_bitwise_independent_of_where_the_pages_lie(env):
    """The plan depends on logical lengths only and no kernel's arithmetic order depends on page numbers, so the
    same batch over two different page permutations (and run twice) must give the same bits, not just the same
    values within tolerance."""
    tide, torch = env
    w = inputs.make_workload(3, n_tasks=12, len_div=8)
    kv_bits = [w.task_kv(b) for b in range(w.B)]
    q_bits = np.concatenate([w.task_q(b) for b in range(w.B)])
    _, indptr, nk, nv = H.oracle_fill(w, kv_bits)
    total_q = q_bits.shape[0]
    results = []
    for seed in (1, 2, 2):
        w.free_order = np.random.default_rng(seed).permutation(w.num_pages).astype(np.int32)
        kv = H.gpu_fill(w, kv_bits, nk, nv, indptr, tide, torch)
        out = torch.zeros((total_q, w.Hq, w.D), dtype=torch.int16, device="cuda")
        lse = torch.zeros((total_q, w.Hq), dtype=torch.float32, device="cuda")
        kv.attend(w.rows(), H.to_dev(q_bits, torch), w.scale, out, lse)
        assert kv.status() == tide.OK
        results.append((out.cpu().numpy().copy(), lse.cpu().numpy().copy()))
        kv.close()
    for o, l in results[1:]:
        assert np.array_equal(o, results[0][0]) and np.array_equal(l.view(np.uint32), results[0][1].view(np.uint32))
