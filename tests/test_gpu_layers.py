"""Multi-layer stepping on the GPU against the layered oracle: one page table and one plan per step serve every
layer; each layer's K/V store receives only its own rows.  Covers tide_kv_extend / tide_kv_write,
tide_step_begin / tide_step_layer (also replayed from a CUDA graph), tide_attend and tide_kv_read on any layer,
and the page copies of fork, copy-on-write and prune on every layer."""
import math

import numpy as np
import pytest

from oracle import cbuild
from oracle.layers import LayeredKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _make(L, HQ, HKV, D, S, num_pages, max_tasks, max_pages, max_rows, max_tokens, rng):
    from paper_2608_10402_b200 import tide
    order = rng.permutation(num_pages).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, num_pages, max_tasks, max_pages, max_rows, max_tokens, free_order=order, num_layers=L)
    orc = LayeredKVOracle(L, num_pages=num_pages, page_size=S, num_kv_heads=HKV, head_dim=D, max_tasks=max_tasks,
                          max_pages_per_task=max_pages, free_order=order)
    return kv, orc


def _same_state(kv, orc, tasks):
    for t in tasks:
        assert kv.task_len(t) == orc.task_len(t)
        assert np.array_equal(kv.page_table(t), orc.page_table(t)), f"page table of task {t}"
        assert np.array_equal(kv.page_refs(t), orc.page_refs(t)), f"page holders of task {t}"
    assert kv.usage() == (orc.used_tokens(), orc.free_pages())


def _same_bits(kv, orc, tasks, L):
    for l in range(L):
        for t in tasks:
            gk, gv = kv.read(t, layer=l)
            ok, ov = orc.read(l, t)
            assert np.array_equal(H.from_dev(gk), ok), f"K bits, layer {l}, task {t}"
            assert np.array_equal(H.from_dev(gv), ov), f"V bits, layer {l}, task {t}"


@pytest.mark.parametrize("geom", [(8, 2, 64, 16), (28, 4, 128, 16), (32, 8, 128, 32)])
def test_steps_over_three_layers_match_the_layered_oracle(geom):
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = geom
    L = 3
    rng = np.random.default_rng(77 + D + S)
    scale = 1.0 / math.sqrt(D)
    kv, orc = _make(L, HQ, HKV, D, S, 700, 12, 96, 12, 2048, rng)
    tasks = list(range(10))
    for t in tasks:
        kv.alloc(t)
        orc.alloc(t)

    def step(ids, cnt, planned):
        indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
        T = int(indptr[-1])
        nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        q = np.stack([inputs.normal_bf16(rng, (T, HQ, D)) for _ in range(L)])
        orc.append(ids, indptr, nk, nv)
        rows = [(t, c, orc.task_len(t)) for t, c in zip(ids, cnt)]
        outs = [torch.zeros((T, HQ, D), dtype=torch.int16, device="cuda") for _ in range(L)]
        lses = [torch.zeros((T, HQ), dtype=torch.float32, device="cuda") for _ in range(L)]
        dk, dv, dq = H.to_dev(nk, torch), H.to_dev(nv, torch), H.to_dev(q, torch)
        if planned:
            kv.step_begin(rows)
            for l in range(L):
                kv.step_layer(l, dk[l], dv[l], dq[l], scale, outs[l], lses[l])
        else:
            kv.extend(ids, indptr)
            for l in reversed(range(L)):          # the order of the layers must not matter
                kv.write(l, ids, indptr, dk[l], dv[l])
            for l in range(L):
                kv.attend(rows, dq[l], scale, outs[l], lses[l], layer=l)
        assert kv.status() == tide.OK
        for l in range(L):
            ref_o, ref_l = cbuild.attend_paged(orc.layer(l), rows, q[l], scale)
            H.check_outputs(H.from_dev(outs[l]), lses[l].cpu().numpy(), ref_o, ref_l, f"layer {l}")
        _same_state(kv, orc, ids)

    # prompts from scratch (decode-style, tile and tcgen05 rows), then decode and resume steps
    step(tasks, [int(rng.integers(3, 260)) for _ in tasks], planned=True)
    step(tasks, [1] * len(tasks), planned=True)
    step(tasks[:6], [int(rng.integers(20, 300)) for _ in range(6)], planned=False)
    step(tasks, [1 if t % 2 else int(rng.integers(2, 90)) for t in tasks], planned=True)
    _same_bits(kv, orc, tasks, L)
    plan = kv.last_plan()
    assert plan["decode_items"] > 0
    kv.close()


def test_fork_copy_on_write_and_prune_cover_every_layer():
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S, L = 8, 2, 64, 16, 4
    rng = np.random.default_rng(5)
    kv, orc = _make(L, HQ, HKV, D, S, 400, 10, 64, 10, 96, rng)   # small staging: long tails move in chunks

    def append(ids, cnt):
        indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
        T = int(indptr[-1])
        nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        orc.append(ids, indptr, nk, nv)
        kv.extend(ids, indptr)
        for l in range(L):
            kv.write(l, ids, indptr, H.to_dev(nk[l], torch), H.to_dev(nv[l], torch))

    for t in (0, 1):
        kv.alloc(t)
        orc.alloc(t)
    append([0, 1], [203, 330])
    # fork with a partial last page: the page copy must happen on every layer
    kv.fork(0, 2)
    orc.fork(0, 2)
    kv.fork(1, 3)
    orc.fork(1, 3)
    append([2, 0, 3], [40, 9, 5])
    _same_state(kv, orc, [0, 1, 2, 3])
    _same_bits(kv, orc, [0, 1, 2, 3], L)
    # truncate into shared pages, then append: copy-on-write on every layer
    kv.truncate(2, 100)
    orc.truncate(2, 100)
    append([2], [30])
    _same_bits(kv, orc, [0, 2], L)
    # prune of a task that shares no page: its tail of 315 tokens moves in place, in chunks of 96
    kv.alloc(4)
    orc.alloc(4)
    append([4], [400])
    kv.prune(4, 70, 85)
    orc.prune(4, 70, 85)
    _same_state(kv, orc, [0, 1, 2, 3, 4])
    _same_bits(kv, orc, [4], L)
    # the same for a task whose shared pages all lie below keep_prefix (task 2: pages up to token 96 are task 0's)
    kv.prune(2, 113, 120)
    orc.prune(2, 113, 120)
    _same_state(kv, orc, [0, 2])
    _same_bits(kv, orc, [0, 2], L)
    # prune of a task that shares pages (its tail fits the staging area)
    assert orc.task_len(3) == 335
    kv.prune(3, 250, 290)
    orc.prune(3, 250, 290)
    _same_state(kv, orc, [0, 1, 2, 3])
    _same_bits(kv, orc, [0, 1, 2, 3], L)
    # ... and one whose tail does not: refused, nothing changes
    with pytest.raises(tide.TideError) as e:
        kv.prune(3, 10, 20)
    assert e.value.code == tide.ERR_WORKSPACE
    _same_state(kv, orc, [0, 1, 2, 3])
    _same_bits(kv, orc, [3], L)
    assert kv.status() == tide.OK
    kv.close()


def test_prune_refusal_for_lack_of_pages_changes_nothing():
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S, L = 8, 2, 64, 16, 2
    rng = np.random.default_rng(6)
    from oracle.paged_kv import ERR_NO_PAGES, OracleError
    kv, orc = _make(L, HQ, HKV, D, S, 4, 2, 4, 2, 64, rng)

    def append(ids, cnt):
        indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
        T = int(indptr[-1])
        nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        orc.append(ids, indptr, nk, nv)
        kv.extend(ids, indptr)
        for l in range(L):
            kv.write(l, ids, indptr, H.to_dev(nk[l], torch), H.to_dev(nv[l], torch))

    kv.alloc(0)
    orc.alloc(0)
    append([0], [2 * S])
    kv.fork(0, 1)
    orc.fork(0, 1)
    append([1], [2 * S])
    with pytest.raises(OracleError) as eo:
        orc.prune(1, S // 2, S)
    assert eo.value.code == ERR_NO_PAGES
    with pytest.raises(tide.TideError) as eg:
        kv.prune(1, S // 2, S)
    assert eg.value.code == tide.ERR_NO_PAGES
    _same_state(kv, orc, [0, 1])
    _same_bits(kv, orc, [0, 1], L)
    kv.release(0)
    orc.release(0)
    kv.prune(1, S // 2, S)
    orc.prune(1, S // 2, S)
    _same_state(kv, orc, [1])
    _same_bits(kv, orc, [1], L)
    kv.close()


def test_layer_argument_and_step_errors():
    import torch
    from paper_2608_10402_b200 import tide
    rng = np.random.default_rng(8)
    kv, orc = _make(2, 8, 2, 64, 16, 64, 4, 16, 4, 64, rng)
    kv.alloc(0)
    z = torch.zeros((8, 2, 64), dtype=torch.int16, device="cuda")
    q = torch.zeros((8, 8, 64), dtype=torch.int16, device="cuda")
    out = torch.zeros_like(q)

    def code(fn, *a, **k):
        with pytest.raises(tide.TideError) as e:
            fn(*a, **k)
        return e.value.code

    assert code(kv.step_layer, 0, z, z, q, 0.125, out) == tide.ERR_INVALID_ARG        # no step is open
    kv.extend([0], [0, 4])
    assert code(kv.write, 2, [0], [0, 4], z, z) == tide.ERR_INVALID_ARG               # layer out of range
    assert code(kv.write, 1, [0], [0, 5], z, z) == tide.ERR_CTX_RANGE                 # more rows than the task holds
    assert code(kv.attend, [(0, 1, 4)], q, 0.125, out, layer=2) == tide.ERR_INVALID_ARG
    assert code(kv.step_begin, [(0, 4, 7)]) == tide.ERR_CTX_RANGE                     # ctx_len != len + q_len
    assert code(kv.step_begin, [(0, 2, 6), (0, 2, 6)]) == tide.ERR_DUPLICATE_TASK
    assert kv.task_len(0) == 4                                                        # refused calls changed nothing
    kv.step_begin([(0, 4, 8)])
    assert code(kv.step_layer, 0, z, z, q, -1.0, out) == tide.ERR_INVALID_ARG         # scale must be positive
    assert code(kv.step_layer, 5, z, z, q, 0.125, out) == tide.ERR_INVALID_ARG
    kv.step_layer(1, z, z, q, 0.125, out)
    kv.truncate(0, 6)                                                                 # a change closes the step
    assert code(kv.step_layer, 0, z, z, q, 0.125, out) == tide.ERR_INVALID_ARG
    assert kv.status() == tide.OK
    kv.close()


def test_layers_of_a_step_replayed_from_a_cuda_graph():
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S, L = 28, 4, 128, 16, 4
    rng = np.random.default_rng(9)
    scale = 1.0 / math.sqrt(D)
    kv, orc = _make(L, HQ, HKV, D, S, 600, 8, 128, 8, 1024, rng)
    tasks = list(range(8))
    for t in tasks:
        kv.alloc(t)
        orc.alloc(t)
    # history
    cnt = [int(rng.integers(100, 900)) for _ in tasks]
    indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
    T = int(indptr[-1])
    hk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
    hv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
    orc.append(tasks, indptr, hk, hv)
    kv.extend(tasks, indptr)
    for l in range(L):
        kv.write(l, tasks, indptr, H.to_dev(hk[l], torch), H.to_dev(hv[l], torch))
    # the step: five decode rows and three resume rows
    cnt = [1, 1, 1, 1, 1, 70, 33, 140]
    indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
    T = int(indptr[-1])
    nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
    nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
    q = np.stack([inputs.normal_bf16(rng, (T, HQ, D)) for _ in range(L)])
    orc.append(tasks, indptr, nk, nv)
    rows = [(t, c, orc.task_len(t)) for t, c in zip(tasks, cnt)]
    dk, dv, dq = H.to_dev(nk, torch), H.to_dev(nv, torch), H.to_dev(q, torch)
    out = torch.zeros((L, T, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((L, T, HQ), dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        kv.step_begin(rows, stream=side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for l in range(L):
                kv.step_layer(l, dk[l], dv[l], dq[l], scale, out[l], lse[l], stream=torch.cuda.current_stream())
        graph.replay()
        side.synchronize()
        first = out.clone()
        out.zero_()
        lse.zero_()
        graph.replay()                      # idempotent: the same rows go to the same places
        side.synchronize()
        assert kv.status(stream=side) == tide.OK
    torch.cuda.current_stream().wait_stream(side)
    assert torch.equal(first, out)
    for l in range(L):
        ref_o, ref_l = cbuild.attend_paged(orc.layer(l), rows, q[l], scale)
        H.check_outputs(H.from_dev(out[l]), lse[l].cpu().numpy(), ref_o, ref_l, f"graph replay, layer {l}")
    _same_state(kv, orc, tasks)
    _same_bits(kv, orc, tasks, L)
    kv.close()


def test_layer_pools_beyond_four_gib():
    """Three layers of 2.46 GB each, with the tasks' pages at the far end of every layer's pool: byte offsets of
    layers 1 and 2 lie beyond 4 GiB, so any 32-bit step in the address arithmetic would show."""
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S, L = 28, 4, 128, 16, 3
    NUM_PAGES, USED = 150000, 64
    free, _ = torch.cuda.mem_get_info()
    if free < 10 * (1 << 30):
        pytest.skip("needs 10 GB of free device memory")
    rng = np.random.default_rng(10)
    scale = 1.0 / math.sqrt(D)
    # the library hands out the last USED pages first; the oracle runs on a pool of just those pages
    order = np.concatenate([np.arange(NUM_PAGES - USED, NUM_PAGES), np.arange(NUM_PAGES - USED)]).astype(np.int32)
    kv = tide.TideKV(HQ, HKV, D, S, NUM_PAGES, 4, 64, 4, 1024, free_order=order, num_layers=L)
    orc = LayeredKVOracle(L, num_pages=USED, page_size=S, num_kv_heads=HKV, head_dim=D, max_tasks=4, max_pages_per_task=64)
    tasks = [0, 1, 2]
    for t in tasks:
        kv.alloc(t)
        orc.alloc(t)
    cnt = [300, 17, 150]
    for step_cnt in (cnt, [1, 40, 200]):
        indptr = np.concatenate([[0], np.cumsum(step_cnt)]).astype(np.int32)
        T = int(indptr[-1])
        nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
        q = np.stack([inputs.normal_bf16(rng, (T, HQ, D)) for _ in range(L)])
        orc.append(tasks, indptr, nk, nv)
        rows = [(t, c, orc.task_len(t)) for t, c in zip(tasks, step_cnt)]
        out = torch.zeros((L, T, HQ, D), dtype=torch.int16, device="cuda")
        lse = torch.zeros((L, T, HQ), dtype=torch.float32, device="cuda")
        dk, dv, dq = H.to_dev(nk, torch), H.to_dev(nv, torch), H.to_dev(q, torch)
        kv.step_begin(rows)
        for l in range(L):
            kv.step_layer(l, dk[l], dv[l], dq[l], scale, out[l], lse[l])
        assert kv.status() == tide.OK
        for l in range(L):
            ref_o, ref_l = cbuild.attend_paged(orc.layer(l), rows, q[l], scale)
            H.check_outputs(H.from_dev(out[l]), lse[l].cpu().numpy(), ref_o, ref_l, f"layer {l}")
    for t in tasks:
        assert np.array_equal(kv.page_table(t), orc.page_table(t) + (NUM_PAGES - USED))
    _same_bits(kv, orc, tasks, L)
    kv.close()


def test_one_graph_replayed_over_a_decode_loop():
    """The generation loop between environment turns: the layers of a step are captured ONCE with fixed launch
    shapes and replayed for every later step; only tide_step_begin (host planning, a small upload, the page-table
    delta) runs between replays.  Lengths cross page boundaries, the KV splits change, and one step in the middle
    also carries resume rows; every step is checked against the oracle."""
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S, L = 28, 4, 128, 16, 3
    B, MAXQ = 6, 256
    rng = np.random.default_rng(12)
    scale = 1.0 / math.sqrt(D)
    kv, orc = _make(L, HQ, HKV, D, S, 900, B, 128, B, MAXQ, rng)
    tasks = list(range(B))
    for t in tasks:
        kv.alloc(t)
        orc.alloc(t)
    cnt = [int(rng.integers(60, 1500)) for _ in tasks]
    indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
    T0 = int(indptr[-1])
    hk = np.stack([inputs.normal_bf16(rng, (T0, HKV, D)) for _ in range(L)])
    hv = np.stack([inputs.normal_bf16(rng, (T0, HKV, D)) for _ in range(L)])
    orc.append(tasks, indptr, hk, hv)
    kv.extend(tasks, indptr)
    for l in range(L):
        kv.write(l, tasks, indptr, H.to_dev(hk[l], torch), H.to_dev(hv[l], torch))
    # static buffers the graph reads and writes; a step uses their first T rows
    dk = torch.zeros((L, MAXQ, HKV, D), dtype=torch.int16, device="cuda")
    dv = torch.zeros_like(dk)
    dq = torch.zeros((L, MAXQ, HQ, D), dtype=torch.int16, device="cuda")
    out = torch.zeros((L, MAXQ, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((L, MAXQ, HQ), dtype=torch.float32, device="cuda")
    kv.step_fix_grids(max_decode_items=1024, max_tile_items=64, max_umma_items=64, max_merge_rows=MAXQ * HQ, max_tokens=MAXQ)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = None
    with torch.cuda.stream(side):
        for step in range(24):
            cnt = [1] * B if step != 9 else [1, 40, 1, 90, 1, 17]        # step 9 mixes in resume rows
            indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
            T = int(indptr[-1])
            nk = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
            nv = np.stack([inputs.normal_bf16(rng, (T, HKV, D)) for _ in range(L)])
            q = np.stack([inputs.normal_bf16(rng, (T, HQ, D)) for _ in range(L)])
            orc.append(tasks, indptr, nk, nv)
            rows = [(t, c, orc.task_len(t)) for t, c in zip(tasks, cnt)]
            dk[:, :T].copy_(H.to_dev(nk, torch))
            dv[:, :T].copy_(H.to_dev(nv, torch))
            dq[:, :T].copy_(H.to_dev(q, torch))
            kv.step_begin(rows, stream=side)
            if graph is None:
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for l in range(L):
                        kv.step_layer(l, dk[l], dv[l], dq[l], scale, out[l], lse[l], stream=torch.cuda.current_stream())
            graph.replay()
            side.synchronize()
            assert kv.status(stream=side) == tide.OK
            for l in range(L):
                ref_o, ref_l = cbuild.attend_paged(orc.layer(l), rows, q[l], scale)
                H.check_outputs(H.from_dev(out[l, :T]), lse[l, :T].cpu().numpy(), ref_o, ref_l, f"step {step}, layer {l}")
            _same_state(kv, orc, tasks)
        # a step that plans more than the fixed shapes allow is refused before anything changes
        kv.step_fix_grids(max_decode_items=2, max_tokens=MAXQ)
        with pytest.raises(tide.TideError) as e:
            kv.step_begin([(t, 1, orc.task_len(t) + 1) for t in tasks], stream=side)
        assert e.value.code == tide.ERR_WORKSPACE
        _same_state(kv, orc, tasks)
    torch.cuda.current_stream().wait_stream(side)
    _same_bits(kv, orc, tasks, L)
    kv.close()
