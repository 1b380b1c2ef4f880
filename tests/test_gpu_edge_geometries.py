"""Parity at the corners of the supported geometry and of the row shapes: one query head per KV head, sixteen
(the most), both head sizes, both page sizes; rows of one key, rows whose chunk is the whole context (a prefill
from scratch) at lengths around the tile sizes (16 / 64 / 128 / 256 packed rows, 64-key tiles, page edges), decode
rows long enough to be split over KV and merged, and the same task in several rows.  Every output element and
every LSE is compared with the float64 oracle."""
import math

import numpy as np
import pytest

from oracle import cbuild
from oracle.paged_kv import PagedKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

GEOMS = [(4, 4, 64, 32), (16, 1, 128, 16), (16, 1, 64, 32), (8, 1, 128, 32), (6, 2, 128, 16), (12, 4, 64, 16),
         (6, 3, 64, 16)]                      # an odd number of KV heads: the append's rounds of four (kv, head) blocks end ragged


@pytest.mark.parametrize("geom", GEOMS)
def test_row_shapes_at_the_corners(geom):
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = geom
    G = HQ // HKV
    rng = np.random.default_rng(HQ * 1000 + HKV * 100 + D + S)
    scale = 1.0 / math.sqrt(D)
    # (prefix, new tokens): one key; whole-context chunks around the tile edges; long decode rows; long resume rows
    shapes = [(0, 1), (0, 2), (0, 15), (0, 16), (0, 17), (0, 63), (0, 64), (0, 65), (0, 129), (0, 257), (S - 1, 1), (S, 1),
              (5000, 1), (12001, 1), (3000, 1), (700, 300), (4097, 40), (64, 64), (1, 200)]
    # rows per packed-row tile edge: q tokens such that q*G straddles 16, 64, 128 and 256 packed rows
    for edge in (16, 64, 128, 256):
        for q in {max(1, edge // G), edge // G + 1}:
            shapes.append((int(rng.integers(0, 400)), q))
    n_tasks = len(shapes)
    max_len = max(p + n for p, n in shapes)
    max_pages = (max_len + S - 1) // S + 1
    num_pages = sum((p + n + S - 1) // S for p, n in shapes) + 8
    order = rng.permutation(num_pages).astype(np.int32)
    total_q = sum(n for _, n in shapes)
    kv = tide.TideKV(HQ, HKV, D, S, num_pages, n_tasks, max_pages, 2 * n_tasks, 2 * total_q, free_order=order)
    orc = PagedKVOracle(num_pages, S, HKV, D, n_tasks, max_pages, free_order=order)
    for t, (p, n) in enumerate(shapes):
        kv.alloc(t)
        orc.alloc(t)
        if p:
            k, v = inputs.normal_bf16(rng, (p, HKV, D)), inputs.normal_bf16(rng, (p, HKV, D))
            kv.append([t], [0, p], H.to_dev(k, torch), H.to_dev(v, torch))
            orc.append([t], [0, p], k, v)
    ids = list(range(n_tasks))
    cnt = [n for _, n in shapes]
    indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
    nk, nv = inputs.normal_bf16(rng, (total_q, HKV, D)), inputs.normal_bf16(rng, (total_q, HKV, D))
    kv.append(ids, indptr, H.to_dev(nk, torch), H.to_dev(nv, torch))
    orc.append(ids, indptr, nk, nv)
    rows = [(t, n, p + n) for t, (p, n) in enumerate(shapes)]
    # the same tasks once more as decode rows over a shorter context, in the same batch
    again = [(t, 1, max(1, (p + n) // 2)) for t, (p, n) in enumerate(shapes) if p + n > 1][:n_tasks]
    rows_all = rows + again
    q = inputs.normal_bf16(rng, (sum(r[1] for r in rows_all), HQ, D))
    out = torch.zeros((q.shape[0], HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((q.shape[0], HQ), dtype=torch.float32, device="cuda")
    kv.attend(rows_all, H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows_all, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, f"geometry {geom}")
    plan = kv.last_plan()
    assert plan["merge_rows"] > 0, "the long rows were meant to be split over KV"
    for t in ids:
        assert np.array_equal(kv.page_table(t), orc.page_table(t))
    kv.close()


@pytest.mark.parametrize("scale", [0.0, -0.07])
def test_non_positive_scale_takes_the_warp_mma_path(scale):
    """The tcgen05 path takes the row maximum before scaling and so needs a positive scale; any other scale must
    fall back to the warp-MMA tile path and still match the oracle (scale 0: every visible key weighs the same)."""
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = 28, 4, 128, 16
    rng = np.random.default_rng(31)
    shapes = [(500, 1), (100, 90), (0, 300), (2100, 33)]
    num_pages = sum((p + n + S - 1) // S for p, n in shapes) + 4
    kv = tide.TideKV(HQ, HKV, D, S, num_pages, 4, 160, 4, 512)
    orc = PagedKVOracle(num_pages, S, HKV, D, 4, 160)
    cnt = [p + n for p, n in shapes]
    indptr = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
    T = int(indptr[-1])
    k, v = inputs.normal_bf16(rng, (T, HKV, D)), inputs.normal_bf16(rng, (T, HKV, D))
    for t in range(4):
        kv.alloc(t)
        orc.alloc(t)
    kv.append(list(range(4)), indptr, H.to_dev(k, torch), H.to_dev(v, torch))
    orc.append(list(range(4)), indptr, k, v)
    rows = [(t, n, p + n) for t, (p, n) in enumerate(shapes)]
    q = inputs.normal_bf16(rng, (sum(n for _, n in shapes), HQ, D))
    out = torch.zeros((q.shape[0], HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((q.shape[0], HQ), dtype=torch.float32, device="cuda")
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, f"scale {scale}")
    if scale == 0.0:
        # closed form: LSE = ln(number of visible keys)
        off = 0
        for (p, n) in shapes:
            want = np.log(np.arange(p + 1, p + n + 1, dtype=np.float64))
            assert np.abs(lse[off:off + n].cpu().numpy() - want[:, None]).max() < 1e-4
            off += n
    kv.close()
