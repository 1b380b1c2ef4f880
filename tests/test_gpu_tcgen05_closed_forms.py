"""Closed-form cases with outputs of order one ON the tcgen05 append-prefill kernel (head size 128, more than 16
packed rows per KV head, positive scale): on random data |O| is a few hundredths and the elementwise tolerance is
loose, so these cases carry the weight there.  A zero query makes every visible key weigh the same, which turns the
log-sum-exp into the logarithm of a count and the output into a running mean; graded needle keys make one key
dominate each query, which turns the output into one row of V and pins the causal edge to the exact position."""
import math

import numpy as np
import pytest

from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

HQ, HKV, D, S = 28, 4, 128, 16
G = HQ // HKV


def _run_row(tide, torch, p, n, k, v, q, scale, expect_umma=True):
    L = p + n
    pages = (L + S - 1) // S + 3
    kv = tide.TideKV(HQ, HKV, D, S, pages, 2, pages, 2, max(n, 4), free_order=np.random.default_rng(L).permutation(pages))
    kv.alloc(0)
    if p:
        kv.append([0], [0, p], H.to_dev(k[:p], torch), H.to_dev(v[:p], torch))   # the preserved prefix ...
    kv.append([0], [0, n], H.to_dev(k[p:], torch), H.to_dev(v[p:], torch))       # ... then the resumed chunk
    out = torch.zeros((n, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((n, HQ), dtype=torch.float32, device="cuda")
    kv.attend([(0, n, L)], H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    plan = kv.last_plan()
    if expect_umma:
        assert plan["prefill_items"] > 0 and plan["decode_items"] == 0
    kv.close()
    return H.oa.bf16_bits_to_f64(H.from_dev(out)), lse.cpu().numpy().astype(np.float64), plan


@pytest.mark.parametrize("p,n", [(1000, 40), (3000, 300), (0, 129), (17, 3), (2500, 37)])
def test_zero_query_on_the_tcgen05_path_counts_keys_and_averages_v(p, n):
    """Q = 0 with scale > 0: LSE(i) = ln(p + i + 1) to 1e-4 (1 / (p + i + 1) apart from its neighbours, so an
    off-by-one in the causal edge, a tile edge, a KV split or the ragged tail shows) and O(i) = mean of the visible
    V rows, here of order one."""
    import torch
    from paper_2608_10402_b200 import tide
    rng = np.random.default_rng(p * 1000 + n)
    L = p + n
    k = inputs.normal_bf16(rng, (L, HKV, D))
    vf = (1.0 + 0.5 * rng.standard_normal((L, HKV, D))).astype(np.float32)
    vf[:, :, ::2] *= -1.0                                     # both signs, |mean| about 1
    v = inputs.f32_to_bf16_bits(vf)
    o, lse, plan = _run_row(tide, torch, p, n, k, v, np.zeros((n, HQ, D), np.uint16), 1.0 / math.sqrt(D), expect_umma=n * G > 16)
    v64 = H.oa.bf16_bits_to_f64(v)
    csum = np.cumsum(v64, axis=0)
    for i in range(n):
        vis = p + i + 1
        assert np.abs(lse[i] - math.log(vis)).max() < 1e-4, (i, lse[i], math.log(vis))
        want = csum[vis - 1] / vis                            # [Hkv, D]
        for h in range(HQ):
            assert np.abs(o[i, h] - want[h // G]).max() < 1e-2 + 1e-2 * np.abs(want[h // G]).max(), (i, h)


def test_graded_needles_on_the_tcgen05_path_pin_the_causal_edge_to_the_position():
    """Needle keys of growing strength at the edges of 64-key tiles and of pages, inside the resumed chunk and in the
    prefix: a query's output must be the V row of the strongest needle it is allowed to see, i.e. of the LAST one at
    or before its own position - one position early or late picks another row."""
    import torch
    from paper_2608_10402_b200 import tide
    rng = np.random.default_rng(5)
    p, n = 2000, 130                                          # 910 packed rows: four row tiles, the last one ragged
    L = p + n
    scale = 1.0 / math.sqrt(D)
    k = np.zeros((L, HKV, D), np.uint16)
    v = inputs.normal_bf16(rng, (L, HKV, D))
    q = inputs.f32_to_bf16_bits(np.full((n, HQ, D), 2.0, np.float32))
    # absolute positions: prefix (tile edge 1023|1024, last prefix key), then the chunk: its first key, the 64-key
    # tile edge at 2047|2048, page edges 2063|2064 and 2079|2080, a mid-page key, the last key
    base = [1023, 1024, p - 1, p, 2047, 2048, 2063, 2064, 2079, 2080, 2101, L - 1]
    needles = {}
    for g in range(HKV):
        pos = sorted({min(L - 1, x + (g if x not in (p - 1, p, L - 1) else 0)) for x in base})
        needles[g] = pos
        for rank, j in enumerate(pos):
            # logit = 2 * strength * 128 * scale = 22.6 * strength: each needle outweighs the one before by e^5.7 ...
            k[j, g] = inputs.f32_to_bf16_bits(np.full(D, 1.0 + 0.25 * rank, np.float32))
    # ... which leaves 0.3 % of the weight to the runner-up; the tolerance below allows for it
    o, lse, plan = _run_row(tide, torch, p, n, k, v, q, scale)
    vf = H.oa.bf16_bits_to_f64(v)
    for i in range(n):
        for h in range(HQ):
            g = h // G
            seen = [j for j in needles[g] if j <= p + i]
            top = seen[-1]
            want = vf[top, g]
            if len(seen) > 1:
                want = (want + math.exp(-0.25 * 2 * D * scale) * vf[seen[-2], g]) / (1 + math.exp(-0.25 * 2 * D * scale))
            assert np.abs(o[i, h] - want).max() < 3e-2, (i, h, top)
