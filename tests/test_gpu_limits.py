"""The limits of the configuration, reached exactly: empty calls, a page-table row filled to its last slot, a pool
handed out to its last page, a batch of max_batch_rows rows and max_batch_tokens tokens, and a decode row long
enough to be cut into the most KV splits the planner allows.  What fits must match the oracle; one more must be
refused with nothing changed."""
import math

import numpy as np
import pytest

from oracle import cbuild
from oracle.paged_kv import PagedKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _fails(tide, code, fn):
    with pytest.raises(tide.TideError) as e:
        fn()
    assert e.value.code == code


def test_empty_calls_are_no_ops():
    import torch
    from paper_2608_10402_b200 import tide
    kv = tide.TideKV(8, 2, 64, 16, 8, 2, 4, 2, 16, num_layers=2)
    z = torch.zeros((1, 2, 64), dtype=torch.int16, device="cuda")
    q = torch.zeros((1, 8, 64), dtype=torch.int16, device="cuda")
    kv.append([], [0], z, z)
    kv.extend([], [0])
    kv.write(1, [], [0], z, z)
    kv.attend([], q, 0.125, q)
    kv.release_many([])
    kv.step_begin([])
    kv.alloc(0)
    kv.append([0], [0, 0], z, z)              # a zero-length entry
    assert kv.task_len(0) == 0 and len(kv.page_table(0)) == 0
    assert kv.usage() == (0, 8)
    kv.prune(0, 0, 0)
    kv.truncate(0, 0)
    k, v = kv.read(0)
    assert k.shape[0] == 0
    assert kv.status() == tide.OK
    kv.close()


def test_full_page_table_row_and_full_pool():
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = 8, 2, 64, 16
    MAXP, NPAGES = 40, 64
    rng = np.random.default_rng(3)
    scale = 1.0 / math.sqrt(D)
    kv = tide.TideKV(HQ, HKV, D, S, NPAGES, 3, MAXP, 3, 700)
    orc = PagedKVOracle(NPAGES, S, HKV, D, 3, MAXP)
    for t in range(3):
        kv.alloc(t)
        orc.alloc(t)
    full = MAXP * S                                   # task 0 fills its row to the last slot
    k, v = inputs.normal_bf16(rng, (full, HKV, D)), inputs.normal_bf16(rng, (full, HKV, D))
    kv.append([0], [0, full - 1], H.to_dev(k[:-1], torch), H.to_dev(v[:-1], torch))
    orc.append([0], [0, full - 1], k[:-1], v[:-1])
    kv.append([0], [0, 1], H.to_dev(k[-1:], torch), H.to_dev(v[-1:], torch))
    orc.append([0], [0, 1], k[-1:], v[-1:])
    assert kv.task_len(0) == full and len(kv.page_table(0)) == MAXP
    z = torch.zeros((64, HKV, D), dtype=torch.int16, device="cuda")
    _fails(tide, tide.ERR_TABLE_FULL, lambda: kv.append([0], [0, 1], z, z))
    # the pool: 24 pages are left; task 1 takes all of them but one token's worth, then exactly the rest
    left = (NPAGES - MAXP) * S
    k1, v1 = inputs.normal_bf16(rng, (left, HKV, D)), inputs.normal_bf16(rng, (left, HKV, D))
    kv.append([1], [0, left - S], H.to_dev(k1[:left - S], torch), H.to_dev(v1[:left - S], torch))
    orc.append([1], [0, left - S], k1[:left - S], v1[:left - S])
    _fails(tide, tide.ERR_NO_PAGES, lambda: kv.append([1, 2], [0, S, S + 1], z, z))      # all-or-nothing: needs 2 pages
    kv.append([1], [0, S], H.to_dev(k1[left - S:], torch), H.to_dev(v1[left - S:], torch))
    orc.append([1], [0, S], k1[left - S:], v1[left - S:])
    assert kv.usage() == (full + left, 0) == (orc.used_tokens(), orc.free_pages())
    _fails(tide, tide.ERR_NO_PAGES, lambda: kv.append([2], [0, 1], z, z))
    _fails(tide, tide.ERR_NO_PAGES, lambda: kv.fork(1, 2) if left % S else kv.append([2], [0, 1], z, z))
    for t in (0, 1):
        assert np.array_equal(kv.page_table(t), orc.page_table(t))
    # attention over the full-length task (every query of its last 600 tokens) and the other one
    rows = [(0, 600, full), (1, 1, left), (0, 1, full)]
    q = inputs.normal_bf16(rng, (602, HQ, D))
    out = torch.zeros((602, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((602, HQ), dtype=torch.float32, device="cuda")
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, "full table row")
    _fails(tide, tide.ERR_WORKSPACE, lambda: kv.attend([(0, 600, full), (1, 101, left)], torch.zeros((701, HQ, D), dtype=torch.int16, device="cuda"),
                                                       scale, torch.zeros((701, HQ, D), dtype=torch.int16, device="cuda")))
    for t in (0, 1):
        gk, gv = kv.read(t)
        ok, ov = orc.read(t)
        assert np.array_equal(H.from_dev(gk), ok) and np.array_equal(H.from_dev(gv), ov)
    kv.close()


def test_batch_of_max_rows_and_most_kv_splits():
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = 4, 1, 128, 16
    B = 256
    LONG = 65536                                      # 128 chunks of 512 keys: the most splits the planner allows
    rng = np.random.default_rng(4)
    scale = 1.0 / math.sqrt(D)
    lens = [int(x) for x in rng.integers(1, 40, size=B - 1)] + [LONG]
    num_pages = sum((n + S - 1) // S for n in lens) + 2
    maxp = (LONG + S - 1) // S
    kv = tide.TideKV(HQ, HKV, D, S, num_pages, B, maxp, B, B)
    orc = PagedKVOracle(num_pages, S, HKV, D, B, maxp)
    indptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(indptr[-1])
    k, v = inputs.normal_bf16(rng, (T, HKV, D)), inputs.normal_bf16(rng, (T, HKV, D))
    for t in range(B):
        kv.alloc(t)
        orc.alloc(t)
    kv.append(list(range(B)), indptr, H.to_dev(k, torch), H.to_dev(v, torch))
    orc.append(list(range(B)), indptr, k, v)
    rows = [(t, 1, lens[t]) for t in range(B)]                      # max_batch_rows rows, max_batch_tokens tokens
    q = inputs.normal_bf16(rng, (B, HQ, D))
    out = torch.zeros((B, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((B, HQ), dtype=torch.float32, device="cuda")
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse)
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, "max rows")
    plan = kv.last_plan()
    assert plan["decode_items"] >= B - 1 + 128, plan             # the long row went out as 128 KV splits
    _fails(tide, tide.ERR_WORKSPACE, lambda: kv.attend(rows + [(0, 1, 1)], H.to_dev(np.concatenate([q, q[:1]]), torch), scale,
                                                       torch.zeros((B + 1, HQ, D), dtype=torch.int16, device="cuda")))
    kv.close()
