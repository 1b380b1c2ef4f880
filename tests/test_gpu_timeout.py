"""The bounded waits inside the attention kernels, made to run out WITHOUT any fault: a test hook lets the K/V
producer of one work item leave out the first stage, so the consumers' wait for it reaches its (shortened) time
limit.  The kernel must return by itself, tide_status must report the time-out exactly once, and the same handle
must then compute correct attention again."""
import math
import time

import numpy as np
import pytest

from oracle import cbuild
from oracle.paged_kv import PagedKVOracle
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kind,geom,p,n", [("warp-MMA decode kernel", (8, 2, 64, 16), 300, 1),
                                           ("warp-MMA decode kernel, head size 128", (28, 4, 128, 16), 700, 1),
                                           ("warp-MMA tile kernel", (8, 2, 64, 16), 150, 40),
                                           ("tcgen05 kernel", (28, 4, 128, 16), 200, 40)])
def test_a_wait_that_runs_out_is_reported_once_and_the_handle_stays_usable(kind, geom, p, n):
    import torch
    from paper_2608_10402_b200 import tide
    HQ, HKV, D, S = geom
    rng = np.random.default_rng(p + n)
    L = p + n
    pages = (L + S - 1) // S + 2
    kv = tide.TideKV(HQ, HKV, D, S, pages, 2, pages, 2, max(n, 4))
    orc = PagedKVOracle(pages, S, HKV, D, 2, pages)
    k, v = inputs.normal_bf16(rng, (L, HKV, D)), inputs.normal_bf16(rng, (L, HKV, D))
    for o in (kv, orc):
        o.alloc(0)
    kv.append([0], [0, L], H.to_dev(k, torch), H.to_dev(v, torch))
    orc.append([0], [0, L], k, v)
    rows = [(0, n, L)]
    q = inputs.normal_bf16(rng, (n, HQ, D))
    scale = 1.0 / math.sqrt(D)
    out = torch.zeros((n, HQ, D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((n, HQ), dtype=torch.float32, device="cuda")
    assert kv.status() == tide.OK

    kv.tune(tide.TUNE_WAIT_LIMIT_US, 2000)                    # 2 ms instead of 2 s
    kv.tune(tide.TUNE_DROP_FIRST_STAGE, 1)                    # armed for the next attention call only
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse)      # the call itself is asynchronous and succeeds
    st = kv.status()                                          # synchronises: the kernel came back by itself
    elapsed = time.perf_counter() - t0
    assert st == tide.ERR_DEVICE_TIMEOUT, f"{kind}: status {st}"
    assert elapsed < 2.0, f"{kind}: {elapsed:.3f} s for waits bounded at 2 ms"
    assert kv.status() == tide.OK                             # reported once, then cleared

    kv.tune(tide.TUNE_WAIT_LIMIT_US, 2_000_000)
    out.zero_()
    lse.zero_()
    kv.attend(rows, H.to_dev(q, torch), scale, out, lse)      # the hook is spent: this is an ordinary call
    assert kv.status() == tide.OK
    ref_o, ref_l = cbuild.attend_paged(orc, rows, q, scale)
    H.check_outputs(H.from_dev(out), lse.cpu().numpy(), ref_o, ref_l, kind + " after the time-out")
    gk, gv = kv.read(0)
    assert np.array_equal(H.from_dev(gk), k) and np.array_equal(H.from_dev(gv), v)     # the cache was never touched
    kv.close()
