"""tide_attend_decode_static — the entry point for callers that cannot allocate (code running during a
global-mode CUDA graph capture, processes whose allocator already owns the device, steps that must avoid
cudaMalloc's device-wide synchronisation).  Its split-KV scratch is a fixed array inside the library.

Checked here through the C ABI against the float64 oracle and against tide_attend on the same cache and
queries, on two calls in a row (the second call reuses the array with the first call's leftovers in it), within
the tolerance the parity tests use.  Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest

from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_static_scratch_attend_matches_tide_attend_twice():
    import torch
    from paper_2608_10402_b200 import tide

    # a decode-only batch with long and short contexts, so that some rows are split over KV and some are not
    w = inputs.make_workload(2, n_tasks=10, len_div=4)
    kv_bits = [w.task_kv(b) for b in range(w.B)]
    c, indptr, nk, nv = H.oracle_fill(w, kv_bits)
    kv = H.gpu_fill(w, kv_bits, nk, nv, indptr, tide, torch)
    rows = w.rows()
    total_q = int(w.n_new.sum())
    rng = np.random.default_rng(123)
    for call in range(2):
        # fresh queries each time, so a stale result cannot pass for a new one
        q = H.to_dev(inputs.normal_bf16(rng, (total_q, w.Hq, w.D)), torch)
        ref_o = torch.zeros((total_q, w.Hq, w.D), dtype=torch.int16, device="cuda")
        ref_l = torch.zeros((total_q, w.Hq), dtype=torch.float32, device="cuda")
        kv.attend(rows, q, w.scale, ref_o, ref_l)
        got_o = torch.zeros_like(ref_o)
        got_l = torch.zeros_like(ref_l)
        kv.attend_decode_static(rows, q, w.scale, got_o, got_l)
        assert kv.status() == tide.OK
        q_bits = H.from_dev(q)
        want_o, want_l = H.oracle_attend(c, w, q_bits)
        H.check_outputs(H.from_dev(got_o), got_l.cpu().numpy(), want_o, want_l, f"static entry point, call {call}")
        a = H.oa.bf16_bits_to_f64(H.from_dev(got_o))
        b = H.oa.bf16_bits_to_f64(H.from_dev(ref_o))
        assert np.isfinite(a).all()
        assert (np.abs(a - b) <= H.ATOL + H.RTOL * np.abs(b)).all(), f"call {call}: max diff {np.abs(a - b).max():.3e}"
        assert np.abs(got_l.cpu().numpy() - ref_l.cpu().numpy()).max() <= H.LSE_TOL
        assert np.linalg.norm(a - b) <= H.REL_FRO_MAX * np.linalg.norm(b)

    # beyond the fixed maximum the call refuses instead of overrunning its array
    too_many = [rows[0]] * (tide.STATIC_MAX_ROWS + 1)
    qq = torch.zeros((len(too_many), w.Hq, w.D), dtype=torch.int16, device="cuda")
    with pytest.raises(tide.TideError) as e:
        kv.attend_decode_static(too_many, qq, w.scale, torch.zeros_like(qq))
    assert e.value.code == tide.ERR_WORKSPACE
    # and it only takes decode-style rows
    t0, _, L0 = rows[0]
    with pytest.raises(tide.TideError) as e:
        kv.attend_decode_static([(t0, 8, L0)], qq, w.scale, torch.zeros_like(qq))
    assert e.value.code == tide.ERR_INVALID_ARG
    kv.close()
