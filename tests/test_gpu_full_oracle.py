"""Every query of a full-size batch against the float64 oracle, element by element (not a sample).

The decode-only batch (64 rows) costs the oracle a second, and the mixed multi-turn text resume batch at its full
size (128 tasks, 96 decode rows, 32 resume rows of 200..2000 appended tokens over contexts of 2k..32k) about three
minutes on 16 host cores: both run with the routine GPU tests.  The long-horizon stress batch (230 decode rows and
26 resume rows of 500..4000 tokens over contexts up to 128k) costs it another three minutes and the multimodal
resume batch (32 rows of 1000..3000 image tokens over contexts up to 64k) 23: they run when
TIDE_FULL_ORACLE_ALL=1.  With TIDE_REPORT_DIR set, a per-row
table (worst error / tolerance, largest absolute error, relative Frobenius error, LSE error) is written there as
full_oracle_config<k>.md; profiles/ holds the committed copies.

    TIDE_FULL_ORACLE_ALL=1 TIDE_REPORT_DIR=<dir> python -m pytest tests/test_gpu_full_oracle.py -m gpu -q -s
"""
import os
import time

import numpy as np
import pytest

from oracle import cbuild
from paper_2608_10402_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

CASES = [2, 3] + ([4, 5] if os.environ.get("TIDE_FULL_ORACLE_ALL") == "1" else [])


@pytest.mark.parametrize("index", CASES)
def test_every_query_of_the_full_size_batch_against_the_oracle(index):
    import torch
    from paper_2608_10402_b200 import tide
    w = inputs.make_workload(index)
    kv_bits = [w.task_kv(b) for b in range(w.B)]
    q_bits = np.concatenate([w.task_q(b) for b in range(w.B)])
    c, indptr, nk, nv = H.oracle_fill(w, kv_bits)
    kv = H.gpu_fill(w, kv_bits, nk, nv, indptr, tide, torch)
    H.compare_bookkeeping(w, c, kv)
    total_q = q_bits.shape[0]
    out = torch.zeros((total_q, w.Hq, w.D), dtype=torch.int16, device="cuda")
    lse = torch.zeros((total_q, w.Hq), dtype=torch.float32, device="cuda")
    kv.attend(w.rows(), H.to_dev(q_bits, torch), w.scale, out, lse)
    assert kv.status() == tide.OK
    plan = kv.last_plan()
    got_o, got_l = H.from_dev(out), lse.cpu().numpy()
    kv.close()
    del kv
    torch.cuda.empty_cache()

    t0 = time.time()
    ref_o, ref_l = H.oracle_attend(c, w, q_bits)              # every query of every row
    oracle_s = time.time() - t0
    qoff = np.concatenate([[0], np.cumsum(w.n_new)])
    lines, worst_all = [], 0.0
    for b in range(w.B):
        a, e = int(qoff[b]), int(qoff[b + 1])
        st = H.check_outputs(got_o[a:e], got_l[a:e], ref_o[a:e], ref_l[a:e], f"configs[{index - 1}] row {b}")
        worst_all = max(worst_all, st["worst_ratio"])
        if w.n_new[b] > 1:
            lines.append(f"| {b} | {int(w.prefix[b])} | {int(w.n_new[b])} | {st['worst_ratio']:.3f} | {st['max_abs']:.2e} | "
                         f"{st['rel_fro']:.2e} | {st['lse_err']:.1e} |")
    total = H.check_outputs(got_o, got_l, ref_o, ref_l, f"configs[{index - 1}] whole batch")
    dec = w.n_new == 1
    idx = np.concatenate([np.arange(qoff[b], qoff[b + 1]) for b in range(w.B) if dec[b]]) if dec.any() else np.zeros(0, np.int64)
    dec_stats = H.check_outputs(got_o[idx], got_l[idx], ref_o[idx], ref_l[idx], "decode rows") if idx.size else None
    print(f"configs[{index - 1}]: {total_q} queries x {w.Hq} heads, oracle {oracle_s:.0f} s on {cbuild.threads()} threads, {total}")
    out_dir = os.environ.get("TIDE_REPORT_DIR", "")
    if out_dir and os.path.isdir(out_dir):
        with open(os.path.join(out_dir, f"full_oracle_config{index}.md"), "w") as f:
            f.write(f"# Full-oracle pass, configs[{index - 1}] ({w.name}), full size\n\n"
                    "Command: `TIDE_FULL_ORACLE_ALL=1 TIDE_REPORT_DIR=<dir> python -m pytest tests/test_gpu_full_oracle.py -m gpu -q -s`\n\n"
                    f"Every one of the {total_q} queries x {w.Hq} heads x {w.D} output elements of one tide_attend call over the whole "
                    f"batch ({w.B} rows: {int(dec.sum())} decode, {int((~dec).sum())} resume) compared with the float64 oracle "
                    f"({oracle_s:.0f} s on {cbuild.threads()} host threads).  Plan: {plan}.\n\n"
                    f"Tolerance: |gpu - oracle| <= {H.ATOL} + {H.RTOL} |oracle| (column `worst` = largest error / tolerance, must be <= 1), "
                    f"LSE within {H.LSE_TOL}, relative Frobenius error <= {H.REL_FRO_MAX}.\n\n"
                    f"Whole batch: worst {total['worst_ratio']:.3f}, max abs {total['max_abs']:.2e}, relFro {total['rel_fro']:.2e}, "
                    f"LSE err {total['lse_err']:.1e}.\n")
            if dec_stats:
                f.write(f"Decode rows together: worst {dec_stats['worst_ratio']:.3f}, max abs {dec_stats['max_abs']:.2e}, "
                        f"relFro {dec_stats['rel_fro']:.2e}, LSE err {dec_stats['lse_err']:.1e}.\n")
            f.write("\nResume rows:\n\n| row | prefix | new tokens | worst | max abs | relFro | LSE err |\n|---|---|---|---|---|---|---|\n")
            f.write("\n".join(lines) + "\n")
    assert worst_all <= 1.0
