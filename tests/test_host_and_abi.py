"""CPU-only checks: the C-ABI library loads and exports every symbol include/tide.h declares (no compute
calls), the host-side size query works, the workload generators match the configured shapes, and the
multi-rank bookkeeping of the replicas path agrees across two gloo ranks."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tide():
    from paper_2608_10402_b200 import build
    build.build()
    from paper_2608_10402_b200 import tide as t
    return t


def test_library_exports_every_declared_symbol(tide):
    header = open(os.path.join(ROOT, "include", "tide.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(tide_[a-z_0-9]+)\s*\(", header))
    assert {"tide_kv_alloc", "tide_kv_append", "tide_attend", "tide_kv_release"} <= declared
    lib = ctypes.CDLL(tide.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/tide.h but not exported"
    assert declared == set(tide.EXPORTS), "binding and header disagree on the entry points"


def test_strerror_and_size_query_need_no_gpu(tide):
    assert tide.strerror(0) == "ok" and "pages" in tide.strerror(tide.ERR_NO_PAGES)
    cfg = tide.make_config(28, 4, 128, 16, 1000, 8, 64, 8, 512)
    pool, ws = tide.tide_kv_required_bytes(cfg)
    assert pool == 1000 * 4 * 2 * 128 * 16 * 2            # pages * Hkv * (K,V) * D * S * 2 bytes
    assert ws > 8 * 64 * 4
    bad = tide.make_config(28, 5, 128, 16, 1000, 8, 64, 8, 512)      # Hq % Hkv != 0
    with pytest.raises(tide.TideError) as e:
        tide.tide_kv_required_bytes(bad)
    assert e.value.code == tide.ERR_INVALID_ARG
    for kw in (dict(D=96), dict(S=8)):
        c = tide.make_config(8, 2, kw.get("D", 64), kw.get("S", 16), 10, 2, 4, 2, 16)
        with pytest.raises(tide.TideError):
            tide.tide_kv_required_bytes(c)


def test_workload_shapes_follow_the_configs():
    from paper_2608_10402_b200 import inputs
    K = 1024
    w1 = inputs.make_workload(1)
    assert (w1.B, w1.Hq, w1.Hkv, w1.D, w1.S) == (4, 8, 2, 64, 16) and w1.scale == 0.125
    assert sorted(w1.n_new)[:2] == [1, 1] and all(32 <= n <= 64 for n in sorted(w1.n_new)[2:])
    assert all(200 <= p <= 600 for p in w1.prefix)
    w2 = inputs.make_workload(2)
    assert w2.B == 64 and (w2.n_new == 1).all() and w2.prefix.min() >= K and w2.prefix.max() == 32 * K
    assert (w2.Hq, w2.Hkv, w2.D, w2.S) == (28, 4, 128, 16) and w2.num_pages >= 4 * w2.live_pages()
    w3 = inputs.make_workload(3)
    assert w3.B == 128 and int((w3.n_new == 1).sum()) == 96
    res = w3.n_new[w3.n_new > 1]
    assert len(res) == 32 and res.min() >= 200 and res.max() <= 2000 and w3.prefix.min() >= 2 * K
    w4 = inputs.make_workload(4)
    assert w4.B == 32 and (w4.Hq, w4.Hkv) == (32, 8) and (w4.n_new > 1).all()
    assert ((w4.n_image >= 1000) & (w4.n_image <= 3000)).all()
    assert (((w4.n_new - w4.n_image) >= 50) & ((w4.n_new - w4.n_image) <= 200)).all()
    assert w4.prefix.min() >= 4 * K and w4.prefix.max() == 64 * K
    w5 = inputs.make_workload(5)
    assert w5.B == 256 and w5.S == 32 and int((w5.n_new > 1).sum()) == 26 and w5.prefix.max() == 128 * K
    for w in (w1, w2, w3, w4, w5):
        assert np.array_equal(np.sort(w.free_order), np.arange(w.num_pages))
        assert w.max_pages_per_task >= ((w.ctx + w.S - 1) // w.S).max()
    # image tokens really are wider: K/V of the image part ~ N(0, 1.5)
    small = inputs.make_workload(4, n_tasks=2, len_div=16)
    k, _ = small.task_kv(0)
    p, ni = int(small.prefix[0]), int(small.n_image[0])
    img = inputs.bf16_bits_to_f32(k[p:p + ni]).std()
    txt = inputs.bf16_bits_to_f32(k[:p]).std()
    assert 1.4 < img < 1.6 and 0.95 < txt < 1.05
    # determinism and bf16 rounding (nearest even)
    again = inputs.make_workload(4, n_tasks=2, len_div=16)
    assert np.array_equal(again.task_kv(0)[0], k)
    x = np.array([1.0, 1.00390625, 1.01171875, -3.140625], dtype=np.float32)   # 1 + 2^-8 ties to even
    assert list(inputs.f32_to_bf16_bits(x)) == [0x3F80, 0x3F80, 0x3F82, 0xC049]
    h = inputs.hashed_bf16_bits(7, 100, 5, 2, 8, 1)
    assert h.shape == (5, 2, 8) and np.array_equal(h, inputs.hashed_bf16_bits(7, 100, 5, 2, 8, 1))
    assert np.isfinite(inputs.bf16_bits_to_f32(h)).all()


RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
from paper_2608_10402_b200 import replicas
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
times, totals = replicas.reduce_step_stats([10.0 + 5 * rank, 2.0 - rank], [100.0 * (rank + 1), 7.0], 2, dist, "cpu")
assert times == [15.0, 2.0] and totals == [300.0, 14.0], (times, totals)
assert replicas.whole_job_rate(totals[0], times[0]) == 300.0 / 0.015
assert replicas.rank_seed(1003, rank) == 1003 + 7919 * rank
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_replica_bookkeeping_two_gloo_ranks(tmp_path):
    port = 29500 + (os.getpid() % 2000)
    script = tmp_path / "rank.py"
    script.write_text(RANK_SCRIPT % (ROOT, port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                              text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, o
        assert f"rank {r} ok" in o


def test_reference_arm_of_bench_prints_the_contract_line():
    """`bench.py --impl reference` times the oracle on the host cores and needs no GPU: one JSON line with the
    contract's keys, the oracle's dtype, and an end-to-end entry without transfers."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                          "--config", "1"], capture_output=True, text=True, timeout=300, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["dtype"] == "f64" and line["vs_baseline"] is None
    assert line["steps"] == 2 and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in line["config"]


def test_bench_gpus_flag_starts_that_many_replica_ranks_by_itself():
    """`bench.py --gpus 2` from a plain process (no launcher in the environment) must start two ranks by itself and
    print ONE line that says n_gpus 2; the reference arm needs no GPU, so this runs on CPU."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "1", "--config", "1"], capture_output=True, text=True, timeout=600, cwd=root, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    assert lines[0]["n_gpus"] == 2 and lines[0]["impl"] == "reference"
    assert lines[0]["config"]["requested"] == {"steps": 1, "warmup": 1} and "clamp" in lines[0]["config"]
