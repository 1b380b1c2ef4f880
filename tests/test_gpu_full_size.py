"""GPU parity at the workloads' full sizes, in the launch configuration bench.py times (same library calls:
per-task prefix appends, one step append, one tide_attend).  Page tables, lengths and cache bits of every task
are compared exactly; attention outputs are compared on a stratified sample of (row, query) items the float64
oracle computes one by one (every decode row; first / last / page-boundary / image-text-boundary and random
queries of every resume row)."""
import numpy as np
import pytest

from paper_2608_10402_b200 import inputs
from tests.test_gpu_parity import run_workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2608_10402_b200 import tide
    assert torch.cuda.is_available()
    return tide, torch


@pytest.mark.parametrize("index", [2, 3, 4, 5])
def test_full_size_config_sampled_oracle(env, index):
    tide, torch = env
    w = inputs.make_workload(index)
    stats = run_workload(w, tide, torch, full_oracle=False, seed=index)
    print(f"config {index}: {stats}")
