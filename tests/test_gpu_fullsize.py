"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  The oracle runs on a fixed sample of elements (small tensors whole,
both ends of every tensor, a stride-997 comb); that is exact for the sampled
elements because the step has no cross-element term."""
import pytest
import torch

import harness
from harness import SampledPair
from paper_2601_07876_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("index,mode", [(1, "last"), (1, "traj_mean"), (2, "last"),
                                        (3, "last"), (3, "traj_mean"), (4, "last"),
                                        (4, "traj_mean")])
def test_fullsize_workload(index, mode):
    wl = W.get_workload(index)
    free, _ = torch.cuda.mem_get_info()
    need = wl.total * 4 * 8
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory")
    harness.MARGINS.clear()
    pair = SampledPair(wl, DEV, dict(lookahead_mode=mode))
    for _ in range(wl.steps):
        pair.step(threads=8)
    pair.check()
    print(f"\nPARITY {wl.name} {mode} steps={wl.steps} sampled={pair.idx.numel()} worst |err|/tol: "
          + ", ".join(f"{k.split()[-1]} {v:.3f}" for k, v in harness.MARGINS.items()))
    k = pair.hyper["lookahead_k"]
    assert pair.sync_steps == list(range(k, wl.steps + 1, k))
    assert pair.rect_flags == [0] * 5 + [1] * (wl.steps - 5)
    info = pair.opt.info()
    assert info["launches"] == wl.steps and info["total_numel"] == wl.total
    misaligned = bool(info["warnings"] & 2)
    assert not misaligned, "every tensor should run on 128-bit accesses"
    del pair
    torch.cuda.empty_cache()
