"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  The ResNet-50-, VGG-16- and ViT-B/16-shaped sets are compared on EVERY
element in both lookahead modes (the oracle runs on all host cores).  For the
1 B-parameter set the oracle follows a fixed sample of elements (small tensors
whole, both ends of every tensor, a stride-997 comb); that is exact for the
sampled elements because the step has no cross-element term."""
import os

import pytest
import torch

import harness
from harness import FullPair, SampledPair
from paper_2601_07876_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CORES = max(1, len(os.sched_getaffinity(0)))


def _report(pair, wl, mode, compared):
    print(f"\nPARITY {wl.name} {mode} steps={wl.steps} compared={compared} worst |err|/tol: "
          + ", ".join(f"{k.split()[-1]} {v:.3f}" for k, v in harness.MARGINS.items())
          + "; moments relative to their rms: "
          + ", ".join(f"{k.split()[-1]} {v:.2e}" for k, v in harness.SCALED.items()))
    k = pair.hyper["lookahead_k"]
    assert pair.sync_steps == list(range(k, wl.steps + 1, k))
    assert pair.rect_flags == [0] * 5 + [1] * (wl.steps - 5)
    info = pair.opt.info()
    assert info["launches"] == wl.steps and info["total_numel"] == wl.total
    misaligned = bool(info["warnings"] & 2)
    assert not misaligned, "every tensor should run on 128-bit accesses"


@pytest.mark.parametrize("index,mode", [(1, "last"), (1, "traj_mean"), (2, "last"),
                                        (2, "traj_mean"), (3, "last"), (3, "traj_mean")])
def test_fullsize_workload_every_element(index, mode):
    wl = W.get_workload(index)
    free, _ = torch.cuda.mem_get_info()
    need = wl.total * 4 * 8
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory")
    harness.MARGINS.clear()
    harness.SCALED.clear()
    pair = FullPair(wl, DEV, dict(lookahead_mode=mode))
    for _ in range(wl.steps):
        pair.step(threads=CORES)
    pair.check()
    assert pair.compared == wl.total
    _report(pair, wl, mode, pair.compared)
    del pair
    torch.cuda.empty_cache()


@pytest.mark.parametrize("mode", ["last", "traj_mean"])
def test_fullsize_1b_set_on_a_sample(mode):
    wl = W.get_workload(4)
    free, _ = torch.cuda.mem_get_info()
    need = wl.total * 4 * 8
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory")
    harness.MARGINS.clear()
    harness.SCALED.clear()
    pair = SampledPair(wl, DEV, dict(lookahead_mode=mode))
    for _ in range(wl.steps):
        pair.step(threads=min(8, CORES))
    pair.check()
    _report(pair, wl, mode, pair.idx.numel())
    del pair
    torch.cuda.empty_cache()


def test_one_tensor_beyond_2_to_the_31_elements():
    """Maximum sizes: element offsets past 2^31 (and chunk counts past 2^20) in one
    tensor, with clipping on so that the statistics kernels cross the boundary too.
    The oracle follows a sample: both ends, a window around element 2^31 and a comb."""
    n = (1 << 31) + 4099                       # ragged: not a multiple of 4
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * (1 << 30):
        pytest.skip("needs about 45 GiB of device memory")
    from oracle import novak_oracle as O
    from paper_2601_07876_b200 import binding as B
    gen = torch.Generator(device=DEV).manual_seed(5)
    p = torch.empty(n, dtype=torch.float32, device=DEV)
    g = torch.empty(n, dtype=torch.float32, device=DEV)
    blk = 1 << 28
    for lo in range(0, n, blk):
        p[lo:lo + blk].normal_(0.0, 0.05, generator=gen)
    edge = 4096
    idx = torch.cat([torch.arange(edge), torch.arange((1 << 31) - edge, (1 << 31) + edge),
                     torch.arange(edge, n - edge, 1000003), torch.arange(n - edge, n)]).to(DEV)
    hyper = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
                 nesterov="approximation", lookahead_k=0, clip_threshold=1.0)
    opt = B.NovakOptimizer([p], **hyper)
    oracle = O.Oracle(harness.oracle_config(dict(hyper, clip_threshold=0.0)),
                      [harness.to_f64(p[idx])])
    for _ in range(3):
        for lo in range(0, n, blk):
            g[lo:lo + blk].normal_(0.0, 1e-3, generator=gen)
        opt.step([g])
        norm, factor = opt.grad_stats()
        # the sample cannot know the global norm: take it from a plain float64 torch sum
        want = float(sum(g[lo:lo + blk].double().square().sum() for lo in range(0, n, blk)) ** 0.5)
        assert abs(norm - want) <= 1e-7 * want and want > 1.0
        assert abs(factor - 1.0 / want) <= 1e-6 / want
        oracle.step([harness.to_f64(g[idx]) * (1.0 / want)])
    torch.cuda.synchronize()
    info = opt.info()
    assert info["total_numel"] == n and info["n_chunks"] == (n + 2047) // 2048
    harness.assert_close(p[idx], oracle.theta[0], "2^31 theta")
    harness.assert_close(opt.state(0)["m"][idx], oracle.m[0], "2^31 m")
    harness.assert_close(opt.state(0)["v"][idx], oracle.v[0], "2^31 v")
    del opt, p, g
    torch.cuda.empty_cache()
