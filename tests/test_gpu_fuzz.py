"""Seeded random combinations of everything the step can be asked to do, on a small
ragged multi-tensor set, against the oracle: variant x lookahead x rectification x
phase 2 x adaptive beta x layer adaptation x auto-LR x gradient type x hyperparameter
values x entry size x (plain | graph-capturable) step.  Each case is a fixed seed."""
import numpy as np
import pytest
import torch

from harness import Pair, make_tensors

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SHAPES = [(8, 3, 3, 3), (33,), (10, 257), (3, 5000), (4097, 2), (1, 7), (2048,), (6, 2048),
          (7, 1000, 3), (1,)]
OFFSETS = [0, 1, 0, 3, 0, 2, 0, 0, 1, 0]


def _case(seed):
    r = np.random.default_rng(seed)
    pick = lambda xs: xs[int(r.integers(len(xs)))]
    hyper = dict(
        lr=float(10.0 ** r.uniform(-4, -2)), betas=(float(r.uniform(0.5, 0.95)),
                                                    float(pick([0.9, 0.99, 0.999]))),
        eps=float(pick([1e-8, 1e-6])), weight_decay=float(pick([0.0, 1e-2, 0.1])),
        nesterov=pick(["none", "approximation", "classical"]),
        nesterov_beta=pick([None, float(r.uniform(0.1, 0.95))]),
        lookahead_k=int(pick([0, 1, 2, 3, 5])), lookahead_alpha=float(r.uniform(0.2, 0.8)),
        lookahead_mode=pick(["last", "traj_mean"]), rectified=bool(r.integers(2)),
        clip_threshold=float(pick([0.0, 0.02, 10.0])), centralize=bool(r.integers(2)),
        adaptive_beta=bool(r.integers(2)), layer_adaptation=bool(r.integers(2)),
        auto_lr=bool(r.integers(2)))
    kwargs = dict(chunk_elems=int(pick([1024, 2048, 4096])),
                  graph_capturable=bool(r.integers(2)))
    gdtype = pick([torch.float32, torch.bfloat16])
    return hyper, kwargs, gdtype, int(r.integers(1 << 30))


@pytest.mark.parametrize("seed", range(48))
def test_random_combination(seed):
    hyper, kwargs, gdtype, gseed = _case(seed)
    numels = [int(np.prod(s)) for s in SHAPES]
    _, views, _ = make_tensors(numels, DEV, OFFSETS)
    gen = torch.Generator(device=DEV).manual_seed(gseed)
    params = [v.view(s) for v, s in zip(views, SHAPES)]
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    pair = Pair(params, hyper, opt_kwargs=kwargs)
    for t in range(9):
        _, gv, _ = make_tensors(numels, DEV, OFFSETS, dtype=gdtype)
        grads = [v.view(s) for v, s in zip(gv, SHAPES)]
        for g in grads:
            g.copy_(torch.empty(g.shape, device=DEV).normal_(2e-4, 10.0 ** (-3 + 0.2 * t), generator=gen))
        pair.step(grads)
        if hyper["clip_threshold"] > 0:
            pair.record_grad_stats()
    pair.check(f"seed {seed}: {hyper} {kwargs} {gdtype}")
