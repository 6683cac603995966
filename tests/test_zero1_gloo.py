"""ZeRO-1 sharding wrapper under gloo on the CPU: two ranks with different
gradients reproduce a single process that steps on the averaged gradient, the
ranks' parameter buffers agree bit for bit after every step, and the owned
ranges cover every element exactly once.  The local step is the CPU oracle
(the CUDA step needs a GPU); the collectives and the bookkeeping are under test."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NUMEL = [5, 64, 1000, 3, 701, 128]
STEPS = 6


class _OracleLocal:
    """Local stepper for the test: the fp64 oracle behind torch views, with the same
    one-call and two-half interface as the CUDA optimizer."""

    def __init__(self, pieces, **cfg):
        from oracle import novak_oracle as O
        self.pieces = pieces
        self.o = O.Oracle(O.Config(lookahead_k=3, **cfg),
                          [p.numpy().astype(np.float64) for p in pieces])

    def _publish(self):
        for p, th in zip(self.pieces, self.o.theta):
            p.copy_(torch.from_numpy(th))

    def step(self, grads):
        self.o.step([g.numpy().astype(np.float64) for g in grads])
        self._publish()

    def step_begin(self, grads):
        self.open = [g.numpy().astype(np.float64) for g in grads]
        self.sums = self.o.local_sums(self.open)

    def copy_local_sums(self, out):
        out.copy_(torch.tensor(self.sums, dtype=torch.float64))

    def step_finish(self, totals):
        self.o.step(self.open, global_sums=(float(totals[0]), float(totals[1])))
        self._publish()


def _inputs(world):
    rng = np.random.default_rng(9)
    total = sum(NUMEL)
    theta = rng.normal(0, 0.05, total)
    grads = rng.normal(0, 1e-2, (STEPS, world, total))
    return theta, grads


def _worker(rank, world, port, out_dir, cfg=None):
    cfg = cfg or {}
    sys.path.insert(0, ROOT)
    from paper_2601_07876_b200 import zero1
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    theta, grads = _inputs(world)
    total = sum(NUMEL)
    n = zero1.padded_numel(total, world)
    flat_p = torch.zeros(n, dtype=torch.float64)
    flat_p[:total] = torch.from_numpy(theta)
    opt = zero1.ShardedNovak(flat_p, NUMEL,
                             make_local=lambda ps: _OracleLocal(ps, **cfg) if ps else None, **cfg)
    # the ranks' owned pieces cover every element of every tensor exactly once
    owned = [None] * world
    dist.all_gather_object(owned, opt.slices)
    seen = [np.zeros(k, dtype=np.int32) for k in NUMEL]
    for pieces in owned:
        assert sum(b - a for _, a, b in pieces) <= n // world
        for t, a, b in pieces:
            seen[t][a:b] += 1
    assert all((x == 1).all() for x in seen)
    for s in range(STEPS):
        flat_g = torch.zeros(n, dtype=torch.float64)
        flat_g[:total] = torch.from_numpy(grads[s, rank])
        opt.step(flat_g)
        gathered = [torch.empty_like(flat_p) for _ in range(world)]
        dist.all_gather(gathered, flat_p)
        assert all(torch.equal(gathered[0], g) for g in gathered)
    if rank == 0:
        np.save(os.path.join(out_dir, "sharded.npy"), flat_p[:total].numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_zero1_equals_one_process_on_the_mean_gradient(tmp_path):
    from oracle import novak_oracle as O
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    theta, grads = _inputs(world)
    ref = O.Oracle(O.Config(lookahead_k=3), [theta])
    for s in range(STEPS):
        ref.step([grads[s].sum(axis=0) / world])
    got = np.load(os.path.join(str(tmp_path), "sharded.npy"))
    np.testing.assert_allclose(got, ref.theta[0], rtol=1e-13, atol=1e-16)
    assert ref.sync_steps == [3, 6]


def test_two_rank_zero1_with_clipping_and_auto_lr_all_reduces_the_norms(tmp_path):
    """Clipping and auto-LR need the norms of the whole group: the two-half step with an
    all-reduce of the ranks' sums of squares reproduces one process on the mean gradient."""
    from oracle import novak_oracle as O
    world = 2
    cfg = dict(clip_threshold=0.05, auto_lr=True)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(world, port, str(tmp_path), cfg), nprocs=world, join=True)
    theta, grads = _inputs(world)
    ref = O.Oracle(O.Config(lookahead_k=3, **cfg), [theta])
    for s in range(STEPS):
        ref.step([grads[s].sum(axis=0) / world])
    got = np.load(os.path.join(str(tmp_path), "sharded.npy"))
    np.testing.assert_allclose(got, ref.theta[0], rtol=1e-12, atol=1e-15)
    assert min(ref.clip_factors) < 1.0 and len(set(ref.auto_scales)) > 1


def test_padding():
    from paper_2601_07876_b200 import zero1
    assert zero1.padded_numel(1, 2) == 128 and zero1.padded_numel(128, 2) == 128
    assert zero1.padded_numel(129, 2) == 256 and zero1.padded_numel(1000, 8) == 1024
