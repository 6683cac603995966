"""Two CPU processes (gloo) each own half of a parameter group: the sharded
run reproduces the unsharded one bit for bit and the ranks agree on the step
counter and on the lookahead synchronisation steps.  The optimizer arithmetic
in this test is the CPU oracle (the CUDA step needs a GPU); what is under test
is the partition and the rank agreement."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NUMEL = [5, 64, 1000, 3, 70001, 128]
STEPS = 7


def _inputs():
    rng = np.random.default_rng(42)
    theta = [rng.normal(0, 0.05, n) for n in NUMEL]
    grads = [[rng.normal(0, 1e-2, n) for n in NUMEL] for _ in range(STEPS)]
    return theta, grads


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from oracle import novak_oracle as O
    from paper_2601_07876_b200 import sharding
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    theta, grads = _inputs()
    mine = sharding.partition_flat(NUMEL, world)[rank]
    cfg = O.Config(lookahead_k=3, lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN)
    o = O.Oracle(cfg, [theta[t][a:b] for t, a, b in mine])
    for s in range(STEPS):
        o.step([grads[s][t][a:b] for t, a, b in mine])
    # ranks agree on counters before anything is published
    meta = [None] * world
    dist.all_gather_object(meta, (o.t, tuple(o.sync_steps), tuple(o.rect_flags)))
    assert all(m == meta[0] for m in meta)
    gathered = [None] * world
    dist.all_gather_object(gathered, [(t, a, b, th) for (t, a, b), th in zip(mine, o.theta)])
    if rank == 0:
        full = [np.zeros(n) for n in NUMEL]
        for part in gathered:
            for t, a, b, th in part:
                full[t][a:b] = th
        np.savez(os.path.join(out_dir, "sharded.npz"), *full)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharded_run_equals_unsharded(tmp_path):
    from oracle import novak_oracle as O
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    theta, grads = _inputs()
    ref = O.Oracle(O.Config(lookahead_k=3, lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN), theta)
    for s in range(STEPS):
        ref.step(grads[s])
    got = np.load(os.path.join(str(tmp_path), "sharded.npz"))
    for i, want in enumerate(ref.theta):
        assert np.array_equal(got[f"arr_{i}"], want)
    assert ref.sync_steps == [3, 6]
