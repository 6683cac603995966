"""The graph-capturable step (NOVAK_OPT_GRAPH_CAPTURABLE): counters and scalars in device
memory.  Eagerly it must match the oracle like the plain step; captured once with stream
capture and replayed, every replay must be the next step (counters, sync steps and the
rectification switch at t = 6 included)."""
import numpy as np
import pytest
import torch

from harness import Pair, assert_close, make_tensors, oracle_config, to_f64
from oracle import novak_oracle as O
from paper_2601_07876_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
RAGGED = [1, 3, 33, 1025, 8193, 70001, 4096]
BASE = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
            nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5)


def _gen(seed):
    return torch.Generator(device=DEV).manual_seed(seed)


def _fresh(numels, offsets=None, seed=1, shapes=None):
    _, views, _ = make_tensors(numels, DEV, offsets)
    g = _gen(seed)
    for v in views:
        v.normal_(0.0, 0.05, generator=g)
    return [v.view(s) for v, s in zip(views, shapes)] if shapes else views


@pytest.mark.parametrize("nesterov", ["none", "approximation", "classical"])
@pytest.mark.parametrize("la", [(0, "last"), (5, "last"), (5, "traj_mean"), (1, "last")])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_eager_steps_match_the_oracle(nesterov, la, gdtype):
    k, mode = la
    offs = [(i % 4) if i % 3 == 2 else 0 for i in range(len(RAGGED))]
    params = _fresh(RAGGED, offs)
    pair = Pair(params, dict(BASE, nesterov=nesterov, lookahead_k=k, lookahead_mode=mode),
                opt_kwargs=dict(graph_capturable=True))
    gen = _gen(9)
    for t in range(12):
        _, grads, _ = make_tensors(RAGGED, DEV, offs, dtype=gdtype)
        for g in grads:
            g.copy_(torch.empty(g.shape, device=DEV).normal_(0.0, 1e-2, generator=gen))
        pair.step(grads)
    pair.check("eager, device plan")
    assert pair.rect_flags == [0] * 5 + [1] * 7
    assert pair.opt.info()["launches"] == 2 * 12 + 1      # step + plan kernel, one arming launch


@pytest.mark.parametrize("extra", [dict(), dict(clip_threshold=0.05, centralize=True),
                                   dict(adaptive_beta=True, lookahead_mode="traj_mean"),
                                   dict(clip_threshold=0.05, copies=True),
                                   dict(layer_adaptation=True, clip_threshold=0.05, centralize=True)])
def test_captured_once_and_replayed(extra):
    extra = dict(extra)
    with_copies = extra.pop("copies", False)
    shapes = [(64, 33), (1000,), (16, 3, 5, 5), (7,), (300, 40)]
    numels = [int(np.prod(s)) for s in shapes]
    params = _fresh(numels, shapes=shapes)
    hyper = dict(BASE, **extra)
    rows = [s[0] if len(s) > 1 else 0 for s in shapes]
    oracle = O.Oracle(oracle_config(hyper), [to_f64(p) for p in params], rows=rows)
    opt = B.NovakOptimizer(params, **hyper, graph_capturable=True)
    copies = None
    if with_copies:                        # bf16 model copies written by the replayed steps
        copies = make_tensors(numels, DEV, dtype=torch.bfloat16)[1]
        opt.set_param_copies(copies)
    _, gviews, _ = make_tensors(numels, DEV)
    static = [v.view(s) for v, s in zip(gviews, shapes)]       # the captured gradient buffers
    gen = _gen(17)

    def new_grads():
        for g in static:
            g.normal_(0.0, 1e-2, generator=gen)
        oracle.step([to_f64(g) for g in static])

    new_grads()
    opt.step(static)                       # outside the capture: allocations and uploads
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    new_grads()
    with torch.cuda.graph(graph):
        opt.step(static)                   # captured (and not run)
    graph.replay()                         # step 2
    for _ in range(11):                    # steps 3 .. 13: sync at 5 and 10, switch at 6
        new_grads()
        graph.replay()
    torch.cuda.synchronize()
    info = opt.info()
    assert info["t"] == 13 == oracle.t
    assert info["n_syncs"] == len(oracle.sync_steps) and info["last_sync_step"] == oracle.sync_steps[-1]
    assert info["rect_branch"] == 1 and info["is_sync"] == 0
    for i, p in enumerate(params):
        assert_close(p, oracle.theta[i], f"replayed theta[{i}]")
        st = opt.state(i)
        assert_close(st["m"], oracle.m[i], f"replayed m[{i}]")
        assert_close(st["v"], oracle.v[i], f"replayed v[{i}]")
        assert_close(st["slow"], oracle.slow[i], f"replayed slow[{i}]")
    if copies is not None:
        for p, c in zip(params, copies):
            assert torch.equal(c.view(p.shape), p.to(torch.bfloat16))
    # a checkpoint taken now carries the device's counters
    assert opt.handle.export_meta().t == 13
    # the learning rate reaches the device at the next CALL; replays keep what they find
    opt.handle.set_option(B.NOVAK_OPT_LR, 5e-4)
    oracle.cfg.lr = 5e-4
    oracle.h.lr = 5e-4
    new_grads()
    opt.step(static)                       # step 14, eager: uploads the new rate
    new_grads()
    graph.replay()                         # step 15 with the new rate
    torch.cuda.synchronize()
    assert opt.info()["t"] == 15
    for i, p in enumerate(params):
        assert_close(p, oracle.theta[i], f"after the rate change theta[{i}]")


def test_bf16_moments_replayed_against_the_plain_step():
    """Moments stored in bfloat16 under replay: the same stored codes and parameters as the
    plain step of a twin (whose parity against the oracle test_gpu_bf16_moments.py holds).
    The two compute their scalars with different math libraries (host, device), so a code
    may differ where a moment sits on a rounding boundary: a handful per million at most."""
    numels = [70001, 33, 8192, 5]
    pa, pb = _fresh(numels, seed=2), _fresh(numels, seed=2)
    hyper = dict(BASE, moment_dtype="bf16", clip_threshold=0.05)
    plain = B.NovakOptimizer(pa, **hyper)
    dyn = B.NovakOptimizer(pb, **hyper, graph_capturable=True)
    _, static, _ = make_tensors(numels, DEV)
    gen = _gen(31)

    def new_grads():
        for g in static:
            g.normal_(0.0, 1e-2, generator=gen)

    new_grads()
    plain.step(static); dyn.step(static)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dyn.step(static)
    for _ in range(11):
        new_grads()
        plain.step(static)
        graph.replay()
    torch.cuda.synchronize()
    assert dyn.info()["t"] == 12 == plain.info()["t"]
    differing = total = 0
    for i in range(len(numels)):
        for k in ("m", "v"):
            a, b = plain.state(i)[k], dyn.state(i)[k]
            assert a.dtype == torch.bfloat16 == b.dtype
            differing += int((a.view(torch.int16) != b.view(torch.int16)).sum())
            total += a.numel()
        torch.testing.assert_close(pb[i], pa[i], rtol=1e-5, atol=2e-6)
    assert differing <= max(2, total // 100_000), (differing, total)


def test_the_plain_step_refuses_to_be_captured():
    """Its scalars are launch parameters: a replay would repeat one step for ever."""
    params = _fresh([4096, 100])
    g = [torch.zeros_like(p) for p in params]
    opt = B.NovakOptimizer(params, **BASE)
    opt.step(g)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with pytest.raises(B.NovakError) as e:
        with torch.cuda.graph(graph):
            opt.step(g)
    assert e.value.status == B.NOVAK_ESTATE and "captured" in str(e.value)
    torch.cuda.synchronize()
    opt.step(g)                                  # the handle and the context are fine
    assert opt.info()["t"] == 2


def test_what_the_mode_does_not_cover_is_refused():
    params = _fresh([4096, 100])
    g = [torch.zeros_like(p) for p in params]
    for kw in (dict(nesterov="true", true_nesterov_steps=3),):
        opt = B.NovakOptimizer(params, **dict(BASE, **kw), graph_capturable=True)
        with pytest.raises(B.NovakError) as e:
            opt.step(g)
        assert e.value.status == B.NOVAK_ESTATE
    opt = B.NovakOptimizer(params, **BASE, graph_capturable=True)
    gl = opt.prepare(g)
    with pytest.raises(B.NovakError):
        opt.handle.step_noalloc(opt._params_arr, gl.arr, opt._numel_arr, opt.n, gl.dtype, 0)
    with pytest.raises(B.NovakError):
        opt.step_begin(g)
    opt.step(g)
    with pytest.raises(B.NovakError):                     # fixed once a step was taken
        opt.handle.set_option(B.NOVAK_OPT_GRAPH_CAPTURABLE, 0)
    assert opt.info()["t"] == 1


def test_fullsize_resnet50_replayed():
    """The ResNet-50-shaped set at full size: one eager step, one captured step, 18 replays
    (gradients refilled in the captured buffer between replays); the oracle follows the
    usual sample of elements."""
    from harness import SampledPair
    from paper_2601_07876_b200 import workloads as W
    wl = W.get_workload(1)
    pair = SampledPair(wl, DEV, opt_kwargs=dict(graph_capturable=True))
    pair.step(threads=8)                                  # eager: t = 1
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    pair.src.fill(pair.flat_g, pair.scratch)
    with torch.cuda.graph(graph):
        pair.opt.step(pair.glist)
    for t in range(2, 21):
        if t > 2:
            pair.src.fill(pair.flat_g, pair.scratch)
        graph.replay()
        pair.oracle.step([to_f64(pair.flat_g[pair.idx])], threads=8)
    torch.cuda.synchronize()
    info = pair.opt.info()
    assert info["t"] == 20 == pair.oracle.t and info["n_syncs"] == 4 and info["last_sync_step"] == 20
    assert_close(pair.flat_p[pair.idx], pair.oracle.theta[0], "resnet50 replayed theta")
    assert_close(pair._gather_state("m"), pair.oracle.m[0], "resnet50 replayed m")
    assert_close(pair._gather_state("v"), pair.oracle.v[0], "resnet50 replayed v")
    assert_close(pair._gather_state("slow"), pair.oracle.slow[0], "resnet50 replayed slow")
    del pair
    torch.cuda.empty_cache()
