"""True Nesterov momentum (Eq. 10-12) through the C ABI against the oracle: the
look-ahead kernel, the bit-exact restore, the closed loop with a synthetic
closure, the fallback after N_taylor steps and the state machine's refusals.

The closure is a fixed seeded map of the look-ahead point, g~ = a * theta~ + b
(a, b per element), evaluated ONCE per step in float64 from the oracle's theta~ and
handed to both sides rounded to fp32, so that the two see the same gradient.
"""
import numpy as np
import pytest
import torch

from harness import Pair, assert_close, make_tensors, to_f64
from paper_2601_07876_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

RAGGED = [1, 2, 3, 5, 31, 33, 1023, 1025, 8191, 8193, 70001, 4096]
BASE = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2, nesterov="true",
            nesterov_beta=0.8, lookahead_k=5, lookahead_alpha=0.5)


def _fresh(numels, offsets=None, seed=1, std=0.05):
    flat, views, _ = make_tensors(numels, DEV, offsets)
    g = torch.Generator(device=DEV).manual_seed(seed)
    for v in views:
        v.normal_(0.0, std, generator=g)
    return flat, views


def _closure(numels, seed=5):
    rng = np.random.default_rng(seed)
    a = [rng.uniform(0.5, 2.0, n) for n in numels]
    b = [rng.normal(0.0, 1e-2, n) for n in numels]
    return lambda points: [ai * x + bi for ai, bi, x in zip(a, b, points)]


def _device_grads(gs64, offsets=None):
    _, views, _ = make_tensors([g.size for g in gs64], DEV, offsets)
    for v, g in zip(views, gs64):
        v.copy_(torch.from_numpy(g.astype(np.float32)).to(DEV))
    return views


@pytest.mark.parametrize("route", ["restore", "fused"])
@pytest.mark.parametrize("offsets", [None, "phased"])
def test_closed_loop_with_fallback(offsets, route):
    """N_taylor = 4 of 9 steps: look ahead, compare theta~ with Eq. 10, restore bit for
    bit (route "restore") or let the step read theta_{t-1} from the save buffer (route
    "fused": no restore pass), step on the closure's gradient; from step 5 on plain steps
    (Eq. 13)."""
    offs = [(i % 4) if i % 3 == 2 else 0 for i in range(len(RAGGED))] if offsets else None
    _, params = _fresh(RAGGED, offs)
    pair = Pair(params, dict(BASE, true_nesterov_steps=4))
    grad_of = _closure(RAGGED)
    wanted = []
    for t in range(1, 10):
        want = pair.opt.wants_extrapolation()
        assert want == pair.oracle.wants_extrapolation()
        wanted.append(want)
        if want:
            before = [p.clone() for p in params]
            pair.opt.extrapolate()
            point = pair.oracle.extrapolated()
            for i, p in enumerate(params):
                assert_close(p, point[i], f"t={t} theta~[{i}]")
            gs = grad_of(point)
            if route == "restore":
                pair.opt.restore()
                for p, b in zip(params, before):
                    assert torch.equal(p, b), "restore must be bit-exact"
        else:
            gs = grad_of(pair.oracle.theta)
        pair.step(_device_grads(gs, offs))
        assert pair.opt.info()["nesterov_variant"] == (
            B.NOVAK_NESTEROV_TRUE if want else B.NOVAK_NESTEROV_APPROX)
        if t in (1, 4, 5):
            pair.check(f"t={t}")
    pair.check("end")
    assert wanted == [True] * 4 + [False] * 5
    assert not pair.opt.info()["warnings"] & B.NOVAK_WARN_TRUE_DOWNGRADED
    assert pair.opt.info()["launches"] == 9 + (8 if route == "restore" else 4)


@pytest.mark.parametrize("extra", [dict(), dict(lookahead_mode="traj_mean", lookahead_k=2),
                                   dict(layer_adaptation=True),
                                   dict(auto_lr=True, clip_threshold=0.05),
                                   dict(moment_dtype="bf16"), dict(lookahead_k=0)])
def test_step_behind_the_look_ahead_equals_restore_then_step(extra):
    """The two routes, side by side on twin handles: extrapolate, restore, step against
    extrapolate, step.  Parameters and every state array bit for bit the same after each
    of 6 steps (4 of them true steps), also where another kernel reads theta_{t-1} first
    (the norms of layer adaptation and of the automatic learning-rate scaling)."""
    offs = [(i % 4) if i % 3 == 2 else 0 for i in range(len(RAGGED))]
    _, pa = _fresh(RAGGED, offs)
    _, pb = _fresh(RAGGED, offs)
    hyper = dict(BASE, true_nesterov_steps=4, **extra)
    a = B.NovakOptimizer(pa, **hyper)
    b = B.NovakOptimizer(pb, **hyper)
    gen = torch.Generator(device=DEV).manual_seed(12)
    for t in range(1, 7):
        _, grads, _ = make_tensors(RAGGED, DEV, offs)
        for g in grads:
            g.normal_(0.0, 1e-2, generator=gen)
        if a.wants_extrapolation():
            a.extrapolate()
            a.restore()
            b.extrapolate()
            if t > 1:
                assert not torch.equal(pb[-2], pa[-2])      # b's parameters still sit at theta~
        a.step(grads)
        b.step(grads)
        torch.cuda.synchronize()
        for x, y in zip(pa, pb):
            assert torch.equal(x, y), f"t={t}"
        for i in range(len(RAGGED)):
            sa, sb = a.state(i), b.state(i)
            for k in ("m", "v", "slow", "acc"):
                assert (sa[k] is None and sb[k] is None) or torch.equal(sa[k], sb[k]), (t, i, k)
    assert a.info()["launches"] - b.info()["launches"] == 4


def test_first_look_ahead_is_the_identity_and_m_is_read_not_written():
    _, params = _fresh([5000, 77])
    opt = B.NovakOptimizer(params, **dict(BASE, true_nesterov_steps=10))
    before = [p.clone() for p in params]
    opt.extrapolate()
    torch.cuda.synchronize()
    for p, b in zip(params, before):
        assert torch.equal(p, b)            # m_0 = 0
    opt.restore()
    g = [torch.full_like(p, 0.5) for p in params]
    opt.step(g)
    m = [opt.state(i)["m"].clone() for i in range(2)]
    th = [p.clone() for p in params]
    opt.extrapolate()
    for i, p in enumerate(params):
        assert torch.equal(opt.state(i)["m"], m[i])
        # one fused multiply-add per element: theta + 0.8 m, rounded once
        want = (th[i].double() + np.float32(0.8).astype(np.float64) * m[i].double()).float()
        assert torch.equal(p, want)
    opt.restore()
    for p, b in zip(params, th):
        assert torch.equal(p, b)


@pytest.mark.parametrize("chunk", [1024, 4096, 8192])
def test_look_ahead_with_other_entry_sizes(chunk):
    """Entries of 1024 ... 8192 elements: the look-ahead kernels loop over more than one
    pair of vectors per thread; same bits as with the default entries."""
    numels = [70001, 33, 9000, 5]
    offs = [0, 2, 0, 1]
    _, pa = _fresh(numels, offs)
    _, pb = _fresh(numels, offs)
    hyper = dict(BASE, true_nesterov_steps=3)
    a = B.NovakOptimizer(pa, **hyper)
    b = B.NovakOptimizer(pb, **hyper, chunk_elems=chunk)
    for t in range(3):
        g = _device_grads([np.full(n, 0.01 * (t + 1)) for n in numels], offs)
        for o in (a, b):
            o.extrapolate()
        for x, y in zip(pa, pb):
            assert torch.equal(x, y)
        for o in (a, b):
            o.restore()
            o.step(g)
    for x, y in zip(pa, pb):
        assert torch.equal(x, y)


def test_state_machine_refusals():
    _, params = _fresh([4096, 100])
    opt = B.NovakOptimizer(params, **dict(BASE, true_nesterov_steps=2))
    g = [torch.zeros_like(p) for p in params]
    with pytest.raises(B.NovakError):
        opt.handle.nesterov_restore(opt._params_arr, params[0].data_ptr(), 1 << 30, opt._numel_arr,
                                    opt.n, 0)                      # nothing to restore
    opt.extrapolate()
    with pytest.raises(B.NovakError):
        opt.extrapolate()                                          # twice
    gl = opt.prepare(g)
    with pytest.raises(B.NovakError):
        opt.handle.step_noalloc(opt._params_arr, gl.arr, opt._numel_arr, opt.n, gl.dtype, 0)
    with pytest.raises(B.NovakError):
        opt.handle.set_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS, 7)
    other = torch.empty(opt.handle.nesterov_save_bytes(), dtype=torch.uint8, device=DEV)
    with pytest.raises(B.NovakError):
        opt.handle.nesterov_restore(opt._params_arr, other.data_ptr(), other.numel(),
                                    opt._numel_arr, opt.n, 0)      # another save buffer
    opt.restore()
    opt.step(g)
    assert opt.info()["t"] == 1
    # novak_step may follow the look-ahead directly; there is nothing to restore afterwards
    opt.extrapolate()
    opt.step(g)
    assert opt.info()["t"] == 2
    with pytest.raises(B.NovakError):
        opt.restore()
    # short and misaligned save buffers
    need = opt.handle.nesterov_save_bytes()
    buf = torch.empty(need + 64, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.NovakError):
        opt.handle.nesterov_extrapolate(opt._params_arr, buf.data_ptr(), need - 4, opt._numel_arr,
                                        opt.n, 0)
    with pytest.raises(B.NovakError):
        opt.handle.nesterov_extrapolate(opt._params_arr, buf.data_ptr() + 4, need, opt._numel_arr,
                                        opt.n, 0)
    # a handle of another variant has no look-ahead
    plain = B.NovakOptimizer(params, **dict(BASE, nesterov="approximation"))
    with pytest.raises(B.NovakError):
        plain.extrapolate()


def test_checkpoint_carries_the_true_variant():
    _, params = _fresh([3000])
    a = B.NovakOptimizer(params, **dict(BASE, true_nesterov_steps=6))
    a.step([torch.ones_like(params[0])])
    sd = a.state_dict()
    b = B.NovakOptimizer(params, **dict(BASE))          # N_taylor = 0 until the import
    b.load_state_dict(sd)
    assert b.handle.get_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS) == 6
    assert b.wants_extrapolation() and b.info()["t"] == 1
    assert not b.info()["warnings"] & B.NOVAK_WARN_TRUE_DOWNGRADED


def test_fullsize_resnet50_launch_configuration():
    """The ResNet-50-shaped set at full size: five true steps, then the fallback; the
    oracle follows the usual sample of elements (gradients are the workload's seeded
    random ones: the kernels do not care where a gradient was evaluated)."""
    from harness import SampledPair
    from paper_2601_07876_b200 import workloads as W
    wl = W.get_workload(1)
    pair = SampledPair(wl, DEV, dict(nesterov="true", nesterov_beta=0.8, true_nesterov_steps=5))
    for t in range(1, 9):
        want = pair.opt.wants_extrapolation()
        assert want == pair.oracle.wants_extrapolation() == (t <= 5)
        if want:
            before = pair.flat_p.clone()
            pair.opt.extrapolate()
            assert_close(pair.flat_p[pair.idx], pair.oracle.extrapolated()[0], f"t={t} theta~")
            if t > 1:
                assert not torch.equal(pair.flat_p, before)
            if t % 2 == 0:
                pair.opt.restore()
                assert torch.equal(pair.flat_p, before)
            del before                   # odd steps: the step reads the save buffer itself
        pair.step(threads=8)
    pair.check()
    assert pair.opt.info()["launches"] == 8 + 2 * 2 + 3
    del pair
    torch.cuda.empty_cache()
