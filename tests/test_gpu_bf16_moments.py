"""Moments stored in bfloat16 (NOVAK_MOMENT_BF16) through the C ABI against the oracle.

The stored moments are 16-bit codes: they are compared BIT FOR BIT.  The decision
which code a value rounds to is taken in fp32 by the kernel and in fp64 by the
oracle; the two can differ only where the unrounded value comes within the
kernel's own rounding error of a rounding boundary.  The oracle reports, per
element, the smallest distance to a boundary over the run relative to the size of
the summed terms; elements that came closer than MARGIN (about ten times the
fp32 error of the three-term update) are set aside, counted, and checked
only loosely; all others must match exactly (m, v) and within the usual
tolerance (theta, slow, running sum).
"""
import numpy as np
import pytest
import torch

from harness import Pair, assert_close, make_tensors, to_f64
from paper_2601_07876_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MARGIN = 3e-6

RAGGED = [1, 2, 3, 5, 31, 33, 1023, 1025, 8191, 8193, 70001, 4096]
BASE = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
            nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5, moment_dtype="bf16")


def _gen(seed):
    return torch.Generator(device=DEV).manual_seed(seed)


def _fresh(numels, offsets=None, seed=1, std=0.05, shapes=None):
    _, views, _ = make_tensors(numels, DEV, offsets)
    g = _gen(seed)
    for v in views:
        v.normal_(0.0, std, generator=g)
    if shapes:
        views = [v.view(s) for v, s in zip(views, shapes)]
    return views


def _grads(numels, gen, dtype=torch.float32, offsets=None, std=1e-2, shapes=None):
    _, views, _ = make_tensors(numels, DEV, offsets, dtype=dtype)
    for v in views:
        v.copy_(torch.empty(v.shape, dtype=torch.float32, device=DEV).normal_(0.0, std, generator=gen))
    if shapes:
        views = [v.view(s) for v, s in zip(views, shapes)]
    return views


def _check(pair, whole_tensors=False, max_fraction=0.08):
    """Bit-exact moments and in-tolerance parameters on every element that stayed clear
    of a rounding boundary; returns the fraction set aside."""
    torch.cuda.synchronize()
    o = pair.oracle
    assert pair.opt.info()["t"] == o.t
    assert pair.sync_steps == o.sync_steps and pair.rect_flags == o.rect_flags
    aside = total = 0
    for i, p in enumerate(pair.params):
        st = pair.opt.state(i)
        assert st["m"].dtype == torch.bfloat16 and st["v"].dtype == torch.bfloat16
        near = o.rounding_margin[i] < MARGIN
        if whole_tensors and near.any():
            near[:] = True        # a norm over the tensor has seen the element
        ok = ~near
        aside += int(near.sum()); total += near.size
        gm, gv = to_f64(st["m"]).reshape(-1), to_f64(st["v"]).reshape(-1)
        assert np.array_equal(gm[ok], o.m[i][ok]), f"m[{i}]: stored codes differ"
        assert np.array_equal(gv[ok], o.v[i][ok]), f"v[{i}]: stored codes differ"
        assert_close(to_f64(p).reshape(-1)[ok], o.theta[i][ok], f"theta[{i}]")
        if st["slow"] is not None:
            assert_close(to_f64(st["slow"]).reshape(-1)[ok], o.slow[i][ok], f"slow[{i}]")
        if st["acc"] is not None:
            assert_close(to_f64(st["acc"]).reshape(-1)[ok], o.acc[i][ok], f"acc[{i}]")
        # the rest: a code or two apart at most, parameters still close
        # (measured against the tensor's own scale: m passes through zero)
        for got, ref in ((gm, o.m[i]), (gv, o.v[i])):
            rms = float(np.sqrt(np.mean(ref * ref)))
            assert np.all(np.abs(got[near] - ref[near]) <= 2.0 ** -5 * (np.abs(ref[near]) + rms))
        np.testing.assert_allclose(to_f64(p).reshape(-1)[near], o.theta[i][near], rtol=1e-3, atol=1e-4)
    frac = aside / max(total, 1)
    assert frac <= max_fraction, f"{frac:.3f} of the elements set aside"
    return frac


@pytest.mark.parametrize("nesterov", ["none", "approximation", "classical"])
@pytest.mark.parametrize("la", [(0, "last"), (5, "last"), (5, "traj_mean")])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_variants_ragged_multi_tensor(nesterov, la, gdtype):
    k, mode = la
    offsets = [(i % 4) if i % 3 == 2 else 0 for i in range(len(RAGGED))]
    params = _fresh(RAGGED, offsets)
    pair = Pair(params, dict(BASE, nesterov=nesterov, lookahead_k=k, lookahead_mode=mode))
    pair.oracle.track_rounding_margin = True
    gen = _gen(100)
    # fp32 gradients: about 0.2 % of the elements per step come within MARGIN of a
    # boundary.  bf16 gradients: beta1 m + (1 - beta1) g with m and g both 8-bit values
    # and beta1 = 0.9 is a multiple of a tenth of a power of two, which lands EXACTLY on
    # a midpoint (up to the representation error of 0.9 and 0.1, 1e-17 in fp64, 1e-8 in
    # fp32) for a few percent of the elements per step: genuine ties, set aside as well.
    cap = 0.08 if gdtype == torch.float32 else 0.5
    for t in range(11):
        pair.step(_grads(RAGGED, gen, gdtype, offsets))
        if t in (0, 5):
            _check(pair, max_fraction=cap)
    frac = _check(pair, max_fraction=cap)
    assert frac > 0.0          # the margin is not vacuous on 100 k elements x 11 steps
    assert not pair.opt.info()["warnings"] & B.NOVAK_WARN_SCALAR_PATH
    assert pair.opt.info()["moment_dtype"] == B.NOVAK_MOMENT_BF16


def test_gradients_at_another_phase_are_fetched_element_by_element():
    """Gradients at another 16-byte phase than the parameters: their loads narrow, the
    64-bit moment accesses stay."""
    numels = [1000, 4099, 7]
    params = _fresh(numels)
    pair = Pair(params, dict(BASE))
    pair.oracle.track_rounding_margin = True
    gen = _gen(3)
    for _ in range(6):
        pair.step(_grads(numels, gen, offsets=[1, 2, 3]))
    _check(pair)
    assert pair.opt.info()["warnings"] & B.NOVAK_WARN_NARROW_GRADIENT
    assert not pair.opt.info()["warnings"] & B.NOVAK_WARN_SCALAR_PATH


def test_state_is_half_the_size_and_rounded_once():
    numels = [4096, 100]
    params = _fresh(numels)
    a = B.NovakOptimizer(params, **dict(BASE, lookahead_k=0))
    b = B.NovakOptimizer([p.clone() for p in params], **dict(BASE, lookahead_k=0, moment_dtype="f32"))
    assert 2 * a.handle.state_bytes(numels) == b.handle.state_bytes(numels)
    g = _grads(numels, _gen(9))
    a.step(g); b.step(g)
    for i in range(2):
        # one step from zero moments: the bf16 state is the rounding of the fp32 state,
        # and the parameters moved exactly as with fp32 state (the step uses unrounded values)
        assert torch.equal(a.state(i)["m"], b.state(i)["m"].to(torch.bfloat16))
        assert torch.equal(a.state(i)["v"], b.state(i)["v"].to(torch.bfloat16))
        assert torch.equal(a.params[i], b.params[i])
    with pytest.raises(B.NovakError):
        a.handle.set_option(B.NOVAK_OPT_MOMENT_DTYPE, B.NOVAK_MOMENT_F32)    # attached


def test_with_clipping_centralization_and_layer_adaptation():
    shapes = [(64, 33), (1000,), (16, 3, 5, 5), (7,), (300, 40)]
    numels = [int(np.prod(s)) for s in shapes]
    params = _fresh(numels, shapes=shapes)
    hyper = dict(BASE, clip_threshold=0.05, centralize=True, layer_adaptation=True)
    pair = Pair(params, hyper)
    pair.oracle.track_rounding_margin = True
    gen = _gen(21)
    for _ in range(8):
        pair.step(_grads(numels, gen, shapes=shapes))
        pair.record_grad_stats()
    np.testing.assert_allclose(pair.grad_norms, pair.oracle.grad_norms, rtol=1e-7)
    # a norm over a tensor has seen every element: tensors with a near-boundary element
    # are set aside whole (the small ones survive)
    _check(pair, whole_tensors=True, max_fraction=1.0)
    tr = np.array(pair.opt.trust_ratios())
    np.testing.assert_allclose(tr, pair.oracle.trust[-1], rtol=2e-3)


def test_centralization_inside_the_step_kernel_with_bf16_moments():
    """The row-owning step kernel (centralization alone) in its bf16-moment instantiation."""
    shapes = [(64, 33), (1000,), (16, 3, 5, 5), (7,), (300, 40), (3, 4608)]
    numels = [int(np.prod(s)) for s in shapes]
    params = _fresh(numels, shapes=shapes)
    pair = Pair(params, dict(BASE, centralize=True))
    pair.oracle.track_rounding_margin = True
    gen = _gen(22)
    for _ in range(8):
        pair.step(_grads(numels, gen, shapes=shapes))
    _check(pair, max_fraction=0.1)
    assert pair.opt.info()["launches"] == 8


def test_true_nesterov_reads_bf16_first_moments():
    numels = [5000, 77, 2048]
    params = _fresh(numels)
    pair = Pair(params, dict(BASE, nesterov="true", nesterov_beta=0.8, true_nesterov_steps=3))
    pair.oracle.track_rounding_margin = True
    gen = _gen(33)
    for t in range(5):
        if pair.opt.wants_extrapolation():
            before = [p.clone() for p in params]
            pair.opt.extrapolate()
            point = pair.oracle.extrapolated()
            near = [m < MARGIN for m in pair.oracle.rounding_margin]
            for i, p in enumerate(params):
                assert_close(to_f64(p).reshape(-1)[~near[i]], point[i][~near[i]], f"theta~[{i}]")
            pair.opt.restore()
            for p, b in zip(params, before):
                assert torch.equal(p, b)
        pair.step(_grads(numels, gen))
    _check(pair)


def test_checkpoint_round_trip_and_dtype_mismatch():
    numels = [3000, 129]
    params = _fresh(numels)
    a = B.NovakOptimizer(params, **BASE)
    gen = _gen(5)
    for _ in range(3):
        a.step(_grads(numels, gen))
    sd = a.state_dict()
    snap = [p.clone() for p in params]
    g = _grads(numels, gen)
    a.step(g)
    want = [p.clone() for p in params]
    for p, s in zip(params, snap):
        p.copy_(s)
    b = B.NovakOptimizer(params, **BASE)
    b.load_state_dict(sd)
    b.step(g)
    for p, w in zip(params, want):
        assert torch.equal(p, w)
    c = B.NovakOptimizer(params, **dict(BASE, moment_dtype="f32"))
    with pytest.raises(B.NovakError):
        c.load_state_dict(sd)


@pytest.mark.parametrize("index", [1, 3])
def test_fullsize_launch_configuration(index):
    """The ResNet-50-shaped (fp32 gradients) and ViT-B/16-shaped (bf16 gradients) sets at
    full size, 12 steps; the oracle follows the usual sample of elements."""
    from harness import SampledPair
    from paper_2601_07876_b200 import workloads as W
    wl = W.get_workload(index)
    pair = SampledPair(wl, DEV, dict(moment_dtype="bf16"))
    o = pair.oracle
    o.track_rounding_margin = True
    for _ in range(12):
        pair.step(threads=8)
    torch.cuda.synchronize()
    assert pair.opt.info()["t"] == o.t and pair.sync_steps == o.sync_steps
    near = o.rounding_margin[0] < MARGIN
    ok = ~near
    frac = float(near.mean())
    assert frac <= (0.12 if wl.grad_dtype == torch.float32 else 0.5), frac
    gm, gv = to_f64(pair._gather_state("m")), to_f64(pair._gather_state("v"))
    assert np.array_equal(gm[ok], o.m[0][ok]) and np.array_equal(gv[ok], o.v[0][ok])
    assert_close(to_f64(pair.flat_p[pair.idx])[ok], o.theta[0][ok], f"{wl.name} theta")
    assert_close(to_f64(pair._gather_state("slow"))[ok], o.slow[0][ok], f"{wl.name} slow")
    print(f"\nBF16 MOMENTS {wl.name}: {ok.sum()} of {ok.size} sampled elements compared bit for bit, "
          f"{frac:.4f} set aside")
    assert pair.opt.info()["launches"] == 12
    del pair
    torch.cuda.empty_cache()


def test_other_entry_points_and_chunk_sizes_give_the_same_bits():
    """novak_step_noalloc, novak_step_host and entries of 1024 / 4096 elements run the same
    kernels on bf16 moments: bit-identical parameters and state to novak_step."""
    numels = [70001, 33, 2048, 1, 9000]
    offs = [0, 1, 0, 3, 2]
    hyper = dict(BASE, lookahead_k=2)

    def fresh(**kw):
        ps = _fresh(numels, offs, seed=4)
        return ps, B.NovakOptimizer(ps, **hyper, **kw)

    (pa, a), (pb, b), (pc, c), (pd, d), (pe, e) = (fresh(), fresh(), fresh(),
                                                   fresh(chunk_elems=1024), fresh(chunk_elems=4096))
    gen = _gen(8)
    total = sum(numels)
    h_g = torch.empty(total, dtype=torch.float32).pin_memory()
    h_p = torch.empty(total, dtype=torch.float32).pin_memory()
    d_g = torch.empty(total, dtype=torch.float32, device=DEV)
    starts = np.concatenate([[0], np.cumsum(numels)])[:-1]
    hg = B.ptr_array([h_g.data_ptr() + 4 * int(o) for o in starts])
    hp = B.ptr_array([h_p.data_ptr() + 4 * int(o) for o in starts])
    dg = B.ptr_array([d_g.data_ptr() + 4 * int(o) for o in starts])
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(5):
        grads = _grads(numels, gen, offsets=offs)
        a.step(grads)
        gl = b.prepare(grads)
        b.handle.step_noalloc(b._params_arr, gl.arr, b._numel_arr, b.n, gl.dtype, stream)
        h_g.copy_(torch.cat([g.reshape(-1) for g in grads]).cpu())
        c.handle.step_host(hp, hg, c._params_arr, dg, c._numel_arr, c.n, B.NOVAK_GRAD_F32, stream)
        d.step(grads)
        e.step(grads)
    torch.cuda.synchronize()
    for other, ps in ((b, pb), (c, pc), (d, pd), (e, pe)):
        for i in range(len(numels)):
            assert torch.equal(ps[i], pa[i])
            for k in ("m", "v", "slow"):
                assert torch.equal(other.state(i)[k], a.state(i)[k])
    assert torch.equal(h_p.to(DEV), torch.cat([p.reshape(-1) for p in pc]))
