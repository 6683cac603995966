"""Phase 2 on the GPU (global-norm clipping, gradient centralization) against
the CPU oracle, element by element, through the C ABI.  Same tolerance as the
other parity tests; the gradient norm itself to 1e-7."""
import math

import numpy as np
import pytest
import torch

import harness
from harness import Pair, make_tensors, to_f64
from paper_2601_07876_b200 import binding as B
from paper_2601_07876_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

BASE = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
            nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5)

# rows shorter, equal to and longer than a chunk-table entry (2048 elements), odd row
# lengths (rows cross 128-bit vectors and entry boundaries), rows of 1 and 2 elements,
# a single row, one-dimensional tensors in between, and some misaligned starts
SHAPES = [(8, 3, 3, 3), (33,), (10, 257), (3, 5000), (4097, 2), (1, 7), (5, 1), (2048,),
          (6, 2048), (7, 1000, 3), (2, 3, 4100)]
OFFSETS = [0, 1, 0, 3, 0, 2, 0, 0, 0, 0, 1]


def _gen(seed):
    return torch.Generator(device=DEV).manual_seed(seed)


def _shaped(shapes, offsets, dtype=torch.float32):
    numels = [math.prod(s) for s in shapes]
    flat, views, _ = make_tensors(numels, DEV, offsets, dtype=dtype)
    return flat, [v.view(s) for v, s in zip(views, shapes)]


def _fill_grads(grads, gen, std, mean=0.0):
    for g in grads:
        g.copy_(torch.empty(g.shape, dtype=torch.float32, device=DEV)
                .normal_(mean, std, generator=gen))


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("phase2", [dict(clip_threshold=0.05), dict(clip_threshold=1e3),
                                    dict(centralize=True),
                                    dict(clip_threshold=0.05, centralize=True)])
@pytest.mark.parametrize("variant", [("approximation", "last"), ("classical", "traj_mean"),
                                     ("none", "last")])
def test_clip_and_centralize_every_element(gdtype, phase2, variant):
    nesterov, mode = variant
    _, params = _shaped(SHAPES, OFFSETS)
    gen = _gen(5)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    hyper = dict(BASE, nesterov=nesterov, lookahead_mode=mode, **phase2)
    pair = Pair(params, hyper)
    _, grads = _shaped(SHAPES, OFFSETS, dtype=gdtype)
    for t in range(7):
        # a non-zero mean makes the row means matter; the norm is ~0.3: clipped at 0.05
        _fill_grads(grads, gen, std=1e-3, mean=5e-4 * (1 + t % 3))
        pair.step(grads)
        if "clip_threshold" in phase2:
            pair.record_grad_stats()
    pair.check(f"phase2 {phase2}")
    info = pair.opt.info()
    assert info["grad_processing"] == (2 if phase2.get("centralize") else 1)
    if phase2 == dict(centralize=True):
        assert info["launches"] == 7          # the step kernel forms the row means itself
    else:
        assert info["launches"] == 3 * 7      # two statistics kernels + the step kernel
    if phase2.get("clip_threshold") == 0.05:
        assert all(f < 1.0 for f in pair.clip_factors)
    if phase2.get("clip_threshold") == 1e3:
        assert all(f == 1.0 for f in pair.clip_factors)


# rows of every kind the row-owning step kernel distinguishes: shorter than a warp's
# vector pass, odd lengths that start off a 16-byte boundary, a row for every warp and
# fewer rows than warps, one row per unit, rows at the largest owned length, and rows
# beyond it (2 x 40000, 1 x 70001) that keep the statistics pass
OWN_SHAPES = SHAPES + [(64, 147), (16, 64), (40, 27), (300, 40), (9, 576), (3, 4608), (2, 32768),
                       (2, 40000), (1, 70001), (5, 32769)]
OWN_OFFSETS = OFFSETS + [0, 0, 1, 0, 2, 0, 0, 3, 0, 1]


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("long_rows", [False, True])
@pytest.mark.parametrize("variant", [("approximation", "last", 5), ("classical", "traj_mean", 2),
                                     ("none", "last", 0)])
@pytest.mark.parametrize("in_step", [1, 0])
def test_centralization_alone_inside_the_step_kernel(in_step, variant, long_rows, gdtype):
    """Eq. 26 with nothing else that needs the whole gradient: the step kernel's CTAs own
    whole rows and form the means themselves (one launch per step); tensors with rows
    beyond the owned length still get theirs from the statistics pass.  Same oracle,
    same tolerance, in both forms."""
    nesterov, mode, k = variant
    n = len(OWN_SHAPES) if long_rows else len(OWN_SHAPES) - 3
    shapes, offsets = OWN_SHAPES[:n], OWN_OFFSETS[:n]
    _, params = _shaped(shapes, offsets)
    gen = _gen(15)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    copies = make_tensors([math.prod(s) for s in shapes], DEV, offsets, dtype=torch.bfloat16)[1]
    hyper = dict(BASE, nesterov=nesterov, lookahead_mode=mode, lookahead_k=k, centralize=True)
    pair = Pair(params, hyper, opt_kwargs=dict(centralize_in_step=in_step, param_copies=copies))
    _, grads = _shaped(shapes, offsets, dtype=gdtype)
    steps = 7
    for t in range(steps):
        _fill_grads(grads, gen, std=1e-3, mean=5e-4 * (1 + t % 3))
        pair.step(grads)
    pair.check(f"centralize, in step {in_step}")
    for p, c in zip(params, copies):
        assert torch.equal(c.view(p.shape), p.to(torch.bfloat16))
    info = pair.opt.info()
    assert info["grad_processing"] == 2
    own = bool(in_step) and not long_rows
    assert info["launches"] == (steps if own else 3 * steps)
    assert not info["warnings"] & (B.NOVAK_WARN_SCALAR_PATH | B.NOVAK_WARN_NARROW_GRADIENT)


def test_row_owning_step_is_bit_identical_from_run_to_run_and_takes_misphased_gradients():
    """Two runs of the row-owning kernel give the same bits (fixed summation order, no
    atomics); a gradient at another 16-byte phase than its parameter only narrows the
    gradient loads."""
    shapes, offsets = OWN_SHAPES[:-3], OWN_OFFSETS[:-3]
    runs = []
    for rep in range(2):
        _, params = _shaped(shapes, offsets)
        gen = _gen(17)
        for p in params:
            p.normal_(0.0, 0.05, generator=gen)
        opt = B.NovakOptimizer(params, **BASE, centralize=True)
        _, grads = _shaped(shapes, offsets)
        for t in range(4):
            _fill_grads(grads, gen, std=1e-3, mean=1e-3)
            opt.step(grads)
        torch.cuda.synchronize()
        assert opt.info()["launches"] == 4
        runs.append([p.clone() for p in params] + [opt.state(i)["v"].clone() for i in range(len(shapes))])
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    _, params = _shaped(shapes, offsets)
    gen = _gen(18)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    pair = Pair(params, dict(BASE, centralize=True, lookahead_k=2))
    goffs = [(o + 1 + i % 3) % 4 for i, o in enumerate(offsets)]
    _, grads = _shaped(shapes, goffs)
    for t in range(5):
        _fill_grads(grads, gen, std=1e-3, mean=1e-3)
        pair.step(grads)
    pair.check("row-owning kernel, gradients off the parameters' phase")
    assert pair.opt.info()["warnings"] & B.NOVAK_WARN_NARROW_GRADIENT
    assert pair.opt.info()["launches"] == 5


def test_row_owning_step_and_host_step_alternate_on_one_handle():
    """novak_step (row-owning kernel) and novak_step_host (statistics pass, the step in
    runs) take turns on one handle with centralization alone: both routes against the
    oracle, and no reallocation of the scratch in between (one layout serves both)."""
    shapes = [(20, 300), (31,), (9, 1000), (3,), (2, 40000)]
    numels = [math.prod(s) for s in shapes]
    _, params = _shaped(shapes, [0] * 5)
    gen = _gen(29)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    pair = Pair(params, dict(BASE, lookahead_k=2, centralize=True))
    opt = pair.opt
    opt.handle.set_option(B.NOVAK_OPT_HOST_SEGMENT_ELEMS, 8192)
    total = sum(numels)
    h_g = torch.empty(total, dtype=torch.float32).pin_memory()
    h_p = torch.empty(total, dtype=torch.float32).pin_memory()
    d_g = torch.empty(total, dtype=torch.float32, device=DEV)
    offs = np.concatenate([[0], np.cumsum(numels)])[:-1]
    hg = B.ptr_array([h_g.data_ptr() + 4 * int(o) for o in offs])
    hp = B.ptr_array([h_p.data_ptr() + 4 * int(o) for o in offs])
    dg = B.ptr_array([d_g.data_ptr() + 4 * int(o) for o in offs])
    stream = torch.cuda.current_stream().cuda_stream
    _, grads = _shaped(shapes, [0] * 5)
    for t in range(6):
        _fill_grads(grads, gen, std=1e-3, mean=1e-3)
        if t % 2 == 0:
            pair.step(grads)
        else:
            h_g.copy_(torch.cat([g.reshape(-1) for g in grads]).cpu())
            opt.handle.step_host(hp, hg, opt._params_arr, dg, opt._numel_arr, len(numels),
                                 B.NOVAK_GRAD_F32, stream)
            info = opt.info()
            if info["is_sync"]:
                pair.sync_steps.append(info["t"])
            pair.rect_flags.append(info["rect_branch"])
            pair.oracle.step([to_f64(g) for g in grads])
            torch.cuda.synchronize()
            assert torch.equal(h_p, torch.cat([p.reshape(-1) for p in params]).cpu())
    pair.check("row-owning step and host step in turns")


def test_phase2_is_bit_identical_from_run_to_run_and_across_launch_options():
    results = []
    for kw in (dict(), dict(), dict(dependent_launch=False), dict(chunk_elems=1024)):
        _, params = _shaped(SHAPES, OFFSETS)
        gen = _gen(9)
        for p in params:
            p.normal_(0.0, 0.05, generator=gen)
        opt = B.NovakOptimizer(params, **BASE, clip_threshold=0.05, centralize=True, **kw)
        _, grads = _shaped(SHAPES, OFFSETS)
        norms = []
        for _ in range(6):
            _fill_grads(grads, gen, std=1e-3, mean=1e-3)
            opt.step(grads)
            norms.append(opt.grad_stats()[0])
        torch.cuda.synchronize()
        results.append((norms, [p.clone() for p in params]))
    for norms, params in results[1:3]:      # same chunking: bit-identical, norm included
        assert norms == results[0][0]
        for a, b in zip(params, results[0][1]):
            assert torch.equal(a, b)
    # another chunk length adds the squares in another order: equal to rounding
    np.testing.assert_allclose(results[3][0], results[0][0], rtol=1e-12)


def test_options_can_change_between_steps_and_rows_can_be_reset():
    shapes = [(12, 300), (50,), (4, 2, 9)]
    _, params = _shaped(shapes, [0, 0, 0])
    gen = _gen(17)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    opt = B.NovakOptimizer(params, **BASE)
    oracle = harness.O.Oracle(harness.oracle_config(dict(BASE)), [to_f64(p) for p in params],
                              rows=harness.tensor_rows(params))
    _, grads = _shaped(shapes, [0, 0, 0])
    plan = [dict(), dict(clip=0.02), dict(clip=0.02, gc=True), dict(gc=True), dict(),
            dict(clip=0.5, gc=True)]
    for cfg in plan:
        _fill_grads(grads, gen, std=1e-3, mean=1e-3)
        opt.handle.set_option(B.NOVAK_OPT_CLIP_THRESHOLD, cfg.get("clip", 0.0))
        if cfg.get("gc"):
            opt.handle.set_tensor_rows(harness.tensor_rows(params))
        opt.handle.set_option(B.NOVAK_OPT_CENTRALIZE, 1 if cfg.get("gc") else 0)
        oracle.cfg.clip_threshold = cfg.get("clip", 0.0)
        oracle.cfg.centralize = bool(cfg.get("gc"))
        opt.step(grads)
        oracle.step([to_f64(g) for g in grads])
    torch.cuda.synchronize()
    for i, p in enumerate(params):
        harness.assert_close(p, oracle.theta[i], f"theta[{i}]")
        harness.assert_close(opt.state(i)["m"], oracle.m[i], f"m[{i}]")
        harness.assert_close(opt.state(i)["v"], oracle.v[i], f"v[{i}]")


def test_set_tensor_rows_rejects_bad_input_and_noalloc_refuses_phase2():
    shapes = [(6, 10), (8,)]
    _, params = _shaped(shapes, [0, 0])
    opt = B.NovakOptimizer(params, **BASE)
    h = opt.handle
    for bad in ([7, 0], [-1, 0], [6], [6, 0, 0]):
        with pytest.raises(B.NovakError) as e:
            h.set_tensor_rows(bad)
        assert e.value.status == B.NOVAK_EINVAL
    with pytest.raises(B.NovakError):
        h.set_option(B.NOVAK_OPT_CLIP_THRESHOLD, -1.0)
    with pytest.raises(B.NovakError) as e:
        h.get_grad_stats()
    assert e.value.status == B.NOVAK_ESTATE
    h.set_option(B.NOVAK_OPT_CLIP_THRESHOLD, 1.0)
    _, grads = _shaped(shapes, [0, 0])
    gl = opt.prepare(grads)
    with pytest.raises(B.NovakError) as e:
        h.step_noalloc(opt._params_arr, gl.arr, opt._numel_arr, opt.n, gl.dtype, opt._stream())
    assert e.value.status == B.NOVAK_ESTATE
    assert opt.info()["t"] == 0


def test_step_host_with_phase2_matches_step():
    shapes = [(20, 300), (31,), (9, 1000), (3,)]
    numels = [math.prod(s) for s in shapes]
    hyper = dict(BASE, lookahead_k=2, clip_threshold=0.02, centralize=True)
    gen = _gen(23)
    _, pa = _shaped(shapes, [0] * 4)
    for p in pa:
        p.normal_(0.0, 0.05, generator=gen)
    _, pb = _shaped(shapes, [0] * 4)
    for x, y in zip(pa, pb):
        y.copy_(x)
    a = B.NovakOptimizer(pa, **hyper)
    b = B.NovakOptimizer(pb, **hyper)
    b.handle.set_option(B.NOVAK_OPT_HOST_SEGMENT_ELEMS, 4096)
    total = sum(numels)
    h_g = torch.empty(total, dtype=torch.float32).pin_memory()
    h_p = torch.empty(total, dtype=torch.float32).pin_memory()
    d_g = torch.empty(total, dtype=torch.float32, device=DEV)
    offs = np.concatenate([[0], np.cumsum(numels)])[:-1]
    hg = B.ptr_array([h_g.data_ptr() + 4 * int(o) for o in offs])
    hp = B.ptr_array([h_p.data_ptr() + 4 * int(o) for o in offs])
    dg = B.ptr_array([d_g.data_ptr() + 4 * int(o) for o in offs])
    stream = torch.cuda.current_stream().cuda_stream
    _, grads = _shaped(shapes, [0] * 4)
    for _ in range(4):
        _fill_grads(grads, gen, std=1e-3, mean=1e-3)
        a.step(grads)
        h_g.copy_(torch.cat([g.reshape(-1) for g in grads]).cpu())
        b.handle.step_host(hp, hg, b._params_arr, dg, b._numel_arr, len(numels),
                           B.NOVAK_GRAD_F32, stream)
        torch.cuda.synchronize()
        assert torch.equal(h_p, torch.cat([p.reshape(-1) for p in pa]).cpu())
    # the two gradient buffers are aligned differently, so the sums run in another order
    np.testing.assert_allclose(a.grad_stats(), b.grad_stats(), rtol=1e-7)


@pytest.mark.parametrize("clip", [1.0, 0.0])
def test_fullsize_resnet50_with_clipping_and_centralization(clip):
    """The benchmark's ResNet-50-shaped set with its real tensor shapes (53 conv / fc
    weights with rows, 108 one-dimensional tensors), every element against the oracle:
    clipping + centralization (statistics pass), and centralization alone (formed inside
    the step kernel, one launch per step)."""
    wl = W.get_workload(1)
    flat_p = W.alloc_flat(wl, torch.float32, DEV)
    W.init_params(wl, flat_p)
    params = [v.view(s) for v, s in zip(W.views(flat_p, wl), wl.shapes)]
    flat_g = W.alloc_flat(wl, torch.float32, DEV)
    grads = [v.view(s) for v, s in zip(W.views(flat_g, wl), wl.shapes)]
    src = W.GradSource(wl, DEV)
    harness.MARGINS.clear()
    pair = Pair(params, dict(wl.hyper, clip_threshold=clip, centralize=True))
    for _ in range(12):
        src.fill(flat_g)
        pair.step(grads, threads=8)
        if clip:
            pair.record_grad_stats()
    pair.check("resnet50 phase2")
    if clip:
        assert all(f < 1.0 for f in pair.clip_factors)     # norm ~ 5: the clipping is active
    assert pair.opt.info()["launches"] == (36 if clip else 12)
    top = sorted(harness.MARGINS.items(), key=lambda kv: -kv[1])[:4]
    print("\nworst tensors:", [(k, round(v, 3), wl.shapes[int(k.split("[")[1][:-1])]) for k, v in top])
    worst = {}
    for k, v in harness.MARGINS.items():
        worst[k.split()[-1].split("[")[0]] = max(worst.get(k.split()[-1].split("[")[0], 0.0), v)
    print(f"\nPARITY resnet50 clip={clip}+centralize steps=12 every element worst |err|/tol: "
          + ", ".join(f"{k} {v:.3f}" for k, v in worst.items()))


def test_fullsize_resnet50_with_layer_adaptation():
    """The benchmark's ResNet-50-shaped set, layer adaptation in one launch (items of four
    chunk-table entries, updates trailing the statistics by the longest tensor's 287 items)
    for 12 steps: every element and every trust ratio against the oracle, and parameters bit
    for bit against a twin that takes the three-launch form."""
    wl = W.get_workload(1)
    flats, sets = [], []
    for _ in range(2):
        flat_p = W.alloc_flat(wl, torch.float32, DEV)
        W.init_params(wl, flat_p)
        flats.append(flat_p)
        sets.append([v.view(s) for v, s in zip(W.views(flat_p, wl), wl.shapes)])
    flat_g = W.alloc_flat(wl, torch.float32, DEV)
    grads = [v.view(s) for v, s in zip(W.views(flat_g, wl), wl.shapes)]
    src = W.GradSource(wl, DEV)
    harness.MARGINS.clear()
    hyper = dict(wl.hyper, layer_adaptation=True)
    pair = Pair(sets[0], hyper)
    twin = B.NovakOptimizer(sets[1], **hyper, layer_adaptation_in_step=0)
    for _ in range(12):
        src.fill(flat_g)
        pair.step(grads, threads=8)
        twin.step(grads)
        np.testing.assert_allclose(pair.opt.trust_ratios(), pair.oracle.trust[-1], rtol=2e-6)
    pair.check("resnet50 layer adaptation")
    assert torch.equal(flats[0], flats[1])
    assert pair.opt.trust_ratios() == twin.trust_ratios()
    assert pair.opt.info()["launches"] == 12 and twin.info()["launches"] == 36
    worst = {}
    for k, v in harness.MARGINS.items():
        worst[k.split()[-1].split("[")[0]] = max(worst.get(k.split()[-1].split("[")[0], 0.0), v)
    print("\nPARITY resnet50 layer adaptation (one launch) steps=12 every element worst |err|/tol: "
          + ", ".join(f"{k} {v:.3f}" for k, v in worst.items()))


# ---------------------------------------------------------------------------
# Phase 7: layer-wise adaptation (Eq. 19 / 25)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("extra", [dict(), dict(clip_threshold=0.05, centralize=True),
                                   dict(adaptive_beta=True, tau1=5.0, tau2=20.0)])
@pytest.mark.parametrize("variant", [("approximation", "last"), ("classical", "traj_mean"),
                                     ("none", "last")])
def test_layer_adaptation_every_element(gdtype, extra, variant):
    nesterov, mode = variant
    _, params = _shaped(SHAPES, OFFSETS)
    gen = _gen(71)
    # parameter scales from 1e-4 to 30: ratios below, inside and above the clip range
    for i, p in enumerate(params):
        p.normal_(0.0, 10.0 ** (-4 + 5.5 * i / (len(params) - 1)), generator=gen)
    pair = Pair(params, dict(BASE, nesterov=nesterov, lookahead_mode=mode,
                             layer_adaptation=True, **extra))
    _, grads = _shaped(SHAPES, OFFSETS, dtype=gdtype)
    for t in range(7):
        _fill_grads(grads, gen, std=1e-3, mean=5e-4)
        pair.step(grads)
        got = pair.opt.trust_ratios()
        np.testing.assert_allclose(got, pair.oracle.trust[-1], rtol=2e-6)
    pair.check(f"layer adaptation {extra}")
    seen = np.array(pair.oracle.trust)
    assert (seen == 0.1).any() and (seen == 10.0).any() and ((seen > 0.1) & (seen < 10.0)).any()
    # statistics and update in one launch, behind the two kernels of the gradient's own statistics
    per_step = 3 if extra.get("centralize") or extra.get("clip_threshold") else 1
    assert pair.opt.info()["launches"] == 7 * per_step
    assert pair.opt.info()["layer_adaptation"] == 1


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("lead,extra", [(0, {}), (20000, {}), (None, {}),
                                        (None, dict(clip_threshold=0.05)),
                                        (0, dict(clip_threshold=0.05, centralize=True)),
                                        (None, dict(auto_lr=True, centralize=True))])
@pytest.mark.parametrize("variant", [("approximation", "last", 5), ("classical", "traj_mean", 2),
                                     ("none", "last", 0)])
def test_layer_adaptation_in_one_launch_equals_the_three_launch_form(gdtype, lead, extra, variant):
    """Statistics and update in one grid (the updates trailing the statistics by what the
    longest tensor needs plus `lead` elements) against the two statistics kernels followed
    by the step: the same sums in the same order, so ratios, parameters and state agree bit
    for bit, over 8 steps with bf16 parameter copies switched on, also behind clipping,
    centralization and the automatic learning-rate scaling; the one-launch form is also
    held against the oracle."""
    nesterov, mode, k = variant
    shapes = SHAPES + [(70001,), (3, 30000)]
    offsets = OFFSETS + [2, 0]
    hyper = dict(BASE, nesterov=nesterov, lookahead_mode=mode, lookahead_k=k, layer_adaptation=True,
                 **extra)
    numels = [math.prod(s) for s in shapes]
    sets = []
    for in_step in (1, 0):
        _, params = _shaped(shapes, offsets)
        gen = _gen(72)
        for i, p in enumerate(params):
            p.normal_(0.0, 10.0 ** (-4 + 5.5 * i / (len(params) - 1)), generator=gen)
        copies = make_tensors(numels, DEV, offsets, dtype=torch.bfloat16)[1]
        kw = dict(layer_adaptation_in_step=in_step, param_copies=copies)
        if lead is not None:
            kw["layer_adaptation_lead"] = lead
        sets.append((params, copies, kw))
    pair = Pair(sets[0][0], hyper, opt_kwargs=sets[0][2])
    twin = B.NovakOptimizer(sets[1][0], **hyper, **sets[1][2])
    gen = _gen(73)
    _, grads = _shaped(shapes, offsets, dtype=gdtype)
    for t in range(8):
        _fill_grads(grads, gen, std=1e-3, mean=5e-4)
        pair.step(grads)
        twin.step(grads)
        assert pair.opt.trust_ratios() == twin.trust_ratios()
        np.testing.assert_allclose(pair.opt.trust_ratios(), pair.oracle.trust[-1], rtol=2e-6)
    pair.check("layer adaptation in one launch")
    for i, (x, y) in enumerate(zip(sets[0][0], sets[1][0])):
        assert torch.equal(x, y)
        assert torch.equal(sets[0][1][i], sets[1][1][i])
        assert torch.equal(sets[0][1][i].view(x.shape), x.to(torch.bfloat16))
        sa, sb = pair.opt.state(i), twin.state(i)
        for key in ("m", "v", "slow", "acc"):
            assert (sa[key] is None and sb[key] is None) or torch.equal(sa[key], sb[key])
    # in front of both: the kernels of the gradient's own statistics where phase 2 is on
    n_pre = 0 if not extra else (3 if extra.get("auto_lr") else 2)
    assert pair.opt.info()["launches"] == 8 * (1 + n_pre) and twin.info()["launches"] == 8 * (3 + n_pre)


def test_layer_adaptation_zero_gradient_and_reruns():
    """A tensor whose direction is zero gets ratio 1 (and only decays); reruns agree bit for bit."""
    shapes = [(5, 300), (4000,), (7,)]
    outs = []
    for _ in range(2):
        _, params = _shaped(shapes, [0, 0, 0])
        gen = _gen(3)
        for p in params:
            p.normal_(0.0, 0.1, generator=gen)
        before = params[2].clone()
        opt = B.NovakOptimizer(params, **BASE, layer_adaptation=True)
        _, grads = _shaped(shapes, [0, 0, 0])
        ratios = []
        for _ in range(3):
            _fill_grads(grads[:2], gen, std=1e-2)
            grads[2].zero_()
            opt.step(grads)
            ratios.append(opt.trust_ratios())
        torch.cuda.synchronize()
        assert all(r[2] == 1.0 for r in ratios)
        d = np.float32(1 - 1e-3 * 1e-2)
        expect = before * d * d * d
        assert torch.allclose(params[2], expect, rtol=1e-6, atol=0)
        outs.append((ratios, [p.clone() for p in params]))
    assert outs[0][0] == outs[1][0]
    for a, b in zip(outs[0][1], outs[1][1]):
        assert torch.equal(a, b)


def test_the_update_part_gives_up_waiting_after_its_bound_and_the_device_stays_usable():
    """The only wait on another CTA in the library (the update part of the one-launch layer
    adaptation waits for its tensor's ratio) run on a word that nothing publishes: it returns
    empty-handed after about two seconds instead of spinning on, and the same handle then
    steps as usual."""
    _, params = _shaped([(300, 40), (5000,)], [0, 0])
    gen = _gen(5)
    for p in params:
        p.normal_(0.0, 0.1, generator=gen)
    pair = Pair(params, dict(BASE, layer_adaptation=True))
    gave_up, seconds = pair.opt.handle.selftest_bounded_wait(pair.opt._stream())
    assert gave_up and 1.5 < seconds < 6.0
    _, grads = _shaped([(300, 40), (5000,)], [0, 0])
    for _ in range(3):
        _fill_grads(grads, gen, std=1e-2)
        pair.step(grads)
    pair.check("after the bounded wait")


# ---------------------------------------------------------------------------
# Phase 8: sparse updates (Eq. 27)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("nesterov", ["approximation", "classical"])
def test_sparse_mask(nesterov):
    """u 1{|u| > tau} is a yes/no decision taken on an fp32 u here and on an fp64 u in
    the oracle: an element whose |u| came within 1e-4 (relative) of tau at any step may
    legitimately differ and is left out; every other element has to match as usual."""
    numels = [70001, 33, 8192]
    tau = 0.3
    flat, views, _ = make_tensors(numels, DEV)
    gen = _gen(81)
    for p in views:
        p.normal_(0.0, 0.05, generator=gen)
    pair = Pair(views, dict(BASE, nesterov=nesterov, sparse_threshold=tau, lookahead_k=3))
    pair.oracle.track_threshold_margin = True
    _, grads, _ = make_tensors(numels, DEV)
    for _ in range(9):
        _fill_grads(grads, gen, std=1e-2)
        pair.step(grads)
    torch.cuda.synchronize()
    o = pair.oracle
    total = kept = 0
    for i, p in enumerate(views):
        sure = o.threshold_margin[i] > 1e-4
        total += sure.size
        kept += int(sure.sum())
        st = pair.opt.state(i)
        harness.assert_close(to_f64(p)[sure], o.theta[i][sure], f"sparse theta[{i}]")
        harness.assert_close(to_f64(st["slow"])[sure], o.slow[i][sure], f"sparse slow[{i}]")
        harness.assert_close(st["m"], o.m[i], f"sparse m[{i}]")      # moments ignore the mask
        harness.assert_close(st["v"], o.v[i], f"sparse v[{i}]")
    assert kept > 0.995 * total                      # only a handful of elements sit at tau
    # the mask does bite: compare with the same run without it
    flat2, views2, _ = make_tensors(numels, DEV)
    gen = _gen(81)
    for p in views2:
        p.normal_(0.0, 0.05, generator=gen)
    plain = B.NovakOptimizer(views2, **dict(BASE, nesterov=nesterov, lookahead_k=3))
    for _ in range(9):
        _fill_grads(grads, gen, std=1e-2)
        plain.step(grads)
    torch.cuda.synchronize()
    assert not torch.allclose(views[0], views2[0], rtol=1e-4, atol=1e-7)
    with pytest.raises(B.NovakError):
        pair.opt.handle.set_option(B.NOVAK_OPT_SPARSE_THRESHOLD, -0.1)


# ---------------------------------------------------------------------------
# Phase 7: automatic learning-rate scaling (Eq. 20-22)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("extra", [dict(), dict(clip_threshold=0.05, centralize=True,
                                                layer_adaptation=True, adaptive_beta=True,
                                                tau1=5.0, tau2=20.0)])
def test_auto_lr_every_element(gdtype, extra):
    _, params = _shaped(SHAPES, OFFSETS)
    gen = _gen(101)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    pair = Pair(params, dict(BASE, auto_lr=True, **extra))
    _, grads = _shaped(SHAPES, OFFSETS, dtype=gdtype)
    for t in range(8):
        # the gradient scale sweeps the ratio through its clip range
        _fill_grads(grads, gen, std=10.0 ** (-4 + 0.7 * t), mean=1e-4)
        pair.step(grads)
        g_bar, theta_bar, scale = pair.opt.handle.get_auto_lr_state(pair.opt._stream())
        o = pair.oracle
        assert abs(g_bar - o.g_bar.value) <= 1e-7 * o.g_bar.value
        assert abs(theta_bar - o.theta_bar.value) <= 1e-6 * o.theta_bar.value
        assert abs(scale - o.auto_scales[-1]) <= 2e-6 * o.auto_scales[-1]
    pair.check(f"auto lr {extra}")
    seen = pair.oracle.auto_scales
    assert min(seen) == 0.1 and max(seen) == 2.0 and any(0.1 < s < 2.0 for s in seen)
    # three statistics kernels, then the step (with layer adaptation: its one-launch form)
    assert pair.opt.info()["launches"] == 8 * (1 + 3)


def test_auto_lr_state_survives_a_checkpoint_and_a_change_of_rows():
    shapes = [(12, 300), (50,), (4, 2, 9)]

    def fresh():
        _, params = _shaped(shapes, [0, 0, 0])
        g = _gen(7)
        for p in params:
            p.normal_(0.0, 0.05, generator=g)
        return params

    def grads_for(step):
        _, grads = _shaped(shapes, [0, 0, 0])
        _fill_grads(grads, _gen(1000 + step), std=1e-2 * (1 + step))
        return grads

    a_params = fresh()
    a = B.NovakOptimizer(a_params, **BASE, auto_lr=True, clip_threshold=0.5)
    for s in range(6):
        if s == 4:      # centralization switched on mid-run re-sizes the scratch: averages kept
            a.handle.set_tensor_rows(harness.tensor_rows(a_params))
            a.handle.set_option(B.NOVAK_OPT_CENTRALIZE, 1)
        a.step(grads_for(s))
    b_params = fresh()
    b = B.NovakOptimizer(b_params, **BASE, auto_lr=True, clip_threshold=0.5)
    for s in range(3):
        b.step(grads_for(s))
    sd = b.state_dict()
    saved = [p.clone() for p in b_params]
    assert sd["auto_lr"][0] > 0 and sd["auto_lr"][1] > 0
    c_params = fresh()
    for p, q in zip(c_params, saved):
        p.copy_(q)
    c = B.NovakOptimizer(c_params, **BASE, auto_lr=True, clip_threshold=0.5)
    c.load_state_dict(sd)
    assert c.handle.get_auto_lr_state()[:2] == sd["auto_lr"]
    for s in range(3, 6):
        if s == 4:
            c.handle.set_tensor_rows(harness.tensor_rows(c_params))
            c.handle.set_option(B.NOVAK_OPT_CENTRALIZE, 1)
        c.step(grads_for(s))
    torch.cuda.synchronize()
    for x, y in zip(a_params, c_params):
        assert torch.equal(x, y)
    assert a.handle.get_auto_lr_state() == c.handle.get_auto_lr_state()
    with pytest.raises(B.NovakError):
        c.handle.set_auto_lr_state(-1.0, 0.0)
    with pytest.raises(B.NovakError):
        c.handle.set_option(B.NOVAK_OPT_AUTO_LR_GAMMA, 0.0)


# ---------------------------------------------------------------------------
# A step in two halves (groups cut across processes)
# ---------------------------------------------------------------------------
def test_two_half_step_equals_the_one_call_and_two_shards_equal_the_whole():
    numels = [70001, 33, 8192, 3000]
    hyper = dict(BASE, clip_threshold=0.02, auto_lr=True)

    def fresh(ns, seed):
        _, views, _ = make_tensors(ns, DEV)
        g = _gen(seed)
        for p in views:
            p.normal_(0.0, 0.05, generator=g)
        return views

    whole = fresh(numels, 5)
    halves = fresh(numels, 5)
    pair = Pair(whole, hyper)
    two = B.NovakOptimizer(halves, **hyper)                 # begin + finish(NULL)
    # the same group cut into two "ranks": tensors 0-1 and tensors 2-3
    cut = fresh(numels, 5)
    ranks = [B.NovakOptimizer(cut[:2], **hyper), B.NovakOptimizer(cut[2:], **hyper)]
    totals = torch.zeros(2, dtype=torch.float64, device=DEV)
    part = torch.zeros(2, dtype=torch.float64, device=DEV)
    gen = _gen(6)
    _, grads, _ = make_tensors(numels, DEV)
    for _ in range(7):
        _fill_grads(grads, gen, std=1e-3)
        pair.step(grads)
        assert two.step_begin(grads) != 0
        with pytest.raises(B.NovakError) as e:              # nothing else while the step is open
            two.step(grads)
        assert e.value.status == B.NOVAK_ESTATE
        two.step_finish(None)
        totals.zero_()
        for r, gs in zip(ranks, (grads[:2], grads[2:])):
            r.step_begin(gs)
            r.copy_local_sums(part)
            totals += part                                   # what the all-reduce would do
        for r in ranks:
            r.step_finish(totals)
    pair.check("whole group")
    for a, b in zip(whole, halves):
        assert torch.equal(a, b)                             # same kernels, same sums
    for a, b in zip(whole, cut):                             # sums added in another order
        assert torch.allclose(a, b, rtol=1e-6, atol=1e-9)
    for r in ranks:
        np.testing.assert_allclose(r.grad_stats(), pair.opt.grad_stats(), rtol=1e-12)
        np.testing.assert_allclose(r.handle.get_auto_lr_state(), pair.opt.handle.get_auto_lr_state(),
                                   rtol=1e-12)
    assert two.info()["t"] == 7 and two.info()["launches"] == pair.opt.info()["launches"] + 7
    with pytest.raises(B.NovakError) as e:
        two.step_finish(None)                                # nothing open
    assert e.value.status == B.NOVAK_ESTATE
    _, shaped = _shaped([(6, 100)], [0])
    gc = B.NovakOptimizer(shaped, **BASE, centralize=True)
    _, sg = _shaped([(6, 100)], [0])
    with pytest.raises(B.NovakError) as e:
        gc.step_begin(sg)
    assert e.value.status == B.NOVAK_ESTATE
    plain = B.NovakOptimizer(fresh([100], 1), **BASE)        # no statistics: begin does nothing
    _, pg, _ = make_tensors([100], DEV)
    assert plain.step_begin(pg) == 0
    plain.step_finish(None)
    assert plain.info()["t"] == 1 and plain.info()["launches"] == 1
