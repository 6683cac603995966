"""CUDA library against the CPU oracle, element by element, through the C ABI.

Tolerance (written in harness.py): |gpu - oracle| <= 1e-7 + 1e-5 |oracle| for
theta, m, v, slow, acc after N steps; step counters, sync-step indices and
the rectification branch flags bit-exact.
"""
import numpy as np
import pytest
import torch

from harness import Pair, assert_close, gaps_mask, make_tensors, to_f64
from paper_2601_07876_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# spans several chunks (2048 elements each) with ragged tails and tiny tensors
RAGGED = [1, 2, 3, 5, 31, 33, 1023, 1025, 8191, 8193, 70001, 4096]
BASE = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
            nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5)


def _gen(seed):
    return torch.Generator(device=DEV).manual_seed(seed)


def _fresh(numels, offsets=None, seed=1, std=0.05):
    flat, views, starts = make_tensors(numels, DEV, offsets)
    g = _gen(seed)
    for v in views:
        v.normal_(0.0, std, generator=g)
    return flat, views, starts


def _grads(numels, gen, dtype=torch.float32, offsets=None, std=1e-2, zero_frac=0.0):
    flat, views, _ = make_tensors(numels, DEV, offsets, dtype=dtype)
    for v in views:
        t = torch.empty(v.shape, dtype=torch.float32, device=DEV).normal_(0.0, std, generator=gen)
        if zero_frac:
            t[torch.rand(t.shape, generator=gen, device=DEV) < zero_frac] = 0.0
        v.copy_(t)
    return views


@pytest.mark.parametrize("nesterov", ["none", "approximation", "classical"])
@pytest.mark.parametrize("la", [(0, "last"), (5, "last"), (5, "traj_mean"), (1, "last"),
                                (1, "traj_mean"), (2, "traj_mean")])
@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_variants_ragged_multi_tensor(nesterov, la, gdtype):
    """Every Nesterov variant x lookahead mode x gradient dtype on a ragged
    multi-tensor set; 13 steps cross the branch switch (t=6) and two syncs."""
    k, mode = la
    offsets = [(i % 4) if i % 3 == 2 else 0 for i in range(len(RAGGED))]
    _, params, _ = _fresh(RAGGED, offsets)
    hyper = dict(BASE, nesterov=nesterov, lookahead_k=k, lookahead_mode=mode)
    pair = Pair(params, hyper)
    gen = _gen(100)
    for t in range(13):
        pair.step(_grads(RAGGED, gen, gdtype, offsets, zero_frac=0.01))
        if t in (0, 4, 5):
            pair.check(f"t={t + 1}")
    pair.check("end")
    if k == 5:
        assert pair.sync_steps == [5, 10]
    assert pair.rect_flags == [0] * 5 + [1] * 8
    # params and grads share their phase, so every tensor runs on 128-bit accesses
    assert not pair.opt.info()["warnings"] & B.NOVAK_WARN_SCALAR_PATH


@pytest.mark.parametrize("mode", ["last", "traj_mean"])
def test_config0_flat_1m_every_element(mode):
    """First benchmark configuration: one flat tensor of 1,048,576, 20 steps, in both
    lookahead modes."""
    from paper_2601_07876_b200 import workloads as W
    wl = W.get_workload(0)
    flat = W.alloc_flat(wl, torch.float32, DEV)
    W.init_params(wl, flat)
    params = W.views(flat, wl)
    pair = Pair(params, dict(wl.hyper, lookahead_mode=mode))
    src = W.GradSource(wl, DEV)
    gflat = W.alloc_flat(wl, torch.float32, DEV)
    for _ in range(wl.steps):
        src.fill(gflat)
        pair.step(W.views(gflat, wl), threads=4)
    pair.check(f"flat-1M {mode}")
    assert pair.sync_steps == [5, 10, 15, 20]
    assert pair.rect_flags == [0] * 5 + [1] * 15
    info = pair.opt.info()
    assert info["n_chunks"] == 1_048_576 // 2048 and info["launches"] == 20


def test_true_nesterov_runs_as_approximation():
    _, pa, _ = _fresh([5000], seed=3)
    _, pb, _ = _fresh([5000], seed=3)
    a = B.NovakOptimizer(pa, **dict(BASE, nesterov="true"))
    b = B.NovakOptimizer(pb, **dict(BASE, nesterov="approximation"))
    gen = _gen(9)
    for _ in range(3):
        g = _grads([5000], gen)
        a.step(g)
        b.step(g)
    assert torch.equal(pa[0], pb[0])
    assert a.info()["warnings"] & B.NOVAK_WARN_TRUE_DOWNGRADED


def test_mismatched_gradient_alignment_narrows_the_gradient_loads_only():
    """Gradients whose offset from a 16-byte boundary differs from the parameters' are
    fetched element by element while parameters and state keep their 128-bit accesses:
    same result, its own warning bit set."""
    numels = [3000, 9001, 17]
    _, params, _ = _fresh(numels, [0, 1, 2])
    pair = Pair(params, dict(BASE, lookahead_mode="traj_mean", lookahead_k=3))
    gen = _gen(5)
    for _ in range(7):
        pair.step(_grads(numels, gen, offsets=[1, 3, 0]))
    pair.check("narrow gradient loads")
    assert pair.opt.info()["warnings"] & B.NOVAK_WARN_NARROW_GRADIENT
    assert not pair.opt.info()["warnings"] & B.NOVAK_WARN_SCALAR_PATH


@pytest.mark.parametrize("gdtype", [torch.float32, torch.bfloat16])
def test_parameters_off_their_state_phase_take_the_scalar_path(gdtype):
    """State attached for one set of parameter addresses, then stepped with tensors at
    another offset from a 16-byte boundary: parameter and state no longer share
    alignment and everything runs on 4-byte (2-byte) accesses."""
    numels = [3000, 9001, 17, 1]
    _, params, _ = _fresh(numels, [0, 1, 2, 3])
    pair = Pair(params, dict(BASE, lookahead_k=2))
    _, moved, _ = _fresh(numels, [1, 3, 0, 1])
    for src, dst in zip(params, moved):
        dst.copy_(src)
    pair.params = moved
    pair.opt.rebind_params(moved)
    gen = _gen(6)
    for _ in range(5):
        pair.step(_grads(numels, gen, gdtype, offsets=[0, 1, 2, 3]))
    pair.check("scalar path")
    assert pair.opt.info()["warnings"] & B.NOVAK_WARN_SCALAR_PATH


def test_no_write_outside_the_tensors():
    """Sentinel-filled gaps around every parameter, gradient and state slice
    stay untouched (stands in for a memory checker)."""
    numels = [1, 7, 33, 1025, 8193, 20000]
    offsets = [0, 1, 2, 3, 0, 1]
    sent = 1234.5
    pflat, params, pstarts = make_tensors(numels, DEV, offsets, fill=sent)
    g = _gen(2)
    for v in params:
        v.normal_(0.0, 0.05, generator=g)
    gflat, grads, gstarts = make_tensors(numels, DEV, offsets, fill=sent)
    for v in grads:
        v.normal_(0.0, 1e-2, generator=g)
    # low-level attach: state buffer with sentinel pads in front and behind
    h = B.Handle(lookahead_k=2)
    h.set_option(B.NOVAK_OPT_LOOKAHEAD_MODE, B.NOVAK_LOOKAHEAD_TRAJ_MEAN)
    need = h.state_bytes(numels)
    pad = 1024
    buf = torch.full((pad + need + pad,), 0x5A, dtype=torch.uint8, device=DEV)
    base = buf.data_ptr()
    front = (-base) % 256 + 256
    stream = torch.cuda.current_stream().cuda_stream
    pp = [p.data_ptr() for p in params]
    h.attach_state(base + front, need, pp, numels, stream)
    pa, ga, na = B.ptr_array(pp), B.ptr_array([x.data_ptr() for x in grads]), B.i64_array(numels)
    g_before = gflat.clone()
    for _ in range(5):
        h.step(pa, ga, na, len(numels), B.NOVAK_GRAD_F32, stream)
    torch.cuda.synchronize()
    assert (buf[:front] == 0x5A).all() and (buf[front + need:] == 0x5A).all()
    pm = gaps_mask(pflat.numel(), pstarts, numels, DEV)
    assert (pflat[pm] == sent).all()
    assert torch.equal(gflat, g_before)                      # gradients are read only
    # inside the state buffer: everything outside the slices is still zero
    state = buf[front:front + need].view(torch.float32)
    used = torch.zeros(state.numel(), dtype=torch.bool, device=DEV)
    for i, n in enumerate(numels):
        for ptr in h.state_ptrs(i):
            off = (ptr - (base + front)) // 4
            assert not used[off:off + n].any()                # slices do not overlap
            used[off:off + n] = True
    assert (state[~used] == 0).all()
    assert h.get_info().t == 5


def test_bit_identical_reruns_and_launch_options():
    """No atomics, no reductions: two runs agree bit for bit, and so do the
    persistent-grid, small-chunk and serpentine launch policies."""
    numels = [70001, 12, 8192, 30000]
    results = []
    for kw in (dict(), dict(), dict(ctas_per_sm=2), dict(chunk_elems=1024),
               dict(serpentine=True), dict(ctas_per_sm=1, serpentine=True, chunk_elems=2048),
               dict(dependent_launch=False), dict(dependent_launch=False, ctas_per_sm=1)):
        _, params, _ = _fresh(numels, seed=4)
        opt = B.NovakOptimizer(params, **BASE, **kw)
        gen = _gen(6)
        for _ in range(6):
            opt.step(_grads(numels, gen))
        torch.cuda.synchronize()
        results.append([p.clone() for p in params] + [opt.state(0)["v"].clone()])
    for r in results[1:]:
        for a, b in zip(results[0], r):
            assert torch.equal(a, b)


def test_checkpoint_resume_is_bit_identical():
    numels = [5000, 33, 9000]
    hyper = dict(BASE, lookahead_mode="traj_mean", lookahead_k=4)
    gen = _gen(8)
    grads = [_grads(numels, gen) for _ in range(10)]
    _, pa, _ = _fresh(numels, seed=12)
    a = B.NovakOptimizer(pa, **hyper)
    for g in grads:
        a.step(g)
    _, pb, _ = _fresh(numels, seed=12)
    b = B.NovakOptimizer(pb, **hyper)
    for g in grads[:5]:
        b.step(g)
    sd = b.state_dict()
    saved = [p.clone() for p in pb]
    # resume in a new handle whose buffers sit at other addresses / phases
    _, pc, _ = _fresh(numels, [1, 2, 3], seed=99)
    for dst, src in zip(pc, saved):
        dst.copy_(src)
    c = B.NovakOptimizer(pc, **hyper)
    c.load_state_dict(sd)
    assert c.info()["t"] == 5 and c.info()["n_syncs"] == 1
    for g in grads[5:]:
        c.step(g)
    torch.cuda.synchronize()
    for x, y in zip(pa, pc):
        assert torch.equal(x, y)
    for i in range(len(numels)):
        for k in ("m", "v", "slow"):
            assert torch.equal(a.state(i)[k], c.state(i)[k])
    assert a.info()["n_syncs"] == c.info()["n_syncs"] == 2


def test_lr_and_weight_decay_schedule_between_steps():
    _, params, _ = _fresh([4097], seed=21)
    pair = Pair(params, dict(BASE))
    gen = _gen(22)
    for t in range(8):
        lr, wd = 1e-3 * (0.5 ** t), 1e-2 * (t % 3)
        pair.opt.handle.set_option(B.NOVAK_OPT_LR, lr)
        pair.opt.handle.set_option(B.NOVAK_OPT_WEIGHT_DECAY, wd)
        pair.oracle.h.lr, pair.oracle.h.weight_decay = lr, wd
        pair.step(_grads([4097], gen))
    pair.check("scheduled lr")


def test_options_rectified_off_and_bias1_power_and_beta_n():
    for extra in (dict(rectified=False), dict(bias1_power=2), dict(nesterov_beta=0.3),
                  dict(betas=(0.0, 0.5)), dict(betas=(0.8, 0.6), weight_decay=0.0)):
        _, params, _ = _fresh([3001, 64], seed=31)
        pair = Pair(params, dict(BASE, **extra))
        gen = _gen(32)
        for _ in range(9):
            pair.step(_grads([3001, 64], gen))
        pair.check(str(extra))


@pytest.mark.parametrize("nesterov", ["approximation", "classical"])
def test_adaptive_beta_warm_up(nesterov):
    """Eq. 3-4 with short time scales so that 30 steps cross most of the warm-up."""
    numels = [9000, 33, 2049]
    _, params, _ = _fresh(numels, seed=51)
    pair = Pair(params, dict(BASE, nesterov=nesterov, adaptive_beta=True, tau1=6.0, tau2=25.0))
    gen = _gen(52)
    for t in range(1, 31):
        pair.step(_grads(numels, gen))
        info, s = pair.opt.info(), pair.oracle.scalars(t)
        assert abs(info["beta1_t"] - s.beta1_t) < 1e-13 and abs(info["beta2_t"] - s.beta2_t) < 1e-13
    assert 0.89 < pair.opt.info()["beta1_t"] < 0.9
    pair.check("adaptive beta")
    # the paper's time scales as the default
    opt = B.NovakOptimizer(_fresh([100], seed=1)[1], **BASE, adaptive_beta=True)
    assert opt.plan(1000)["beta1_t"] == pytest.approx(0.9 * (1 - np.exp(-1.0)), rel=1e-12)


@pytest.mark.parametrize("copy_offsets", [None, [0, 1, 0, 2, 0, 3, 0, 0, 0, 0, 0, 0]])
def test_bf16_parameter_copies_are_the_rounded_master(copy_offsets):
    """The step also writes a bf16 copy of every updated parameter: the fp32 master matches
    the oracle as always, the copy equals the master rounded to nearest even bit for bit
    (torch's conversion as the independent check), and nothing is written beside it."""
    offsets = [0, 1, 2, 3, 0, 0, 1, 0, 3, 0, 0, 2]
    _, params, _ = _fresh(RAGGED, offsets=offsets, seed=91)
    # copies share the parameters' alignment phase, or deliberately do not
    cflat, copies, cstarts = make_tensors(RAGGED, DEV, copy_offsets or offsets,
                                          dtype=torch.bfloat16, fill=7.0)
    pair = Pair(params, dict(BASE, lookahead_k=2), opt_kwargs=dict(param_copies=copies))
    gen = _gen(92)
    for _ in range(5):
        pair.step(_grads(RAGGED, gen, offsets=offsets))
    pair.check("bf16 copies")
    for p, c in zip(params, copies):
        assert torch.equal(c, p.to(torch.bfloat16))
    gaps = gaps_mask(cflat.numel(), cstarts, RAGGED, DEV)
    assert bool((cflat[gaps] == 7.0).all())
    scalar = bool(pair.opt.info()["warnings"] & B.NOVAK_WARN_SCALAR_PATH)
    assert scalar == (copy_offsets is not None)
    # the no-allocation entry point writes them too; NULL switches them off again
    gl = pair.opt.prepare(_grads(RAGGED, gen, offsets=offsets))
    pair.opt.handle.step_noalloc(pair.opt._params_arr, gl.arr, pair.opt._numel_arr, pair.opt.n,
                                 gl.dtype, pair.opt._stream())
    torch.cuda.synchronize()
    for p, c in zip(params, copies):
        assert torch.equal(c, p.to(torch.bfloat16))
    pair.opt.set_param_copies(None)
    before = [c.clone() for c in copies]
    pair.opt.step(_grads(RAGGED, gen, offsets=offsets))
    torch.cuda.synchronize()
    for b, c in zip(before, copies):
        assert torch.equal(b, c)
    with pytest.raises(B.NovakError):
        pair.opt.handle.set_param_copies([c.data_ptr() for c in copies[:-1]])
    with pytest.raises(B.NovakError):
        pair.opt.handle.set_param_copies([c.data_ptr() + 1 for c in copies])


def test_gradient_pointers_may_change_every_step():
    numels = [9000, 100]
    _, params, _ = _fresh(numels, seed=41)
    pair = Pair(params, dict(BASE))
    gen = _gen(42)
    pool = [_grads(numels, gen) for _ in range(3)]
    for t in range(9):
        pair.step(pool[t % 3])
    pair.check("rotating pool")


def test_record_tables_are_reused_and_evicted_least_recently_used_first():
    """A pointer list seen before costs no upload; the handle keeps 8 lists and
    replaces the least recently used one.  Results match the oracle either way."""
    numels = [9000, 100, 2049]
    _, params, _ = _fresh(numels, seed=43)
    pair = Pair(params, dict(BASE))
    gen = _gen(44)
    pool = [_grads(numels, gen) for _ in range(10)]
    for t in range(12):                      # lists 0..3 in rotation: 4 uploads
        pair.step(pool[t % 4])
    assert pair.opt.info()["record_uploads"] == 4
    for i in range(4, 10):                   # 6 more lists: 10 > 8, lists 0 and 1 evicted
        pair.step(pool[i])
    assert pair.opt.info()["record_uploads"] == 10
    pair.step(pool[3])                       # still resident
    pair.step(pool[9])
    assert pair.opt.info()["record_uploads"] == 10
    pair.step(pool[0])                       # was evicted: uploaded again
    assert pair.opt.info()["record_uploads"] == 11
    pair.check("record tables")
    assert pair.opt.info()["launches"] == 21


def test_error_paths_leave_the_handle_unchanged():
    numels = [1000, 2000]
    _, params, _ = _fresh(numels, seed=51)
    opt = B.NovakOptimizer(params, **BASE)
    gen = _gen(52)
    good = _grads(numels, gen)
    opt.step(good)
    h, stream = opt.handle, torch.cuda.current_stream().cuda_stream
    pa, na = opt._params_arr, opt._numel_arr
    ga = B.ptr_array([g.data_ptr() for g in good])

    def expect(status, *args):
        with pytest.raises(B.NovakError) as e:
            h.step(*args)
        assert e.value.status == status and h.last_error()
        assert h.get_info().t == 1

    expect(B.NOVAK_ESTATE, pa, ga, B.i64_array([1000, 2001]), 2, B.NOVAK_GRAD_F32, stream)
    expect(B.NOVAK_ESTATE, pa, ga, na, 1, B.NOVAK_GRAD_F32, stream)
    expect(B.NOVAK_EINVAL, pa, ga, na, 2, 7, stream)
    expect(B.NOVAK_EINVAL, pa, B.ptr_array([good[0].data_ptr(), 0]), na, 2, B.NOVAK_GRAD_F32, stream)
    expect(B.NOVAK_EINVAL, pa, B.ptr_array([good[0].data_ptr() + 2, good[1].data_ptr()]), na, 2,
           B.NOVAK_GRAD_F32, stream)
    expect(B.NOVAK_EINVAL, None, ga, na, 2, B.NOVAK_GRAD_F32, stream)
    # layout-changing option after attach
    with pytest.raises(B.NovakError) as e:
        h.set_option(B.NOVAK_OPT_LOOKAHEAD_MODE, 1)
    assert e.value.status == B.NOVAK_ESTATE
    with pytest.raises(B.NovakError) as e:
        h.set_option(B.NOVAK_OPT_CHUNK_ELEMS, 2048)
    assert e.value.status == B.NOVAK_ESTATE
    # attach errors
    h2 = B.Handle()
    buf = torch.zeros(4096, dtype=torch.uint8, device=DEV)
    for args in ((buf.data_ptr() + 4, 2048, None, [16]), (buf.data_ptr(), 16, None, [16]),
                 (buf.data_ptr(), 4096, None, [0]), (buf.data_ptr(), 4096, [2], [16])):
        with pytest.raises(B.NovakError) as e:
            h2.attach_state(*args, stream)
        assert e.value.status == B.NOVAK_EINVAL
    # the handle still works after all of that
    opt.step(good)
    assert opt.info()["t"] == 2


@pytest.mark.parametrize("segment_elems,gdtype", [(None, torch.float32), (2048, torch.float32),
                                                  (4096, torch.bfloat16), (0, torch.float32)])
def test_step_host_matches_step_and_returns_parameters(segment_elems, gdtype):
    """novak_step_host = upload gradients, the same step, download parameters, pipelined
    in runs of the chunk table: bit-identical to novak_step whatever the run length."""
    numels = [6000, 31, 8192, 20000, 3]
    hyper = dict(BASE, lookahead_k=2)
    _, pa, _ = _fresh(numels, seed=61)
    pflat_b, pb, _ = _fresh(numels, seed=61)
    a = B.NovakOptimizer(pa, **hyper)
    b = B.NovakOptimizer(pb, **hyper)
    if segment_elems is not None:
        b.handle.set_option(B.NOVAK_OPT_HOST_SEGMENT_ELEMS, segment_elems)
    gen = _gen(62)
    total = sum(numels)
    esz = 2 if gdtype == torch.bfloat16 else 4
    gdt = B.NOVAK_GRAD_BF16 if gdtype == torch.bfloat16 else B.NOVAK_GRAD_F32
    h_g = torch.empty(total, dtype=gdtype).pin_memory()
    h_p = torch.empty(total, dtype=torch.float32).pin_memory()
    d_g = torch.empty(total, dtype=gdtype, device=DEV)
    offs = np.concatenate([[0], np.cumsum(numels)])[:-1]
    hg_arr = B.ptr_array([h_g.data_ptr() + esz * int(o) for o in offs])
    hp_arr = B.ptr_array([h_p.data_ptr() + 4 * int(o) for o in offs])
    dg_arr = B.ptr_array([d_g.data_ptr() + esz * int(o) for o in offs])
    stream = torch.cuda.current_stream().cuda_stream
    launches = 0
    for _ in range(4):
        grads = _grads(numels, gen, dtype=gdtype)
        a.step(grads)
        h_g.copy_(torch.cat([g.reshape(-1) for g in grads]).cpu())
        h_p.fill_(float("nan"))
        before = b.info()["launches"]
        b.handle.step_host(hp_arr, hg_arr, b._params_arr, dg_arr, b._numel_arr, len(numels),
                           gdt, stream)
        # work enqueued on the caller's stream afterwards sees the step finished
        seen = torch.cat([p.reshape(-1) for p in pb]).clone()
        torch.cuda.synchronize()
        launches = b.info()["launches"] - before
        expect = torch.cat([p.reshape(-1) for p in pa])
        assert torch.equal(seen, expect)
        assert torch.equal(h_p, expect.cpu())
    for x, y in zip(pa, pb):
        assert torch.equal(x, y)
    for i in range(len(numels)):
        for key in ("m", "v", "slow"):
            assert torch.equal(a.state(i)[key], b.state(i)[key])
    assert b.info()["t"] == 4 and b.info()["n_syncs"] == 2
    if segment_elems in (None, 0):
        assert launches == 1
    else:
        assert 2 <= launches <= 32


def test_zero1_wrapper_drives_the_cuda_step_world_1():
    """One rank over NCCL: reduce-scatter and all-gather degenerate to copies, the local
    CUDA step runs on views of the flat buffer and matches the oracle, also with clipping
    and auto-LR (two-half step, all-reduce of the sums of squares); options that need whole
    tensors are refused."""
    import os
    import socket
    import torch.distributed as dist
    from harness import oracle_config
    from oracle import novak_oracle as O
    from paper_2601_07876_b200 import zero1
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        numel = [5000, 33, 9000, 64]
        total = sum(numel)
        n = zero1.padded_numel(total, 1)
        gen = _gen(111)
        flat_p = torch.zeros(n, device=DEV)
        flat_p[:total].normal_(0.0, 0.05, generator=gen)
        oracle = O.Oracle(oracle_config(dict(BASE)), [to_f64(flat_p[:total])])
        opt = zero1.ShardedNovak(flat_p, numel, **BASE)
        for _ in range(6):
            flat_g = torch.zeros(n, device=DEV)
            flat_g[:total].normal_(0.0, 1e-2, generator=gen)
            oracle.step([to_f64(flat_g[:total])])
            opt.step(flat_g)
        torch.cuda.synchronize()
        assert_close(flat_p[:total], oracle.theta[0], "zero1 theta")
        assert bool((flat_p[total:] == 0).all())
        assert opt.local.info()["t"] == 6 and opt.local.info()["n_syncs"] == 1
        # clipping and auto-LR go through the two-half step with an all-reduce of two doubles
        hyper = dict(BASE, clip_threshold=0.05, auto_lr=True)
        flat_q = torch.zeros(n, device=DEV)
        flat_q[:total].normal_(0.0, 0.05, generator=gen)
        oracle = O.Oracle(oracle_config(dict(hyper)), [to_f64(flat_q[:total])])
        opt = zero1.ShardedNovak(flat_q, numel, **hyper)
        for _ in range(6):
            flat_g = torch.zeros(n, device=DEV)
            flat_g[:total].normal_(0.0, 1e-2, generator=gen)
            oracle.step([to_f64(flat_g[:total])])
            opt.step(flat_g)
        torch.cuda.synchronize()
        assert_close(flat_q[:total], oracle.theta[0], "zero1 clipped theta")
        assert min(oracle.clip_factors) < 1.0
        with pytest.raises(ValueError):
            zero1.ShardedNovak(flat_p, numel, centralize=True, **BASE)
    finally:
        dist.destroy_process_group()
