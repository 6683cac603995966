"""novak_step_noalloc against novak_step, through the C ABI.

Some users of this library run where device memory cannot be allocated any
more once training has started: a framework's caching pool has reserved the
whole GPU, or the call happens at a point (an allocator callback, a latency
critical loop) where cudaMalloc is off limits.  novak_step's first call
allocates a small work table on the device; novak_step_noalloc keeps that table
in an array compiled into the library instead.  This test drives both entry
points with identical inputs and requires identical results, on two calls in a
row and beyond, with two handles taking turns on the one shared table.

Collected last on purpose (file name), and written to pass both alone in a
fresh process and after every other test.
"""
import pytest
import torch

from harness import ATOL, RTOL, make_tensors
from paper_2601_07876_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
HYPER = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
             nesterov="approximation", lookahead_k=2, lookahead_alpha=0.5)
NUMELS = [70001, 33, 2048, 1, 9000]
OFFSETS = [0, 1, 0, 3, 2]


def _setup(seed, mode="last"):
    _, params, _ = make_tensors(NUMELS, DEV, OFFSETS)
    gen = torch.Generator(device=DEV).manual_seed(seed)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    return params, B.NovakOptimizer(params, **HYPER, lookahead_mode=mode)


def _grads(gen):
    _, grads, _ = make_tensors(NUMELS, DEV, OFFSETS)
    for g in grads:
        g.normal_(0.0, 1e-2, generator=gen)
    return grads


def _close(a, b):
    return bool(((a - b).abs() <= ATOL + RTOL * b.abs()).all())


def _step_noalloc(opt, grads):
    gl = opt.prepare(grads)
    opt.handle.step_noalloc(opt._params_arr, gl.arr, opt._numel_arr, opt.n, gl.dtype,
                            torch.cuda.current_stream().cuda_stream)
    return gl


def test_noalloc_matches_step_on_consecutive_calls():
    pa, a = _setup(7)                      # reference: novak_step
    pb, b = _setup(7)                      # under test: novak_step_noalloc
    pc, c = _setup(8, mode="traj_mean")    # a second user of the shared table
    pd, d = _setup(8, mode="traj_mean")
    gen = torch.Generator(device=DEV).manual_seed(70)
    keep = []
    for t in range(1, 6):
        grads = _grads(gen)
        a.step(grads)
        keep.append(_step_noalloc(b, grads))
        if t >= 2:
            # handles c (noalloc) and d (step) join: the table now changes owner every call
            d.step(grads)
            keep.append(_step_noalloc(c, grads))
        torch.cuda.synchronize()
        for x, y in zip(pa, pb):
            assert _close(y, x), f"step {t}: parameters differ"
            assert torch.equal(x, y)       # same kernel, same table contents: same bits
        for i in range(len(NUMELS)):
            sa, sb = a.state(i), b.state(i)
            for k in ("m", "v", "slow"):
                assert _close(sb[k], sa[k]) and torch.equal(sa[k], sb[k])
        for x, y in zip(pd, pc):
            assert torch.equal(x, y)
    ia, ib = a.info(), b.info()
    assert ia["t"] == ib["t"] == 5 and ia["n_syncs"] == ib["n_syncs"] == 2
    assert ib["launches"] == 5 and ib["n_chunks"] == 0    # no allocated table behind b
    # both entry points may be mixed on one handle
    grads = _grads(gen)
    a.step(grads)
    b.step(grads)
    torch.cuda.synchronize()
    for x, y in zip(pa, pb):
        assert torch.equal(x, y)


def test_noalloc_rejects_sizes_beyond_the_static_table():
    # too many chunk-table entries: 131073 x 1024 elements at the smallest chunk size
    n = 131073 * 1024
    big = torch.zeros(n, dtype=torch.float32, device=DEV)
    g = torch.zeros(n, dtype=torch.float32, device=DEV)
    opt = B.NovakOptimizer([big], **HYPER, chunk_elems=1024)
    with pytest.raises(B.NovakError) as e:
        _step_noalloc(opt, [g])
    assert e.value.status == B.NOVAK_EINVAL and "131072" in str(e.value)
    assert opt.info()["t"] == 0
    opt.step([g])                          # the allocating entry point still takes it
    assert opt.info()["t"] == 1
    del opt, big, g
    # too many tensors
    flat = torch.zeros(4097 * 64, dtype=torch.float32, device=DEV)
    many = [flat[i * 64:i * 64 + 8] for i in range(4097)]
    opt = B.NovakOptimizer(many, **HYPER)
    with pytest.raises(B.NovakError) as e:
        _step_noalloc(opt, many)
    assert e.value.status == B.NOVAK_EINVAL and "4096" in str(e.value)
    assert opt.info()["t"] == 0
    torch.cuda.synchronize()


def test_noalloc_against_the_oracle():
    """The entry point on its own merits: 12 steps of novak_step_noalloc against the CPU
    oracle on every element (rectification switch at t = 6, six lookahead syncs), rather
    than only through its agreement with novak_step."""
    from harness import Pair
    _, params, _ = make_tensors(NUMELS, DEV, OFFSETS)
    gen = torch.Generator(device=DEV).manual_seed(9)
    for p in params:
        p.normal_(0.0, 0.05, generator=gen)
    for mode in ("last", "traj_mean"):
        pair = Pair([p.clone() for p in params], dict(HYPER, lookahead_mode=mode))
        keep = []
        pair.opt.step = lambda grads: keep.append(_step_noalloc(pair.opt, grads))
        for _ in range(12):
            pair.step(_grads(gen))
        pair.check(f"noalloc {mode}")
        assert pair.sync_steps == [2, 4, 6, 8, 10, 12]
        assert pair.rect_flags == [0] * 5 + [1] * 7
        info = pair.opt.info()
        assert info["launches"] == 12 and info["n_chunks"] == 0   # nothing was allocated for it


def test_noalloc_two_host_threads_on_one_stream():
    """Two host threads, a handle each, call novak_step_noalloc at the same time.  Both
    enqueue on ONE stream, so the GPU side is ordered and only the host side interleaves:
    the table must always hold the calling handle's own records when its kernel is
    enqueued.  Each result has to equal, bit for bit, what novak_step gives that handle's
    twin from the same gradients."""
    import threading
    steps = 150
    pa, a = _setup(21)                     # thread 1, noalloc
    pb, b = _setup(22, mode="traj_mean")   # thread 2, noalloc
    ra, ta = _setup(21)                    # their twins on novak_step
    rb, tb = _setup(22, mode="traj_mean")
    gen = torch.Generator(device=DEV).manual_seed(23)
    ga = [_grads(gen) for _ in range(3)]
    gb = [_grads(gen) for _ in range(3)]
    la, lb = [a.prepare(g) for g in ga], [b.prepare(g) for g in gb]
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    raw = stream.cuda_stream
    start = threading.Barrier(2)
    errors = []

    def run(opt, lists):
        try:
            start.wait()
            for i in range(steps):
                gl = lists[i % 3]
                opt.handle.step_noalloc(opt._params_arr, gl.arr, opt._numel_arr, opt.n, gl.dtype, raw)
        except Exception as exc:            # pragma: no cover
            errors.append(exc)

    threads = [threading.Thread(target=run, args=(a, la)), threading.Thread(target=run, args=(b, lb))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    stream.synchronize()
    assert not errors, errors
    for i in range(steps):
        ta.step(ga[i % 3])
        tb.step(gb[i % 3])
    torch.cuda.synchronize()
    assert a.info()["t"] == b.info()["t"] == steps
    for x, y in zip(ra, pa):
        assert torch.equal(x, y)
    for x, y in zip(rb, pb):
        assert torch.equal(x, y)
    for i in range(len(NUMELS)):
        for k in ("m", "v", "slow"):
            assert torch.equal(ta.state(i)[k], a.state(i)[k])
            assert torch.equal(tb.state(i)[k], b.state(i)[k])
