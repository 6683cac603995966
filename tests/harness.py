"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU
oracle on the same seeded inputs and compare element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import novak_oracle as O
from paper_2601_07876_b200 import binding as B
from paper_2601_07876_b200 import workloads as W

# Tolerance of the fp32 CUDA path against the fp64 oracle after N steps:
# |gpu - oracle| <= ATOL + RTOL * |oracle| for theta, m, v, slow, acc.
RTOL, ATOL = 1e-5, 1e-7

def oracle_config(hyper: dict) -> O.Config:
    return O.Config.from_hyper(hyper)


def tensor_rows(tensors):
    """Dimension 0 of every tensor with more than one dimension, else 0 (Eq. 26
    applies to tensors of dimension > 1)."""
    return [int(t.shape[0]) if t.dim() > 1 else 0 for t in tensors]


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


# Worst error seen per quantity since the last reset, as a fraction of the
# tolerance (printed by the full-size tests so that the margin is on record).
MARGINS: dict = {}
# Worst error of the moments relative to the root mean square of the quantity (the
# contract's absolute tolerance of 1e-7 is far above v ~ 1e-7 itself, so it alone
# would let a wrong second moment through).
SCALED: dict = {}
SCALED_RTOL = 1e-5


def assert_close_scaled(gpu, ref: np.ndarray, what: str):
    """|gpu - oracle| <= 1e-5 (|oracle| + rms(oracle)): a relative check at the
    quantity's own scale, for arrays whose values sit below the absolute tolerance."""
    got = to_f64(gpu) if isinstance(gpu, torch.Tensor) else np.asarray(gpu, np.float64)
    got, ref = got.reshape(-1), np.asarray(ref).reshape(-1)
    if ref.size == 0:
        return
    rms = float(np.sqrt(np.mean(ref * ref)))
    if rms == 0.0:
        assert not got.any(), f"{what}: expected all zeros"
        return
    err = np.abs(got - ref) / (np.abs(ref) + rms)
    key = what.split("[")[0]
    SCALED[key] = max(SCALED.get(key, 0.0), float(err.max()))
    i = int(err.argmax())
    assert err[i] <= SCALED_RTOL, (
        f"{what}: relative error {err[i]:.3e} at {i} (gpu={got[i]!r} oracle={ref[i]!r} rms={rms:.3e})")


def assert_close(gpu, ref: np.ndarray, what: str):
    got = to_f64(gpu) if isinstance(gpu, torch.Tensor) else np.asarray(gpu, np.float64)
    got, ref = got.reshape(-1), np.asarray(ref).reshape(-1)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = np.abs(got - ref)
    tol = ATOL + RTOL * np.abs(ref)
    if err.size:
        MARGINS[what] = max(MARGINS.get(what, 0.0), float((err / tol).max()))
    bad = err > tol
    if bad.any():
        i = int(np.argmax(err - tol))
        raise AssertionError(
            f"{what}: {int(bad.sum())}/{bad.size} elements out of tolerance; worst at {i}: "
            f"gpu={got.flat[i]!r} oracle={ref.flat[i]!r} err={err.flat[i]:.3e} tol={tol.flat[i]:.3e}")
    assert np.isfinite(got).all(), f"{what}: non-finite values"


class Pair:
    """CUDA optimizer and oracle over the same tensors (every element)."""

    def __init__(self, params, hyper: dict, opt_kwargs: dict | None = None, lib=None):
        self.params = params
        self.hyper = hyper
        self.oracle = O.Oracle(oracle_config(hyper), [to_f64(p) for p in params],
                               rows=tensor_rows(params))
        self.opt = B.NovakOptimizer(params, **hyper, **(opt_kwargs or {}), lib=lib)
        self.sync_steps = []
        self.rect_flags = []
        self.grad_norms, self.clip_factors = [], []

    def record_grad_stats(self):
        """Reads the step's gradient norm and clip factor back (synchronises)."""
        norm, factor = self.opt.grad_stats()
        self.grad_norms.append(norm)
        self.clip_factors.append(factor)

    def step(self, grads, threads=1):
        self.opt.step(grads)
        info = self.opt.info()
        if info["is_sync"]:
            self.sync_steps.append(info["t"])
        self.rect_flags.append(info["rect_branch"])
        self.oracle.step([to_f64(g) for g in grads], threads=threads)

    def check(self, what=""):
        torch.cuda.synchronize()
        o, info = self.oracle, self.opt.info()
        assert info["t"] == o.t
        assert self.sync_steps == o.sync_steps
        assert info["n_syncs"] == len(o.sync_steps)
        assert info["last_sync_step"] == (o.sync_steps[-1] if o.sync_steps else 0)
        assert self.rect_flags == o.rect_flags
        if self.grad_norms:
            # four squares at a time are added in fp32, the rest in double; the factor
            # is rounded to fp32
            np.testing.assert_allclose(self.grad_norms, o.grad_norms, rtol=1e-7)
            np.testing.assert_allclose(self.clip_factors, o.clip_factors, rtol=1e-6)
        for i, p in enumerate(self.params):
            st = self.opt.state(i)
            assert_close(p, o.theta[i], f"{what} theta[{i}]")
            assert_close(st["m"], o.m[i], f"{what} m[{i}]")
            assert_close(st["v"], o.v[i], f"{what} v[{i}]")
            assert_close_scaled(st["m"], o.m[i], f"{what} m[{i}]")
            assert_close_scaled(st["v"], o.v[i], f"{what} v[{i}]")
            if o.slow is not None:
                assert_close(st["slow"], o.slow[i], f"{what} slow[{i}]")
            else:
                assert st["slow"] is None
            if o.acc is not None and (o.cfg.lookahead_k > 1):
                # between syncs the running sum is defined; right after a sync the
                # oracle holds 0 and the kernel leaves the old sum (never read again)
                if o.t % o.cfg.lookahead_k != 0:
                    assert_close(st["acc"], o.acc[i], f"{what} acc[{i}]")


def make_tensors(numels, device, offsets=None, dtype=torch.float32, fill=None):
    """Views of one flat buffer; offsets[i] extra elements of misalignment
    (relative to a 256-byte boundary) per tensor.  Gaps hold `fill`."""
    offsets = offsets or [0] * len(numels)
    starts, cur = [], 64
    for n, o in zip(numels, offsets):
        cur = (cur + 63) // 64 * 64 + o
        starts.append(cur)
        cur += n
    total = (cur + 63) // 64 * 64 + 64
    flat = torch.zeros(total, dtype=dtype, device=device)
    if fill is not None:
        flat.fill_(fill)
    return flat, [flat[s:s + n] for s, n in zip(starts, numels)], starts


def gaps_mask(total, starts, numels, device):
    m = torch.ones(total, dtype=torch.bool, device=device)
    for s, n in zip(starts, numels):
        m[s:s + n] = False
    return m


class FullPair:
    """Full-size workload on the GPU and the oracle on EVERY element of it.

    The oracle sees the workload's flat buffer as one tensor (the step has no
    cross-element term), so its arrays line up with the flat parameter and gradient
    buffers; every tensor's elements are compared, the padding between tensors is left
    out (and must still be zero on the GPU).  The library's own state layout is
    compared tensor by tensor through novak_state_ptrs."""

    def __init__(self, wl: W.Workload, device, hyper_override: dict | None = None,
                 opt_kwargs: dict | None = None):
        self.wl = wl
        self.hyper = dict(wl.hyper, **(hyper_override or {}))
        self.flat_p = W.alloc_flat(wl, torch.float32, device)
        W.init_params(wl, self.flat_p)
        self.flat_g = W.alloc_flat(wl, wl.grad_dtype, device)
        self.scratch = (W.alloc_flat(wl, torch.float32, device)
                        if wl.grad_dtype != torch.float32 else None)
        self.params = W.views(self.flat_p, wl)
        self.grads = W.views(self.flat_g, wl)
        self.offs, _ = W.element_offsets(wl)
        self.src = W.GradSource(wl, device)
        self.oracle = O.Oracle(oracle_config(self.hyper), [to_f64(self.flat_p)])
        self.opt = B.NovakOptimizer(self.params, **self.hyper, **(opt_kwargs or {}))
        self.glist = self.opt.prepare(self.grads)
        self.sync_steps, self.rect_flags = [], []
        self.compared = 0

    def step(self, threads=1):
        self.src.fill(self.flat_g, self.scratch)
        self.opt.step(self.glist)
        info = self.opt.info()
        if info["is_sync"]:
            self.sync_steps.append(info["t"])
        self.rect_flags.append(info["rect_branch"])
        self.oracle.step([to_f64(self.flat_g)], threads=threads)

    def check(self):
        torch.cuda.synchronize()
        o, info = self.oracle, self.opt.info()
        assert info["t"] == o.t and self.sync_steps == o.sync_steps
        assert self.rect_flags == o.rect_flags
        assert info["n_syncs"] == len(o.sync_steps)
        name = self.wl.name
        # the padding between tensors is not the library's to write: still zero (the
        # gradient generator may have put numbers there, which the oracle then followed)
        pad = torch.ones(self.flat_p.numel(), dtype=torch.bool, device=self.flat_p.device)
        for off, n in zip(self.offs, self.wl.numel):
            pad[off:off + n] = False
        assert not bool(self.flat_p[pad].any()), f"{name}: padding between tensors was written"
        del pad
        theta_gpu = to_f64(self.flat_p)
        with_acc = o.acc is not None and o.cfg.lookahead_k > 1 and o.t % o.cfg.lookahead_k != 0
        for i, (off, n) in enumerate(zip(self.offs, self.wl.numel)):
            st = self.opt.state(i)
            assert_close(theta_gpu[off:off + n], o.theta[0][off:off + n], f"{name} theta")
            assert_close(st["m"], o.m[0][off:off + n], f"{name} m")
            assert_close(st["v"], o.v[0][off:off + n], f"{name} v")
            if n >= 1024:     # a root mean square needs a population
                assert_close_scaled(st["m"], o.m[0][off:off + n], f"{name} m")
                assert_close_scaled(st["v"], o.v[0][off:off + n], f"{name} v")
            if o.slow is not None:
                assert_close(st["slow"], o.slow[0][off:off + n], f"{name} slow")
            if with_acc:
                assert_close(st["acc"], o.acc[0][off:off + n], f"{name} acc")
            self.compared += n


class SampledPair:
    """Full-size workload on the GPU, oracle on a fixed sample of elements
    (exact for them: the step has no cross-element term)."""

    def __init__(self, wl: W.Workload, device, hyper_override: dict | None = None,
                 opt_kwargs: dict | None = None):
        self.wl = wl
        self.hyper = dict(wl.hyper, **(hyper_override or {}))
        self.flat_p = W.alloc_flat(wl, torch.float32, device)
        W.init_params(wl, self.flat_p)
        self.flat_g = W.alloc_flat(wl, wl.grad_dtype, device)
        self.scratch = (W.alloc_flat(wl, torch.float32, device)
                        if wl.grad_dtype != torch.float32 else None)
        self.params = W.views(self.flat_p, wl)
        self.grads = W.views(self.flat_g, wl)
        idx, tid, local = W.sample_indices(wl)
        self.idx = idx.to(device)
        self.tid, self.local = tid, local
        self.src = W.GradSource(wl, device)
        self.oracle = O.Oracle(oracle_config(self.hyper), [to_f64(self.flat_p[self.idx])])
        self.opt = B.NovakOptimizer(self.params, **self.hyper, **(opt_kwargs or {}))
        self.glist = self.opt.prepare(self.grads)
        self.sync_steps, self.rect_flags = [], []

    def step(self, threads=1):
        self.src.fill(self.flat_g, self.scratch)
        self.opt.step(self.glist)
        info = self.opt.info()
        if info["is_sync"]:
            self.sync_steps.append(info["t"])
        self.rect_flags.append(info["rect_branch"])
        self.oracle.step([to_f64(self.flat_g[self.idx])], threads=threads)

    def _gather_state(self, key):
        out = torch.empty(self.idx.numel(), dtype=torch.float32, device=self.idx.device)
        bounds = torch.searchsorted(self.tid, torch.arange(len(self.wl.numel) + 1))
        for i in range(len(self.wl.numel)):
            lo, hi = int(bounds[i]), int(bounds[i + 1])
            if hi > lo:
                out[lo:hi] = self.opt.state(i)[key][self.local[lo:hi].to(out.device)]
        return out

    def check(self):
        torch.cuda.synchronize()
        o, info = self.oracle, self.opt.info()
        assert info["t"] == o.t and self.sync_steps == o.sync_steps
        assert self.rect_flags == o.rect_flags
        assert info["n_syncs"] == len(o.sync_steps)
        name = self.wl.name
        assert_close(self.flat_p[self.idx], o.theta[0], f"{name} theta")
        assert_close(self._gather_state("m"), o.m[0], f"{name} m")
        assert_close(self._gather_state("v"), o.v[0], f"{name} v")
        assert_close_scaled(self._gather_state("m"), o.m[0], f"{name} m")
        assert_close_scaled(self._gather_state("v"), o.v[0], f"{name} v")
        if o.slow is not None:
            assert_close(self._gather_state("slow"), o.slow[0], f"{name} slow")
        if o.acc is not None and o.cfg.lookahead_k > 1 and o.t % o.cfg.lookahead_k != 0:
            assert_close(self._gather_state("acc"), o.acc[0], f"{name} acc")
