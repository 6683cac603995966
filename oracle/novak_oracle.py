"""ctypes front end of the CPU oracle (``novak_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this module, and this module imports nothing from them.

The arithmetic lives in the C file; this module only compiles it (gcc, no
fast-math), keeps the double-precision state arrays, counts steps and records
on which steps a lookahead synchronisation happened.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "novak_oracle.c")
_LIB = os.path.join(_HERE, "libnovak_oracle.so")

NESTEROV_NONE, NESTEROV_APPROX, NESTEROV_CLASSICAL, NESTEROV_TRUE = 0, 1, 2, 3
LOOKAHEAD_LAST, LOOKAHEAD_TRAJ_MEAN = 0, 1


class HParams(ctypes.Structure):
    _fields_ = [
        ("lr", ctypes.c_double),
        ("beta1", ctypes.c_double),
        ("beta2", ctypes.c_double),
        ("eps", ctypes.c_double),
        ("weight_decay", ctypes.c_double),
        ("nesterov_beta", ctypes.c_double),
        ("lookahead_alpha", ctypes.c_double),
        ("nesterov_variant", ctypes.c_int32),
        ("lookahead_k", ctypes.c_int32),
        ("lookahead_mode", ctypes.c_int32),
        ("rectified", ctypes.c_int32),
        ("bias1_power", ctypes.c_int32),
        ("adaptive_beta", ctypes.c_int32),
        ("tau1", ctypes.c_double),
        ("tau2", ctypes.c_double),
        ("sparse_threshold", ctypes.c_double),
        ("true_steps", ctypes.c_int32),
        ("moment_bf16", ctypes.c_int32),
    ]


class Scalars(ctypes.Structure):
    _fields_ = [
        ("bc1", ctypes.c_double),
        ("bc2", ctypes.c_double),
        ("rho_inf", ctypes.c_double),
        ("rho_t", ctypes.c_double),
        ("r_t", ctypes.c_double),
        ("step_size", ctypes.c_double),
        ("decay", ctypes.c_double),
        ("rect_branch", ctypes.c_int32),
        ("is_sync", ctypes.c_int32),
        ("beta1_t", ctypes.c_double),
        ("beta2_t", ctypes.c_double),
    ]


def compile_oracle(src: str = _SRC, out: str = _LIB, force: bool = False) -> str:
    """Compile the C oracle into a shared object (skipped when up to date)."""
    if (not force and os.path.exists(out)
            and os.path.getmtime(out) >= os.path.getmtime(src)):
        return out
    tmp = f"{out}.{os.getpid()}.tmp"
    subprocess.run(
        ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math",
         "-ffp-contract=off", "-o", tmp, src, "-lm"],
        check=True)
    os.replace(tmp, out)
    return out


def load_library(path: str | None = None) -> ctypes.CDLL:
    lib = ctypes.CDLL(path or compile_oracle())
    lib.novak_oracle_scalars_at.argtypes = [
        ctypes.POINTER(HParams), ctypes.c_int64, ctypes.POINTER(Scalars)]
    lib.novak_oracle_scalars_at.restype = None
    dp = ctypes.POINTER(ctypes.c_double)
    lib.novak_oracle_step.argtypes = [
        ctypes.POINTER(HParams), ctypes.c_int64, ctypes.c_int64,
        dp, dp, dp, dp, dp, dp, ctypes.c_double]
    lib.novak_oracle_step.restype = None
    lib.novak_oracle_trust_ratio.argtypes = [
        ctypes.POINTER(HParams), ctypes.c_int64, ctypes.c_int64, dp, dp, dp, dp]
    lib.novak_oracle_trust_ratio.restype = ctypes.c_double
    lib.novak_oracle_direction.argtypes = [
        ctypes.POINTER(HParams), ctypes.c_int64, ctypes.c_int64, dp, dp, dp, dp]
    lib.novak_oracle_direction.restype = None
    lib.novak_oracle_auto_lr.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                         dp, dp]
    lib.novak_oracle_auto_lr.restype = ctypes.c_double
    lib.novak_oracle_global_norm.argtypes = [
        ctypes.c_int32, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(dp)]
    lib.novak_oracle_global_norm.restype = ctypes.c_double
    lib.novak_oracle_clip_factor.argtypes = [ctypes.c_double, ctypes.c_double]
    lib.novak_oracle_clip_factor.restype = ctypes.c_double
    lib.novak_oracle_scale.argtypes = [ctypes.c_int64, ctypes.c_double, dp]
    lib.novak_oracle_scale.restype = None
    lib.novak_oracle_centralize.argtypes = [ctypes.c_int64, ctypes.c_int64, dp]
    lib.novak_oracle_centralize.restype = None
    lib.novak_oracle_round_bf16.argtypes = [ctypes.c_double]
    lib.novak_oracle_round_bf16.restype = ctypes.c_double
    lib.novak_oracle_rounding_margin.argtypes = [
        ctypes.POINTER(HParams), ctypes.c_int64, ctypes.c_int64, dp, dp, dp, dp]
    lib.novak_oracle_rounding_margin.restype = None
    lib.novak_oracle_extrapolate.argtypes = [ctypes.c_double, ctypes.c_int64, dp, dp, dp]
    lib.novak_oracle_extrapolate.restype = None
    lib.novak_oracle_wants_extrapolation.argtypes = [ctypes.POINTER(HParams), ctypes.c_int64]
    lib.novak_oracle_wants_extrapolation.restype = ctypes.c_int32
    return lib


_lib_lock = threading.Lock()
_default_lib: ctypes.CDLL | None = None


def default_library() -> ctypes.CDLL:
    global _default_lib
    with _lib_lock:
        if _default_lib is None:
            _default_lib = load_library()
        return _default_lib


@dataclass
class Config:
    """Hyperparameters in the paper's notation (Algorithm 1, Input)."""
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 1e-2
    nesterov_variant: int = NESTEROV_APPROX
    lookahead_k: int = 5
    lookahead_alpha: float = 0.5
    nesterov_beta: float | None = None   # None -> beta1
    lookahead_mode: int = LOOKAHEAD_LAST
    rectified: bool = True
    bias1_power: int = 1
    clip_threshold: float = 0.0          # c_clip; 0 = clipping off
    centralize: bool = False             # Eq. 26 on tensors given with rows > 0
    layer_adaptation: bool = False       # Eq. 19 / 25, one trust ratio per tensor
    adaptive_beta: bool = False          # Eq. 3-4
    tau1: float = 1000.0
    tau2: float = 5000.0
    sparse_threshold: float = 0.0        # tau of Eq. 27; 0 = off
    auto_lr: bool = False                # Eq. 20-22
    auto_lr_gamma: float = 0.1
    true_steps: int = 0                  # N_taylor of the true variant (Section 5.2)
    moment_bf16: bool = False            # m, v stored rounded to bfloat16

    @classmethod
    def from_hyper(cls, hyper: dict) -> "Config":
        """From the keyword spelling the workloads and tests use (``betas=(b1, b2)``,
        ``nesterov="approximation"``, ``lookahead_mode="last"``, ``moment_dtype="bf16"`` ...);
        absent keys take the defaults of the benchmark configurations; keys that only
        concern an implementation's launch (chunk sizes and the like) are ignored."""
        h = dict(hyper)
        b1, b2 = h.pop("betas", (0.9, 0.999))
        nest = {"none": NESTEROV_NONE, "approximation": NESTEROV_APPROX,
                "classical": NESTEROV_CLASSICAL, "true": NESTEROV_TRUE}
        mode = {"last": LOOKAHEAD_LAST, "traj_mean": LOOKAHEAD_TRAJ_MEAN}
        return cls(
            lr=h.pop("lr", 1e-3), beta1=b1, beta2=b2, eps=h.pop("eps", 1e-8),
            weight_decay=h.pop("weight_decay", 1e-2),
            nesterov_variant=nest[h.pop("nesterov", "approximation")],
            lookahead_k=h.pop("lookahead_k", 5), lookahead_alpha=h.pop("lookahead_alpha", 0.5),
            nesterov_beta=h.pop("nesterov_beta", None),
            lookahead_mode=mode[h.pop("lookahead_mode", "last")],
            rectified=h.pop("rectified", True), bias1_power=h.pop("bias1_power", 1),
            clip_threshold=h.pop("clip_threshold", 0.0), centralize=h.pop("centralize", False),
            layer_adaptation=h.pop("layer_adaptation", False),
            sparse_threshold=h.pop("sparse_threshold", 0.0),
            auto_lr=h.pop("auto_lr", False), auto_lr_gamma=h.pop("auto_lr_gamma", None) or 0.1,
            adaptive_beta=h.pop("adaptive_beta", False), tau1=h.pop("tau1", None) or 1000.0,
            tau2=h.pop("tau2", None) or 5000.0,
            true_steps=h.pop("true_nesterov_steps", 0),
            moment_bf16=h.pop("moment_dtype", "f32") == "bf16")

    def to_c(self) -> HParams:
        nb = self.beta1 if self.nesterov_beta is None else self.nesterov_beta
        return HParams(self.lr, self.beta1, self.beta2, self.eps,
                       self.weight_decay, nb, self.lookahead_alpha,
                       self.nesterov_variant, self.lookahead_k,
                       self.lookahead_mode, int(self.rectified),
                       self.bias1_power, int(self.adaptive_beta), self.tau1, self.tau2,
                       self.sparse_threshold, self.true_steps, int(self.moment_bf16))


def _dptr(a: np.ndarray, offset: int = 0):
    assert a.dtype == np.float64 and a.flags.c_contiguous
    return ctypes.cast(a.ctypes.data + 8 * offset,
                       ctypes.POINTER(ctypes.c_double))


class Oracle:
    """The optimizer over a list of tensors, state held in float64.

    ``params`` are the initial values (any float dtype; widened exactly).
    ``step(grads)`` advances every tensor by one NOVAK step.
    """

    def __init__(self, cfg: Config, params, lib: ctypes.CDLL | None = None, rows=None):
        """``rows[i]``: size of dimension 0 of tensor i when it has more than
        one dimension (it is then centralized when cfg.centralize), else 0."""
        self.cfg = cfg
        self.rows = list(rows) if rows is not None else None
        self.trust: list[list[float]] = []   # per step, per tensor (layer adaptation)
        self.g_bar = ctypes.c_double(0.0)    # Eq. 20
        self.theta_bar = ctypes.c_double(0.0)  # Eq. 21
        self.auto_scales: list[float] = []
        self.grad_norms: list[float] = []
        self.clip_factors: list[float] = []
        self.h = cfg.to_c()
        self.lib = lib or default_library()
        self.theta = [np.ascontiguousarray(np.asarray(p, dtype=np.float64)).reshape(-1).copy()
                      for p in params]
        self.m = [np.zeros_like(p) for p in self.theta]
        self.v = [np.zeros_like(p) for p in self.theta]
        self.slow = [p.copy() for p in self.theta] if cfg.lookahead_k > 0 else None
        self.acc = ([np.zeros_like(p) for p in self.theta]
                    if cfg.lookahead_k > 0 and cfg.lookahead_mode == LOOKAHEAD_TRAJ_MEAN
                    else None)
        self.t = 0
        self.track_threshold_margin = False
        self.track_rounding_margin = False
        self.rounding_margin = [np.full(p.size, np.inf) for p in self.theta]
        self.threshold_margin = [np.full(p.size, np.inf) for p in self.theta]
        self.sync_steps: list[int] = []
        self.rect_flags: list[int] = []

    def scalars(self, t: int) -> Scalars:
        s = Scalars()
        self.lib.novak_oracle_scalars_at(ctypes.byref(self.h), t, ctypes.byref(s))
        return s

    def wants_extrapolation(self) -> bool:
        """Whether the NEXT step expects the gradient of Eq. 11 (true variant,
        first N_taylor steps)."""
        return bool(self.lib.novak_oracle_wants_extrapolation(ctypes.byref(self.h), self.t + 1))

    def extrapolated(self):
        """Eq. 10 for every tensor: theta + beta_N m, as new arrays (the oracle's
        own parameters stay where they are, which is the save and restore of
        Section 5.8 written out)."""
        out = []
        for th, m in zip(self.theta, self.m):
            tt = np.empty_like(th)
            self.lib.novak_oracle_extrapolate(self.h.nesterov_beta, th.size, _dptr(th),
                                              _dptr(m), _dptr(tt))
            out.append(tt)
        return out

    def _run(self, i: int, g: np.ndarray, lo: int, hi: int, trust: float = 1.0):
        null = ctypes.POINTER(ctypes.c_double)()
        self.lib.novak_oracle_step(
            ctypes.byref(self.h), self.t, hi - lo,
            _dptr(self.theta[i], lo), _dptr(g, lo),
            _dptr(self.m[i], lo), _dptr(self.v[i], lo),
            _dptr(self.slow[i], lo) if self.slow is not None else null,
            _dptr(self.acc[i], lo) if self.acc is not None else null, trust)

    def _global_norm(self, arrays) -> float:
        n = len(arrays)
        numel = (ctypes.c_int64 * n)(*[a.size for a in arrays])
        ptrs = (ctypes.POINTER(ctypes.c_double) * n)(*[_dptr(a) for a in arrays])
        return self.lib.novak_oracle_global_norm(n, numel, ptrs)

    def process_gradients(self, gs):
        """Phase 2 before the Nesterov approximation: clipping on the global norm
        of the raw gradient, then centralization (both in the C file)."""
        cfg = self.cfg
        if cfg.clip_threshold <= 0 and not cfg.centralize:
            return gs
        gs = [g.copy() for g in gs]
        if cfg.clip_threshold > 0:
            n = len(gs)
            numel = (ctypes.c_int64 * n)(*[g.size for g in gs])
            ptrs = (ctypes.POINTER(ctypes.c_double) * n)(*[_dptr(g) for g in gs])
            norm = self.lib.novak_oracle_global_norm(n, numel, ptrs)
            if getattr(self, "_norms", None):
                norm = self._norms[0]
            factor = self.lib.novak_oracle_clip_factor(norm, cfg.clip_threshold)
            self.grad_norms.append(norm)
            self.clip_factors.append(factor)
            for g in gs:
                self.lib.novak_oracle_scale(g.size, factor, _dptr(g))
        if cfg.centralize:
            assert self.rows is not None and len(self.rows) == len(gs)
            for g, r in zip(gs, self.rows):
                if r > 0:
                    assert g.size % r == 0
                    self.lib.novak_oracle_centralize(r, g.size // r, _dptr(g))
        return gs

    def local_sums(self, grads):
        """(sum of squares of these gradients, sum of squares of the parameters): what one
        process of a sharded group contributes to the norms of the whole group."""
        gs = [np.ascontiguousarray(np.asarray(g, dtype=np.float64)).reshape(-1) for g in grads]
        return self._global_norm(gs) ** 2, self._global_norm(self.theta) ** 2

    def step(self, grads, threads: int = 1, global_sums=None):
        """One step.  ``threads`` > 1 splits each tensor into disjoint element
        ranges handled by separate host threads (elements are independent).
        ``global_sums``: (sum of g^2, sum of theta^2) over the WHOLE group when this
        oracle holds only a shard of it; the norms then come from these."""
        assert len(grads) == len(self.theta)
        self._norms = (None if global_sums is None
                       else (float(np.sqrt(global_sums[0])), float(np.sqrt(global_sums[1]))))
        self.t += 1
        s = self.scalars(self.t)
        self.rect_flags.append(int(s.rect_branch))
        if s.is_sync:
            self.sync_steps.append(self.t)
        gs = [np.ascontiguousarray(np.asarray(g, dtype=np.float64)).reshape(-1)
              for g in grads]
        for i, g in enumerate(gs):
            assert g.size == self.theta[i].size
        auto = 1.0
        if self.cfg.auto_lr:
            auto = self.lib.novak_oracle_auto_lr(
                self.cfg.auto_lr_gamma,
                self._norms[0] if self._norms else self._global_norm(gs),
                self._norms[1] if self._norms else self._global_norm(self.theta),
                ctypes.byref(self.g_bar), ctypes.byref(self.theta_bar))
            self.auto_scales.append(auto)
        gs = self.process_gradients(gs)
        if self.cfg.sparse_threshold > 0 and self.track_threshold_margin:
            # how close |u| comes to tau, per element, over the whole run (for tests: a
            # lower-precision implementation may decide Eq. 27 differently right at tau)
            for i, g in enumerate(gs):
                u = np.empty_like(g)
                self.lib.novak_oracle_direction(ctypes.byref(self.h), self.t, g.size, _dptr(g),
                                                _dptr(self.m[i]), _dptr(self.v[i]), _dptr(u))
                rel = np.abs(np.abs(u) / self.cfg.sparse_threshold - 1.0)
                self.threshold_margin[i] = np.minimum(self.threshold_margin[i], rel)
        if self.cfg.moment_bf16 and self.track_rounding_margin:
            # how close the unrounded moments come to a bfloat16 rounding boundary, per
            # element, over the whole run (for tests: fp32 arithmetic may round an
            # element the other way right at a boundary)
            for i, g in enumerate(gs):
                mg = np.empty_like(g)
                self.lib.novak_oracle_rounding_margin(ctypes.byref(self.h), self.t, g.size,
                                                      _dptr(g), _dptr(self.m[i]),
                                                      _dptr(self.v[i]), _dptr(mg))
                self.rounding_margin[i] = np.minimum(self.rounding_margin[i], mg)
        trust = [1.0] * len(gs)
        if self.cfg.layer_adaptation:
            trust = [self.lib.novak_oracle_trust_ratio(
                ctypes.byref(self.h), self.t, g.size, _dptr(self.theta[i]), _dptr(g),
                _dptr(self.m[i]), _dptr(self.v[i])) for i, g in enumerate(gs)]
            self.trust.append(trust)
        trust = [x * auto for x in trust]    # Eq. 24a: both multiply the step size
        if threads <= 1:
            for i, g in enumerate(gs):
                self._run(i, g, 0, g.size, trust[i])
            return
        jobs = []
        for i, g in enumerate(gs):
            n = g.size
            parts = min(threads, max(1, n // 65536))
            bounds = [n * j // parts for j in range(parts + 1)]
            jobs += [(i, g, bounds[j], bounds[j + 1], trust[i]) for j in range(parts)]
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(lambda a: self._run(*a), jobs))
