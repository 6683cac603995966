"""Python binding of the NOVAK step library (``libnovak.so``, see include/novak.h).

Argument marshalling only: every function here has the name of the C entry
point it calls and passes plain pointers and sizes through ``ctypes``.  No
arithmetic of the method runs in Python and there is no fallback: if the
library cannot be loaded (or built with nvcc) the import of this module's
users fails with the reason.

PyTorch appears only as the owner of device memory and streams:
``NovakOptimizer`` takes ``torch`` tensors, hands their ``data_ptr()`` to the
library and keeps the state buffer alive.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import (POINTER, Structure, byref, c_char_p, c_double, c_int, c_int32,
                    c_int64, c_size_t, c_uint32, c_uint64, c_void_p)

from . import build as _build

# ---- constants of include/novak.h ------------------------------------------
NOVAK_OK, NOVAK_EINVAL, NOVAK_ESTATE, NOVAK_ECUDA, NOVAK_ENOMEM = range(5)
NOVAK_NESTEROV_NONE, NOVAK_NESTEROV_APPROX, NOVAK_NESTEROV_CLASSICAL, NOVAK_NESTEROV_TRUE = range(4)
NOVAK_GRAD_F32, NOVAK_GRAD_BF16 = 0, 1
NOVAK_LOOKAHEAD_LAST, NOVAK_LOOKAHEAD_TRAJ_MEAN = 0, 1
(NOVAK_OPT_NESTEROV_BETA, NOVAK_OPT_LOOKAHEAD_MODE, NOVAK_OPT_RECTIFIED, NOVAK_OPT_LR,
 NOVAK_OPT_BIAS1_POWER, NOVAK_OPT_CHUNK_ELEMS, NOVAK_OPT_CTAS_PER_SM, NOVAK_OPT_SERPENTINE,
 NOVAK_OPT_WEIGHT_DECAY, NOVAK_OPT_DEPENDENT_LAUNCH, NOVAK_OPT_HOST_SEGMENT_ELEMS,
 NOVAK_OPT_CLIP_THRESHOLD, NOVAK_OPT_CENTRALIZE, NOVAK_OPT_ADAPTIVE_BETA, NOVAK_OPT_BETA1_TAU,
 NOVAK_OPT_BETA2_TAU, NOVAK_OPT_LAYER_ADAPTATION, NOVAK_OPT_SPARSE_THRESHOLD, NOVAK_OPT_AUTO_LR,
 NOVAK_OPT_AUTO_LR_GAMMA, NOVAK_OPT_TRUE_NESTEROV_STEPS, NOVAK_OPT_MOMENT_DTYPE,
 NOVAK_OPT_GRAPH_CAPTURABLE, NOVAK_OPT_CENTRALIZE_IN_STEP, NOVAK_OPT_LAYER_ADAPTATION_IN_STEP,
 NOVAK_OPT_LAYER_ADAPTATION_LEAD, NOVAK_OPT_LAYER_ADAPTATION_GROUP) = range(1, 28)
NOVAK_MOMENT_F32, NOVAK_MOMENT_BF16 = 0, 1
NOVAK_WARN_TRUE_DOWNGRADED, NOVAK_WARN_SCALAR_PATH, NOVAK_WARN_NARROW_GRADIENT = 1, 2, 4

_STATUS = {0: "NOVAK_OK", 1: "NOVAK_EINVAL", 2: "NOVAK_ESTATE", 3: "NOVAK_ECUDA", 4: "NOVAK_ENOMEM"}


class novak_info(Structure):
    _fields_ = [
        ("t", c_int64), ("n_syncs", c_int64), ("last_sync_step", c_int64),
        ("total_numel", c_int64), ("launches", c_int64), ("record_uploads", c_int64),
        ("bc1", c_double), ("bc2", c_double), ("rho_inf", c_double), ("rho_t", c_double),
        ("r_t", c_double), ("step_size", c_double), ("decay", c_double),
        ("rect_branch", c_int32), ("is_sync", c_int32), ("nesterov_variant", c_int32),
        ("lookahead_mode", c_int32), ("lookahead_k", c_int32), ("n_tensors", c_int32),
        ("n_chunks", c_int32), ("grid", c_int32), ("block", c_int32), ("warnings", c_uint32),
        ("grad_processing", c_int32), ("reserved", c_int32),
        ("beta1_t", c_double), ("beta2_t", c_double),
        ("layer_adaptation", c_int32), ("moment_dtype", c_int32),
    ]

    def as_dict(self) -> dict:
        return {name: getattr(self, name) for name, _ in self._fields_}


class novak_meta(Structure):
    _fields_ = [
        ("magic", c_uint64), ("t", c_int64), ("n_syncs", c_int64), ("last_sync_step", c_int64),
        ("total_numel", c_int64),
        ("lr", c_double), ("beta1", c_double), ("beta2", c_double), ("eps", c_double),
        ("weight_decay", c_double), ("nesterov_beta", c_double), ("lookahead_alpha", c_double),
        ("nesterov_variant", c_int32), ("lookahead_k", c_int32), ("lookahead_mode", c_int32),
        ("rectified", c_int32), ("bias1_power", c_int32), ("n_tensors", c_int32),
        ("warnings", c_uint32), ("centralize", c_int32), ("clip_threshold", c_double),
        ("beta1_tau", c_double), ("beta2_tau", c_double), ("adaptive_beta", c_int32),
        ("layer_adaptation", c_int32), ("sparse_threshold", c_double),
        ("auto_lr_gamma", c_double), ("auto_lr", c_int32), ("true_nesterov_steps", c_int32),
        ("moment_dtype", c_int32), ("reserved", c_int32),
    ]


class NovakError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = f"{where}: {_STATUS.get(status, status)}"
        super().__init__(f"{msg} ({detail})" if detail else msg)


_lib = None


def load_library(path: str | None = None) -> ctypes.CDLL:
    """Loads ``libnovak.so``; builds it first when it is missing or stale and
    nvcc is present.  Raises when neither works: there is no other path."""
    global _lib
    if path is None and _lib is not None:
        return _lib
    if path is None:
        path = _build.LIB
        if not _build.up_to_date():
            try:
                _build.build()
            except Exception as exc:  # a stale but loadable library is still refused
                if not os.path.exists(path):
                    raise RuntimeError(
                        f"libnovak.so is missing and could not be built: {exc}") from exc
                raise
    lib = ctypes.CDLL(path)
    vp, i64p = c_void_p, POINTER(c_int64)
    vpp = POINTER(c_void_p)
    sigs = {
        "novak_create": (c_int, [POINTER(vp), c_double, c_double, c_double, c_double, c_double,
                                 c_int, c_int, c_double]),
        "novak_destroy": (None, [vp]),
        "novak_set_option": (c_int, [vp, c_int, c_double]),
        "novak_get_option": (c_int, [vp, c_int, POINTER(c_double)]),
        "novak_state_bytes": (c_size_t, [vp, i64p, c_int]),
        "novak_attach_state": (c_int, [vp, vp, c_size_t, vpp, i64p, c_int, vp]),
        "novak_step": (c_int, [vp, vpp, vpp, i64p, c_int, c_int, vp]),
        "novak_step_noalloc": (c_int, [vp, vpp, vpp, i64p, c_int, c_int, vp]),
        "novak_step_begin": (c_int, [vp, vpp, vpp, i64p, c_int, c_int, vp]),
        "novak_local_sums": (c_int, [vp, POINTER(c_void_p)]),
        "novak_copy_local_sums": (c_int, [vp, vp, vp]),
        "novak_step_finish": (c_int, [vp, vp, vp]),
        "novak_step_host": (c_int, [vp, vpp, vpp, vpp, vpp, i64p, c_int, c_int, vp]),
        "novak_set_tensor_rows": (c_int, [vp, i64p, c_int]),
        "novak_set_param_copies": (c_int, [vp, vpp, c_int]),
        "novak_get_grad_stats": (c_int, [vp, POINTER(c_double), POINTER(c_double), vp]),
        "novak_get_auto_lr_state": (c_int, [vp, POINTER(c_double), POINTER(c_double),
                                            POINTER(c_double), vp]),
        "novak_set_auto_lr_state": (c_int, [vp, c_double, c_double]),
        "novak_get_trust_ratios": (c_int, [vp, POINTER(ctypes.c_float), c_int, vp]),
        "novak_selftest_bounded_wait": (c_int, [vp, POINTER(c_int), POINTER(c_double), vp]),
        "novak_nesterov_save_bytes": (c_size_t, [vp]),
        "novak_nesterov_extrapolate": (c_int, [vp, vpp, vp, c_size_t, i64p, c_int, vp]),
        "novak_nesterov_restore": (c_int, [vp, vpp, vp, c_size_t, i64p, c_int, vp]),
        "novak_get_info": (c_int, [vp, POINTER(novak_info)]),
        "novak_plan": (c_int, [vp, c_int64, POINTER(novak_info)]),
        "novak_state_ptrs": (c_int, [vp, c_int, vpp, vpp, vpp, vpp]),
        "novak_export_meta": (c_int, [vp, POINTER(novak_meta)]),
        "novak_import_meta": (c_int, [vp, POINTER(novak_meta)]),
        "novak_build_chunks": (c_int64, [i64p, POINTER(c_int32), c_int, c_int64,
                                         POINTER(c_int32), i64p, POINTER(c_int32), c_int64]),
        "novak_build_own_units": (c_int64, [i64p, i64p, c_int, POINTER(c_int32), i64p, i64p, c_int64]),
        "novak_build_adapt_order": (c_int64, [POINTER(c_int32), c_int, c_int64, c_int,
                                              POINTER(c_int32), POINTER(c_int32), c_int64, i64p]),
        "novak_build_row_units": (c_int64, [i64p, i64p, c_int, POINTER(c_int32), i64p, i64p, i64p,
                                            i64p, c_int64]),
        "novak_last_error": (c_char_p, [vp]),
    }
    for name, (res, args) in sigs.items():
        try:
            fn = getattr(lib, name)
        except AttributeError:
            # an alternative build given by path (tuning, A/B against an older build) may
            # lack the host-only table-builder hooks; the library proper must have everything
            if path != _build.LIB and name.startswith("novak_build_"):
                continue
            raise
        fn.restype = res
        fn.argtypes = args
    if path == _build.LIB:
        _lib = lib
    return lib


def _check(lib, handle, status: int, where: str):
    if status != NOVAK_OK:
        detail = lib.novak_last_error(handle).decode() if handle else ""
        raise NovakError(status, where, detail)


def ptr_array(ptrs):
    """Host array of pointers (``void* const*``) from Python ints."""
    return (c_void_p * len(ptrs))(*ptrs)


def i64_array(vals):
    return (c_int64 * len(vals))(*vals)


def novak_build_chunks(numel, phase=None, chunk_elems=8192, lib=None):
    """Host-only chunk-table builder; returns (tensor, offset, len) lists."""
    lib = lib or load_library()
    n = len(numel)
    num = i64_array(numel)
    ph = (c_int32 * n)(*phase) if phase is not None else None
    need = lib.novak_build_chunks(num, ph, n, chunk_elems, None, None, None, 0)
    if need < 0:
        raise NovakError(NOVAK_EINVAL, "novak_build_chunks")
    t, o, ln = (c_int32 * need)(), (c_int64 * need)(), (c_int32 * need)()
    lib.novak_build_chunks(num, ph, n, chunk_elems, t, o, ln, need)
    return list(t), list(o), list(ln)


def novak_build_row_units(numel, rows, lib=None):
    """Host-only: the statistics pass's units for tensors with rows, as a list of
    (tensor, row0, n_rows, part_off, part_len)."""
    lib = lib or load_library()
    n = len(numel)
    num, rw = i64_array(numel), i64_array(rows)
    need = lib.novak_build_row_units(num, rw, n, None, None, None, None, None, 0)
    if need < 0:
        raise NovakError(NOVAK_EINVAL, "novak_build_row_units")
    t = (c_int32 * need)()
    cols = [(c_int64 * need)() for _ in range(4)]
    lib.novak_build_row_units(num, rw, n, t, *cols, need)
    return list(zip(list(t), *[list(c) for c in cols]))


def novak_build_own_units(numel, rows, lib=None):
    """Host-only: the units of the step kernel that centralizes by itself, as a list of
    (tensor, row0, n_rows)."""
    lib = lib or load_library()
    n = len(numel)
    num, rw = i64_array(numel), i64_array(rows)
    need = lib.novak_build_own_units(num, rw, n, None, None, None, 0)
    if need < 0:
        raise NovakError(NOVAK_EINVAL, "novak_build_own_units")
    t = (c_int32 * need)()
    cols = [(c_int64 * need)() for _ in range(2)]
    lib.novak_build_own_units(num, rw, n, t, *cols, need)
    return list(zip(list(t), *[list(c) for c in cols]))


def novak_build_adapt_order(tensor_first, lead_entries, group=1, lib=None):
    """Host-only: the work list of the one-launch layer adaptation, as a list of
    (first chunk index, number of entries), and the lag between a CTA's statistics
    item and its update item."""
    lib = lib or load_library()
    n = len(tensor_first) - 1
    first = (c_int32 * (n + 1))(*tensor_first)
    need = lib.novak_build_adapt_order(first, n, lead_entries, group, None, None, 0, None)
    if need < 0:
        raise NovakError(NOVAK_EINVAL, "novak_build_adapt_order")
    out = (c_int32 * need)()
    cnt = (c_int32 * need)()
    lag = c_int64(0)
    lib.novak_build_adapt_order(first, n, lead_entries, group, out, cnt, need, ctypes.byref(lag))
    return list(zip(out, cnt)), lag.value


_NESTEROV = {"none": NOVAK_NESTEROV_NONE, "approximation": NOVAK_NESTEROV_APPROX,
             "approx": NOVAK_NESTEROV_APPROX, "classical": NOVAK_NESTEROV_CLASSICAL,
             "true": NOVAK_NESTEROV_TRUE}
_LA_MODE = {"last": NOVAK_LOOKAHEAD_LAST, "traj_mean": NOVAK_LOOKAHEAD_TRAJ_MEAN}


class Handle:
    """A ``novak_opt*`` with the C calls as methods of the same names (minus
    the prefix).  No torch here: pointers are Python ints."""

    def __init__(self, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-2,
                 nesterov_variant=NOVAK_NESTEROV_APPROX, lookahead_k=5, lookahead_alpha=0.5,
                 lib=None):
        self.lib = lib or load_library()
        h = c_void_p()
        st = self.lib.novak_create(byref(h), lr, beta1, beta2, eps, weight_decay,
                                   nesterov_variant, lookahead_k, lookahead_alpha)
        if st != NOVAK_OK:
            raise NovakError(st, "novak_create", "hyperparameter validation failed")
        self.h = h

    def destroy(self):
        if getattr(self, "h", None):
            self.lib.novak_destroy(self.h)
            self.h = None

    __del__ = destroy

    def set_option(self, key: int, value: float):
        _check(self.lib, self.h, self.lib.novak_set_option(self.h, key, float(value)),
               "novak_set_option")

    def get_option(self, key: int) -> float:
        v = c_double()
        _check(self.lib, self.h, self.lib.novak_get_option(self.h, key, byref(v)),
               "novak_get_option")
        return v.value

    def state_bytes(self, numel) -> int:
        return self.lib.novak_state_bytes(self.h, i64_array(numel), len(numel))

    def attach_state(self, d_state: int, nbytes: int, d_params, numel, stream: int = 0):
        pa = ptr_array(d_params) if d_params is not None else None
        _check(self.lib, self.h,
               self.lib.novak_attach_state(self.h, d_state, nbytes, pa, i64_array(numel),
                                           len(numel), stream),
               "novak_attach_state")

    def step(self, params_arr, grads_arr, numel_arr, n: int, grad_dtype: int, stream: int = 0):
        """``*_arr`` are ctypes arrays made with ptr_array / i64_array."""
        st = self.lib.novak_step(self.h, params_arr, grads_arr, numel_arr, n, grad_dtype, stream)
        if st != NOVAK_OK:
            _check(self.lib, self.h, st, "novak_step")

    def step_begin(self, params_arr, grads_arr, numel_arr, n: int, grad_dtype: int,
                   stream: int = 0):
        _check(self.lib, self.h,
               self.lib.novak_step_begin(self.h, params_arr, grads_arr, numel_arr, n, grad_dtype,
                                         stream), "novak_step_begin")

    def local_sums(self) -> int:
        """Device address of the two local sums of squares (0 when no statistics ran)."""
        p = c_void_p()
        _check(self.lib, self.h, self.lib.novak_local_sums(self.h, byref(p)), "novak_local_sums")
        return p.value or 0

    def copy_local_sums(self, d_dst: int, stream: int = 0):
        _check(self.lib, self.h, self.lib.novak_copy_local_sums(self.h, d_dst, stream),
               "novak_copy_local_sums")

    def step_finish(self, d_total_sums: int = 0, stream: int = 0):
        _check(self.lib, self.h, self.lib.novak_step_finish(self.h, d_total_sums or None, stream),
               "novak_step_finish")

    def step_noalloc(self, params_arr, grads_arr, numel_arr, n: int, grad_dtype: int,
                     stream: int = 0):
        """novak_step for callers that must not allocate device memory: the work
        table lives in an array inside the library (see novak.h for its limits)."""
        st = self.lib.novak_step_noalloc(self.h, params_arr, grads_arr, numel_arr, n,
                                         grad_dtype, stream)
        if st != NOVAK_OK:
            _check(self.lib, self.h, st, "novak_step_noalloc")

    def step_host(self, h_params_arr, h_grads_arr, d_params_arr, d_grads_arr, numel_arr, n,
                  grad_dtype: int, stream: int = 0):
        st = self.lib.novak_step_host(self.h, h_params_arr, h_grads_arr, d_params_arr,
                                      d_grads_arr, numel_arr, n, grad_dtype, stream)
        if st != NOVAK_OK:
            _check(self.lib, self.h, st, "novak_step_host")

    def set_tensor_rows(self, rows):
        _check(self.lib, self.h,
               self.lib.novak_set_tensor_rows(self.h, i64_array(rows), len(rows)),
               "novak_set_tensor_rows")

    def set_param_copies(self, d_copies):
        arr = ptr_array(d_copies) if d_copies is not None else None
        n = len(d_copies) if d_copies is not None else 0
        _check(self.lib, self.h, self.lib.novak_set_param_copies(self.h, arr, n),
               "novak_set_param_copies")

    def get_grad_stats(self, stream: int = 0):
        """(global gradient norm, clip factor) of the last step; synchronises the stream."""
        norm, factor = c_double(), c_double()
        _check(self.lib, self.h,
               self.lib.novak_get_grad_stats(self.h, byref(norm), byref(factor), stream),
               "novak_get_grad_stats")
        return norm.value, factor.value

    def get_auto_lr_state(self, stream: int = 0):
        """(g_bar, theta_bar, last factor) of Eq. 20-22; synchronises the stream."""
        a, b, c = c_double(), c_double(), c_double()
        _check(self.lib, self.h,
               self.lib.novak_get_auto_lr_state(self.h, byref(a), byref(b), byref(c), stream),
               "novak_get_auto_lr_state")
        return a.value, b.value, c.value

    def set_auto_lr_state(self, g_bar: float, theta_bar: float):
        _check(self.lib, self.h, self.lib.novak_set_auto_lr_state(self.h, g_bar, theta_bar),
               "novak_set_auto_lr_state")

    def get_trust_ratios(self, n: int, stream: int = 0):
        """Per-tensor trust ratios of the last step; synchronises the stream."""
        out = (ctypes.c_float * n)()
        _check(self.lib, self.h, self.lib.novak_get_trust_ratios(self.h, out, n, stream),
               "novak_get_trust_ratios")
        return list(out)

    def selftest_bounded_wait(self, stream: int = 0):
        """Runs the one-launch layer adaptation's wait on a word nobody publishes:
        (gave_up, seconds waited on the device).  Takes about two seconds."""
        gave_up, seconds = c_int(-1), c_double(0.0)
        _check(self.lib, self.h,
               self.lib.novak_selftest_bounded_wait(self.h, byref(gave_up), byref(seconds), stream),
               "novak_selftest_bounded_wait")
        return bool(gave_up.value), float(seconds.value)

    def nesterov_save_bytes(self) -> int:
        return int(self.lib.novak_nesterov_save_bytes(self.h))

    def nesterov_extrapolate(self, params_arr, d_save: int, save_bytes: int, numel_arr, n: int,
                             stream: int = 0):
        _check(self.lib, self.h,
               self.lib.novak_nesterov_extrapolate(self.h, params_arr, d_save, save_bytes, numel_arr,
                                                   n, stream), "novak_nesterov_extrapolate")

    def nesterov_restore(self, params_arr, d_save: int, save_bytes: int, numel_arr, n: int,
                         stream: int = 0):
        _check(self.lib, self.h,
               self.lib.novak_nesterov_restore(self.h, params_arr, d_save, save_bytes, numel_arr,
                                               n, stream), "novak_nesterov_restore")

    def get_info(self) -> novak_info:
        out = novak_info()
        _check(self.lib, self.h, self.lib.novak_get_info(self.h, byref(out)), "novak_get_info")
        return out

    def plan(self, t: int) -> novak_info:
        out = novak_info()
        _check(self.lib, self.h, self.lib.novak_plan(self.h, t, byref(out)), "novak_plan")
        return out

    def state_ptrs(self, tensor: int):
        m, v, s, a = c_void_p(), c_void_p(), c_void_p(), c_void_p()
        _check(self.lib, self.h,
               self.lib.novak_state_ptrs(self.h, tensor, byref(m), byref(v), byref(s), byref(a)),
               "novak_state_ptrs")
        return m.value, v.value, s.value, a.value

    def export_meta(self) -> novak_meta:
        out = novak_meta()
        _check(self.lib, self.h, self.lib.novak_export_meta(self.h, byref(out)),
               "novak_export_meta")
        return out

    def import_meta(self, meta: novak_meta):
        _check(self.lib, self.h, self.lib.novak_import_meta(self.h, byref(meta)),
               "novak_import_meta")

    def last_error(self) -> str:
        return self.lib.novak_last_error(self.h).decode()


class GradList:
    """Marshalled gradient list (pointer array + dtype), reusable across steps."""

    def __init__(self, grads):
        import torch
        dts = {g.dtype for g in grads}
        if dts == {torch.float32}:
            self.dtype = NOVAK_GRAD_F32
        elif dts == {torch.bfloat16}:
            self.dtype = NOVAK_GRAD_BF16
        else:
            raise TypeError(f"gradients must be all float32 or all bfloat16, got {dts}")
        for g in grads:
            if not g.is_contiguous() or not g.is_cuda:
                raise ValueError("gradients must be contiguous CUDA tensors")
        self.tensors = list(grads)           # keeps the memory alive
        self.numel = [g.numel() for g in grads]
        self.arr = ptr_array([g.data_ptr() for g in grads])


class NovakOptimizer:
    """NOVAK over a list of fp32 CUDA tensors (one parameter group).

    ``step(grads)`` enqueues one fused kernel on the current torch stream.  The
    tensors are updated in place; optimizer state lives in one torch-owned
    byte buffer carved by the library.
    """

    def __init__(self, params, lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
                 nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5, *,
                 nesterov_beta=None, lookahead_mode="last", rectified=True, bias1_power=1,
                 clip_threshold=0.0, centralize=False, adaptive_beta=False, tau1=None, tau2=None,
                 layer_adaptation=False, sparse_threshold=0.0, param_copies=None,
                 auto_lr=False, auto_lr_gamma=None, true_nesterov_steps=0, moment_dtype="f32",
                 graph_capturable=False, centralize_in_step=None, layer_adaptation_in_step=None,
                 layer_adaptation_lead=None, layer_adaptation_group=None,
                 chunk_elems=None, ctas_per_sm=None, serpentine=None, dependent_launch=None,
                 lib=None):
        import torch
        self.params = list(params)
        if not self.params:
            raise ValueError("empty parameter list")
        for p in self.params:
            if p.dtype != torch.float32 or not p.is_cuda or not p.is_contiguous():
                raise ValueError("parameters must be contiguous float32 CUDA tensors")
        self.device = self.params[0].device
        self._raw_stream = None
        variant = _NESTEROV[nesterov] if isinstance(nesterov, str) else int(nesterov)
        self.handle = Handle(lr, betas[0], betas[1], eps, weight_decay, variant, lookahead_k,
                             lookahead_alpha, lib=lib)
        h = self.handle
        if nesterov_beta is not None:
            h.set_option(NOVAK_OPT_NESTEROV_BETA, nesterov_beta)
        mode = _LA_MODE[lookahead_mode] if isinstance(lookahead_mode, str) else int(lookahead_mode)
        h.set_option(NOVAK_OPT_LOOKAHEAD_MODE, mode)
        self.moment_bf16 = moment_dtype in ("bf16", NOVAK_MOMENT_BF16)
        if not self.moment_bf16 and moment_dtype not in ("f32", NOVAK_MOMENT_F32):
            raise ValueError("moment_dtype must be 'f32' or 'bf16'")
        h.set_option(NOVAK_OPT_MOMENT_DTYPE, NOVAK_MOMENT_BF16 if self.moment_bf16 else NOVAK_MOMENT_F32)
        h.set_option(NOVAK_OPT_RECTIFIED, 1 if rectified else 0)
        h.set_option(NOVAK_OPT_BIAS1_POWER, bias1_power)
        if graph_capturable:
            h.set_option(NOVAK_OPT_GRAPH_CAPTURABLE, 1)
        if layer_adaptation_in_step is not None:
            h.set_option(NOVAK_OPT_LAYER_ADAPTATION_IN_STEP, 1 if layer_adaptation_in_step else 0)
        if layer_adaptation_lead is not None:
            h.set_option(NOVAK_OPT_LAYER_ADAPTATION_LEAD, layer_adaptation_lead)
        if layer_adaptation_group is not None:
            h.set_option(NOVAK_OPT_LAYER_ADAPTATION_GROUP, layer_adaptation_group)
        if centralize_in_step is not None:
            h.set_option(NOVAK_OPT_CENTRALIZE_IN_STEP, 1 if centralize_in_step else 0)
        if chunk_elems is not None:
            h.set_option(NOVAK_OPT_CHUNK_ELEMS, chunk_elems)
        if ctas_per_sm is not None:
            h.set_option(NOVAK_OPT_CTAS_PER_SM, ctas_per_sm)
        if serpentine is not None:
            h.set_option(NOVAK_OPT_SERPENTINE, 1 if serpentine else 0)
        if dependent_launch is not None:
            h.set_option(NOVAK_OPT_DEPENDENT_LAUNCH,
                         (7 if dependent_launch else 0) if isinstance(dependent_launch, bool)
                         else int(dependent_launch))
        self.numel = [p.numel() for p in self.params]
        self.n = len(self.params)
        self._numel_arr = i64_array(self.numel)
        self._param_ptrs = [p.data_ptr() for p in self.params]
        self._params_arr = ptr_array(self._param_ptrs)
        nbytes = h.state_bytes(self.numel)
        if nbytes == 0:
            raise ValueError("every parameter tensor needs at least one element")
        with torch.cuda.device(self.device):
            self.state_buffer = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            h.attach_state(self.state_buffer.data_ptr(), nbytes, self._param_ptrs, self.numel,
                           self._stream())
        self._last_grads = None
        if tau1 is not None:
            h.set_option(NOVAK_OPT_BETA1_TAU, tau1)
        if tau2 is not None:
            h.set_option(NOVAK_OPT_BETA2_TAU, tau2)
        if adaptive_beta:
            h.set_option(NOVAK_OPT_ADAPTIVE_BETA, 1)
        if layer_adaptation:
            h.set_option(NOVAK_OPT_LAYER_ADAPTATION, 1)
        if sparse_threshold:
            h.set_option(NOVAK_OPT_SPARSE_THRESHOLD, sparse_threshold)
        if auto_lr_gamma is not None:
            h.set_option(NOVAK_OPT_AUTO_LR_GAMMA, auto_lr_gamma)
        if auto_lr:
            h.set_option(NOVAK_OPT_AUTO_LR, 1)
        if clip_threshold:
            h.set_option(NOVAK_OPT_CLIP_THRESHOLD, clip_threshold)
        if centralize:
            # Eq. 26 applies to tensors with more than one dimension
            h.set_tensor_rows([p.shape[0] if p.dim() > 1 else 0 for p in self.params])
            h.set_option(NOVAK_OPT_CENTRALIZE, 1)
        self.param_copies = None
        if param_copies is not None:
            self.set_param_copies(param_copies)
        self._save = None
        if true_nesterov_steps:
            h.set_option(NOVAK_OPT_TRUE_NESTEROV_STEPS, true_nesterov_steps)

    def wants_extrapolation(self) -> bool:
        """Whether the NEXT step is a true-Nesterov step (Section 5.2: the first
        N_taylor steps), i.e. expects a gradient evaluated between extrapolate()
        and restore()."""
        t = self.handle.get_info().t + 1
        return self.handle.plan(t).nesterov_variant == NOVAK_NESTEROV_TRUE

    def extrapolate(self):
        """Eq. 10: saves the parameters and moves them to theta + beta_N m, in place."""
        import torch
        if self._save is None:
            self._save = torch.empty(self.handle.nesterov_save_bytes(), dtype=torch.uint8,
                                     device=self.device)
        self.handle.nesterov_extrapolate(self._params_arr, self._save.data_ptr(),
                                         self._save.numel(), self._numel_arr, self.n,
                                         self._stream())

    def restore(self):
        """Puts the parameters saved by extrapolate() back, bit for bit.  Only needed when
        the step is abandoned: step() called directly after extrapolate() reads the saved
        parameters itself."""
        self.handle.nesterov_restore(self._params_arr, self._save.data_ptr(), self._save.numel(),
                                     self._numel_arr, self.n, self._stream())

    def set_param_copies(self, copies):
        """bf16 tensors (one per parameter) that every step fills with the updated
        parameters rounded to nearest even; None switches them off."""
        import torch
        if copies is None:
            self.handle.set_param_copies(None)
            self.param_copies = None
            return
        copies = list(copies)
        if len(copies) != self.n:
            raise ValueError("one copy per parameter tensor")
        for c, p in zip(copies, self.params):
            if (c.dtype != torch.bfloat16 or not c.is_cuda or not c.is_contiguous()
                    or c.numel() != p.numel()):
                raise ValueError("copies must be contiguous bfloat16 CUDA tensors of the "
                                 "parameters' sizes")
        self.handle.set_param_copies([c.data_ptr() for c in copies])
        self.param_copies = copies              # keeps the memory alive

    def trust_ratios(self):
        return self.handle.get_trust_ratios(self.n, self._stream())

    def grad_stats(self):
        return self.handle.get_grad_stats(self._stream())

    def _stream(self) -> int:
        """Handle of torch's current stream on the parameters' device (the raw lookup
        where torch has it: the Stream object costs 2 us per step)."""
        raw = self._raw_stream
        if raw is None:
            import torch
            raw = getattr(torch._C, "_cuda_getCurrentRawStream", False)
            if raw:
                index = self.device.index
                if index is None:
                    index = torch.cuda.current_device()
                self._raw_stream = raw = (raw, index)
            else:
                self._raw_stream = raw = False
        if raw:
            return raw[0](raw[1])
        import torch
        return torch.cuda.current_stream(self.device).cuda_stream

    def rebind_params(self, params):
        """The same parameters at new addresses (tensors that were moved or re-created):
        later steps take these pointers; the attached state stays as it is.  State
        slices keep the alignment phase of the tensors given at construction, so
        tensors at another offset from a 16-byte boundary run on narrow accesses."""
        params = list(params)
        if [p.numel() for p in params] != self.numel:
            raise ValueError("parameter shapes do not match the attached layout")
        for p in params:
            if p.dtype != self.params[0].dtype or not p.is_cuda or not p.is_contiguous():
                raise ValueError("parameters must be contiguous float32 CUDA tensors")
        self.params = params
        self._param_ptrs = [p.data_ptr() for p in params]
        self._params_arr = ptr_array(self._param_ptrs)

    def prepare(self, grads) -> GradList:
        gl = GradList(grads)
        if gl.numel != self.numel:
            raise ValueError("gradient shapes do not match the parameters")
        return gl

    def step(self, grads):
        """One step.  ``grads``: list of tensors, or a ``GradList`` from prepare()."""
        gl = grads if isinstance(grads, GradList) else self.prepare(grads)
        h = self.handle
        st = h.lib.novak_step(h.h, self._params_arr, gl.arr, self._numel_arr, self.n, gl.dtype,
                              self._stream())
        if st != NOVAK_OK:
            _check(h.lib, h.h, st, "novak_step")
        self._last_grads = gl

    def step_begin(self, grads):
        """First half of a step for a group cut across processes: local statistics.
        Returns the device address of the two local sums of squares (0: none needed)."""
        gl = grads if isinstance(grads, GradList) else self.prepare(grads)
        self.handle.step_begin(self._params_arr, gl.arr, self._numel_arr, self.n, gl.dtype,
                               self._stream())
        self._last_grads = gl
        return self.handle.local_sums()

    def copy_local_sums(self, out):
        """Copies the open step's two local sums into ``out`` (CUDA float64, 2 elements)."""
        self.handle.copy_local_sums(out.data_ptr(), self._stream())

    def step_finish(self, total_sums=None):
        """Second half: ``total_sums`` is a CUDA float64 tensor of 2 elements holding the
        all-reduced sums (None: the local ones)."""
        ptr = total_sums.data_ptr() if total_sums is not None else 0
        self.handle.step_finish(ptr, self._stream())

    def info(self) -> dict:
        return self.handle.get_info().as_dict()

    def plan(self, t: int) -> dict:
        return self.handle.plan(t).as_dict()

    def _view(self, ptr, numel, bf16=False):
        import torch
        if not ptr:
            return None
        off = ptr - self.state_buffer.data_ptr()
        if bf16:
            return self.state_buffer[off: off + 2 * numel].view(torch.bfloat16)
        return self.state_buffer[off: off + 4 * numel].view(self.params[0].dtype)

    def state(self, i: int) -> dict:
        """Views (no copies) of tensor i's state slices inside the state buffer."""
        m, v, s, a = self.handle.state_ptrs(i)
        n = self.numel[i]
        b = self.moment_bf16
        return {"m": self._view(m, n, b), "v": self._view(v, n, b), "slow": self._view(s, n),
                "acc": self._view(a, n)}

    def state_dict(self) -> dict:
        """Layout-independent checkpoint: counters + per-tensor copies of the state
        (+ the two averages of the automatic learning-rate scaling)."""
        meta = self.handle.export_meta()
        tensors = []
        for i in range(self.n):
            tensors.append({k: (t.clone() if t is not None else None)
                            for k, t in self.state(i).items()})
        g_bar, theta_bar, _ = self.handle.get_auto_lr_state(self._stream())
        return {"meta": bytes(meta), "tensors": tensors, "auto_lr": (g_bar, theta_bar)}

    def load_state_dict(self, sd: dict):
        meta = novak_meta.from_buffer_copy(sd["meta"])
        self.handle.import_meta(meta)
        if "auto_lr" in sd:
            self.handle.set_auto_lr_state(*sd["auto_lr"])
        for i, saved in enumerate(sd["tensors"]):
            for k, dst in self.state(i).items():
                if dst is not None:
                    dst.copy_(saved[k])
