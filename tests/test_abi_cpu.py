"""Host-side checks of the C-ABI library that need no GPU: exported symbols,
hyperparameter validation, the downgrade rule, the scalar planner against the
oracle's independently computed scalars, the chunk-table builder."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import novak_oracle as O
from paper_2601_07876_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "novak.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(novak_[a-z_]+)\s*\(", header))
    assert {"novak_create", "novak_step", "novak_destroy"} <= names
    for name in sorted(names):
        assert hasattr(lib, name), f"{name} declared in novak.h but not exported"
    # and the binding declares a signature for each of them
    src = open(os.path.join(ROOT, "paper_2601_07876_b200", "binding.py")).read()
    for name in sorted(names):
        assert f'"{name}"' in src, f"binding has no signature for {name}"


def test_struct_layouts_match_header(lib, tmp_path):
    """gcc compiles include/novak.h and prints sizeof / offsetof of every field;
    the ctypes mirrors must agree (a drifted or missing field shifts an offset)."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("gcc not found")
    lines = ["#include <stdio.h>", "#include <stddef.h>", '#include "novak.h"', "int main(void){"]
    for cls in (B.novak_info, B.novak_meta):
        name = cls.__name__
        lines.append(f'printf("{name} %zu\\n", sizeof({name}));')
        for field, _ in cls._fields_:
            lines.append(f'printf("{name}.{field} %zu\\n", offsetof({name}, {field}));')
    lines.append("return 0;}")
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([gcc, "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    got = dict(l.split() for l in subprocess.run([str(exe)], capture_output=True, text=True,
                                                 check=True).stdout.splitlines())
    for cls in (B.novak_info, B.novak_meta):
        name = cls.__name__
        assert int(got[name]) == ctypes.sizeof(cls)
        for field, _ in cls._fields_:
            assert int(got[f"{name}.{field}"]) == getattr(cls, field).offset, field


GOOD = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-2,
            nesterov_variant=1, lookahead_k=5, lookahead_alpha=0.5)


@pytest.mark.parametrize("bad", [
    dict(lr=0.0), dict(lr=-1.0), dict(lr=float("nan")), dict(lr=float("inf")),
    dict(beta1=1.0), dict(beta1=-0.1), dict(beta2=1.0), dict(beta2=1 - 1e-9),
    dict(beta2=float("nan")), dict(eps=0.0), dict(eps=-1e-8), dict(weight_decay=-1e-3),
    dict(nesterov_variant=4), dict(nesterov_variant=-1), dict(lookahead_k=-1),
    dict(lookahead_alpha=0.0), dict(lookahead_alpha=1.0), dict(lookahead_alpha=float("nan")),
])
def test_create_rejects_invalid_hyperparameters(bad):
    """Section 5.8, hyperparameter validation."""
    with pytest.raises(B.NovakError) as e:
        B.Handle(**{**GOOD, **bad})
    assert e.value.status == B.NOVAK_EINVAL


def test_create_accepts_boundaries():
    B.Handle(**{**GOOD, "beta1": 0.0, "beta2": 0.0, "weight_decay": 0.0}).destroy()
    # lookahead off: alpha is not looked at
    B.Handle(**{**GOOD, "lookahead_k": 0, "lookahead_alpha": 7.0}).destroy()


def test_true_nesterov_is_downgraded_with_warning():
    """Section 7.3: the fast path runs 'true' as 'approximation' and warns."""
    h = B.Handle(**{**GOOD, "nesterov_variant": B.NOVAK_NESTEROV_TRUE})
    info = h.get_info()
    assert info.nesterov_variant == B.NOVAK_NESTEROV_APPROX
    assert info.warnings & B.NOVAK_WARN_TRUE_DOWNGRADED
    h2 = B.Handle(**GOOD)
    assert h2.get_info().warnings == 0


def test_true_nesterov_steps_then_fallback_to_the_approximation():
    """Section 5.2: with N_taylor > 0 the first N_taylor steps are true steps (no Eq. 13
    correction to the gradient given), later ones the approximation; the warning goes."""
    h = B.Handle(**{**GOOD, "nesterov_variant": B.NOVAK_NESTEROV_TRUE})
    assert h.get_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS) == 0
    h.set_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS, 3)
    assert h.get_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS) == 3
    assert not (h.get_info().warnings & B.NOVAK_WARN_TRUE_DOWNGRADED)
    got = [h.plan(t).nesterov_variant for t in range(1, 7)]
    assert got == [B.NOVAK_NESTEROV_TRUE] * 3 + [B.NOVAK_NESTEROV_APPROX] * 3
    # the oracle takes the same decision
    from oracle import novak_oracle as O
    olib = O.default_library()
    hp = O.Config(nesterov_variant=O.NESTEROV_TRUE, true_steps=3).to_c()
    import ctypes
    assert [olib.novak_oracle_wants_extrapolation(ctypes.byref(hp), t) for t in range(1, 7)] == \
        [int(v == B.NOVAK_NESTEROV_TRUE) for v in got]
    h.set_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS, 0)
    assert h.get_info().warnings & B.NOVAK_WARN_TRUE_DOWNGRADED
    assert h.plan(1).nesterov_variant == B.NOVAK_NESTEROV_APPROX
    for bad in (-1, 2.5, float("nan"), 2.0 ** 31):
        with pytest.raises(B.NovakError):
            h.set_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS, bad)
    meta = h.export_meta()
    assert meta.nesterov_variant == B.NOVAK_NESTEROV_TRUE and meta.true_nesterov_steps == 0
    h.destroy()
    # any other variant: the option is refused, the helpers too (nothing attached either)
    g = B.Handle(**GOOD)
    with pytest.raises(B.NovakError):
        g.set_option(B.NOVAK_OPT_TRUE_NESTEROV_STEPS, 5)
    assert g.nesterov_save_bytes() == 0
    g.destroy()


def test_graph_capturable_option():
    h = B.Handle(**GOOD)
    assert h.get_option(B.NOVAK_OPT_GRAPH_CAPTURABLE) == 0
    h.set_option(B.NOVAK_OPT_GRAPH_CAPTURABLE, 1)
    assert h.get_option(B.NOVAK_OPT_GRAPH_CAPTURABLE) == 1
    for bad in (2, -1, 0.5, float("nan")):
        with pytest.raises(B.NovakError):
            h.set_option(B.NOVAK_OPT_GRAPH_CAPTURABLE, bad)
    assert h.get_info().t == 0          # nothing on the device yet: no read-back, no CUDA call
    h.destroy()


def test_in_step_options_roundtrip_and_defaults():
    """Centralization inside the step kernel and the one-launch layer adaptation are on
    by default; its lead is an element count, its group a number of entries."""
    h = B.Handle(**GOOD)
    assert h.get_option(B.NOVAK_OPT_CENTRALIZE_IN_STEP) == 1
    assert h.get_option(B.NOVAK_OPT_LAYER_ADAPTATION_IN_STEP) == 1
    assert h.get_option(B.NOVAK_OPT_LAYER_ADAPTATION_LEAD) == 0
    assert h.get_option(B.NOVAK_OPT_LAYER_ADAPTATION_GROUP) == 4
    h.set_option(B.NOVAK_OPT_LAYER_ADAPTATION_GROUP, 8)
    assert h.get_option(B.NOVAK_OPT_LAYER_ADAPTATION_GROUP) == 8
    h.set_option(B.NOVAK_OPT_CENTRALIZE_IN_STEP, 0)
    h.set_option(B.NOVAK_OPT_LAYER_ADAPTATION_IN_STEP, 0)
    h.set_option(B.NOVAK_OPT_LAYER_ADAPTATION_LEAD, 2 ** 20)
    assert h.get_option(B.NOVAK_OPT_CENTRALIZE_IN_STEP) == 0
    assert h.get_option(B.NOVAK_OPT_LAYER_ADAPTATION_IN_STEP) == 0
    assert h.get_option(B.NOVAK_OPT_LAYER_ADAPTATION_LEAD) == 2 ** 20
    for key, bad in ((B.NOVAK_OPT_CENTRALIZE_IN_STEP, 2), (B.NOVAK_OPT_LAYER_ADAPTATION_IN_STEP, -1),
                     (B.NOVAK_OPT_LAYER_ADAPTATION_LEAD, -1), (B.NOVAK_OPT_LAYER_ADAPTATION_LEAD, 0.5),
                     (B.NOVAK_OPT_LAYER_ADAPTATION_LEAD, 2.0 ** 31),
                     (B.NOVAK_OPT_LAYER_ADAPTATION_GROUP, 0), (B.NOVAK_OPT_LAYER_ADAPTATION_GROUP, 9),
                     (B.NOVAK_OPT_LAYER_ADAPTATION_GROUP, 2.5)):
        with pytest.raises(B.NovakError) as e:
            h.set_option(key, bad)
        assert e.value.status == B.NOVAK_EINVAL
    h.destroy()


def test_options_validate_and_roundtrip():
    h = B.Handle(**GOOD)
    assert h.get_option(B.NOVAK_OPT_NESTEROV_BETA) == 0.9   # default beta_N = beta1
    h.set_option(B.NOVAK_OPT_NESTEROV_BETA, 0.5)
    assert h.get_option(B.NOVAK_OPT_NESTEROV_BETA) == 0.5
    for key, bad in ((B.NOVAK_OPT_NESTEROV_BETA, 1.0), (B.NOVAK_OPT_LOOKAHEAD_MODE, 2),
                     (B.NOVAK_OPT_RECTIFIED, 3), (B.NOVAK_OPT_LR, 0.0),
                     (B.NOVAK_OPT_BIAS1_POWER, 3), (B.NOVAK_OPT_CHUNK_ELEMS, 1000),
                     (B.NOVAK_OPT_CTAS_PER_SM, -1), (B.NOVAK_OPT_WEIGHT_DECAY, -1.0),
                     (99, 1.0)):
        with pytest.raises(B.NovakError) as e:
            h.set_option(key, bad)
        assert e.value.status == B.NOVAK_EINVAL
        assert h.last_error()
    h.set_option(B.NOVAK_OPT_LR, 5e-4)
    assert h.get_option(B.NOVAK_OPT_LR) == 5e-4


def test_step_without_state_is_estate():
    h = B.Handle(**GOOD)
    arr = B.ptr_array([16])
    with pytest.raises(B.NovakError) as e:
        h.step(arr, arr, B.i64_array([4]), 1, B.NOVAK_GRAD_F32)
    assert e.value.status == B.NOVAK_ESTATE
    assert h.get_info().t == 0


def test_state_bytes():
    h = B.Handle(**GOOD)                       # lookahead LAST: m, v, slow
    # each tensor gets a slot of round_up(numel + 31, 32) elements
    assert h.state_bytes([1]) == 3 * 32 * 4
    assert h.state_bytes([32, 33]) == 3 * (64 + 64) * 4
    assert h.state_bytes([0]) == 0 and h.state_bytes([5, -1]) == 0
    h.set_option(B.NOVAK_OPT_LOOKAHEAD_MODE, B.NOVAK_LOOKAHEAD_TRAJ_MEAN)
    assert h.state_bytes([1]) == 4 * 32 * 4
    h0 = B.Handle(**{**GOOD, "lookahead_k": 0})
    assert h0.state_bytes([1]) == 2 * 32 * 4


@pytest.mark.parametrize("kw", [
    dict(), dict(beta1=0.8, beta2=0.99), dict(beta2=0.6), dict(beta1=0.0, beta2=0.5),
    dict(beta2=0.9999, lr=3e-2, weight_decay=0.3), dict(lookahead_k=1), dict(lookahead_k=7),
])
def test_planner_agrees_with_oracle_scalars(kw):
    """The library's scalar plan (-expm1(t log beta), double) against the
    oracle's (powl, long double): Eq. 5-9, 18 and the sync schedule."""
    g = {**GOOD, **kw}
    h = B.Handle(**g)
    o = O.Oracle(O.Config(lr=g["lr"], beta1=g["beta1"], beta2=g["beta2"], eps=g["eps"],
                          weight_decay=g["weight_decay"], lookahead_k=g["lookahead_k"],
                          lookahead_alpha=g["lookahead_alpha"]), [np.zeros(1)])
    for t in list(range(1, 40)) + [100, 999, 1000, 1001, 12345, 10 ** 6, 10 ** 8]:
        a, b = h.plan(t), o.scalars(t)
        assert a.rect_branch == b.rect_branch and a.is_sync == b.is_sync, t
        for name in ("bc1", "bc2", "rho_inf", "r_t", "step_size", "decay"):
            x, y = getattr(a, name), getattr(b, name)
            assert abs(x - y) <= 1e-12 * abs(y), (t, name, x, y)
        assert abs(a.rho_t - b.rho_t) <= 1e-9 * max(1.0, b.rho_inf), (t, a.rho_t, b.rho_t)


def test_planner_options():
    h = B.Handle(**GOOD)
    h.set_option(B.NOVAK_OPT_RECTIFIED, 0)
    assert h.plan(50).rect_branch == 0 and h.plan(50).r_t == 1.0
    h.set_option(B.NOVAK_OPT_RECTIFIED, 1)
    p1 = h.plan(7)
    h.set_option(B.NOVAK_OPT_BIAS1_POWER, 2)
    p2 = h.plan(7)
    assert abs(p2.step_size * p2.bc1 - p1.step_size) < 1e-18


def test_planner_adaptive_beta_agrees_with_oracle():
    """Eq. 3-4 in the library's plan (-expm1(-t/tau)) against the oracle's (1 - exp)."""
    h = B.Handle(**GOOD)
    for name in ("beta1_t", "beta2_t"):
        assert getattr(h.plan(3), name) == GOOD[name[:5]]        # off: the base values
    h.set_option(B.NOVAK_OPT_ADAPTIVE_BETA, 1)
    assert h.get_option(B.NOVAK_OPT_BETA1_TAU) == 1000.0
    assert h.get_option(B.NOVAK_OPT_BETA2_TAU) == 5000.0
    for taus in ((1000.0, 5000.0), (7.0, 20.0), (500.0, 2500.0)):
        h.set_option(B.NOVAK_OPT_BETA1_TAU, taus[0])
        h.set_option(B.NOVAK_OPT_BETA2_TAU, taus[1])
        o = O.Oracle(O.Config(adaptive_beta=True, tau1=taus[0], tau2=taus[1]), [np.zeros(1)])
        ref = B.Handle(**GOOD)
        for t in [1, 2, 5, 6, 100, 1000, 5000, 10 ** 5, 10 ** 7]:
            a, b, r = h.plan(t), o.scalars(t), ref.plan(t)
            assert abs(a.beta1_t - b.beta1_t) <= 1e-13 * b.beta1_t, (t, a.beta1_t, b.beta1_t)
            assert abs(a.beta2_t - b.beta2_t) <= 1e-13 * b.beta2_t, (t, a.beta2_t, b.beta2_t)
            # nothing else of the plan moves (Eq. 5-9 keep the base coefficients)
            for name in ("bc1", "bc2", "rho_t", "r_t", "step_size", "rect_branch"):
                assert getattr(a, name) == getattr(r, name), name
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(B.NovakError):
            h.set_option(B.NOVAK_OPT_BETA1_TAU, bad)
    with pytest.raises(B.NovakError):
        h.set_option(B.NOVAK_OPT_ADAPTIVE_BETA, 2)


def test_row_units_cover_every_row_once():
    """The statistics pass's row table: rows of up to 8192 elements whole, in groups of about
    16384 elements; longer rows in consecutive slices of at most 16384 elements; tensors
    without rows left out."""
    shapes = [(8, 27), (33,), (10, 257), (3, 5000), (4097, 2), (1, 7), (5, 1), (2048,), (6, 2048),
              (7, 3000), (2, 12300), (1, 100000), (3, 8192), (2, 8193), (3, 16384), (2, 16385),
              (2, 40000), (300, 127), (300, 128)]
    numel = [int(np.prod(sh)) for sh in shapes]
    rows = [sh[0] if len(sh) > 1 else 0 for sh in shapes]
    units = B.novak_build_row_units(numel, rows)
    seen = [np.zeros((r, numel[i] // r), dtype=np.int32) if r else None for i, r in enumerate(rows)]
    prev = None
    for t, row0, n_rows, part_off, part_len in units:
        L = numel[t] // rows[t]
        assert rows[t] > 0 and n_rows >= 1 and row0 + n_rows <= rows[t]
        if part_len:
            assert L > 8192 and n_rows == 1 and 0 < part_len <= 16384 and part_off % 16384 == 0
            assert part_off + part_len <= L
            if part_off:          # slices of a row are consecutive, in order
                assert prev[:2] == (t, row0) and prev[3] + prev[4] == part_off
            seen[t][row0, part_off:part_off + part_len] += 1
        else:
            assert L <= 8192
            assert n_rows * L <= max(16384, 8 * L) if L >= 128 else n_rows <= 256
            seen[t][row0:row0 + n_rows, :] += 1
        prev = (t, row0, n_rows, part_off, part_len)
    for i, sarr in enumerate(seen):
        if sarr is not None:
            assert (sarr == 1).all(), shapes[i]
    assert {u[0] for u in units} == {i for i, r in enumerate(rows) if r}
    for bad in ([10], [3]), ([10], [-1]), ([0], [0]):
        with pytest.raises(B.NovakError):
            B.novak_build_row_units(*bad)


def test_chunk_builder_covers_every_element_once():
    numel = [1, 31, 32, 33, 8192, 8193, 100_000, 5]
    phase = [0, 3, 31, 0, 7, 0, 16, 30]
    for C in (1024, 8192):
        t, o, ln = B.novak_build_chunks(numel, phase, C)
        seen = [np.zeros(n, dtype=np.int32) for n in numel]
        for ti, oi, li in zip(t, o, ln):
            assert 0 < li <= C
            seen[ti][oi:oi + li] += 1
            # every entry after a tensor's head starts on a 128-byte boundary
            if oi > 0:
                assert (phase[ti] + oi) % 32 == 0
        assert all((s == 1).all() for s in seen)
        # a tensor with phase 0 has no head entry
        assert [li for ti, li in zip(t, ln) if ti == 3] == [33]
        assert [li for ti, li in zip(t, ln) if ti == 1] == [29, 2]
    with pytest.raises(B.NovakError):
        B.novak_build_chunks([0], None, 1024)
    with pytest.raises(B.NovakError):
        B.novak_build_chunks([5], [32], 1024)
