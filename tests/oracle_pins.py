"""Pins for the CPU oracle: facts fixed by the paper and by mathematics.

Every pin is a function ``pin_xxx(lib)`` that raises AssertionError when the
oracle library ``lib`` (a ctypes handle of the compiled C file) violates it.
They are collected in ``ALL_PINS`` so that ``test_oracle_pins.py`` can run
them on the real oracle and ``test_oracle_mutants.py`` on deliberately broken
copies of it (each planted mistake has to trip at least one pin).

None of the pins re-types the oracle's recurrences: they use closed forms
(geometric series), explicit unrolled sums, library routines
(torch.optim.AdamW / RAdam, torch.nn.utils.clip_grad_norm_, tensor.mean, all
in float64), worked examples and invariants (Prop. 6.3-6.5).
"""
from __future__ import annotations

import ctypes
import math

import numpy as np
import torch

from oracle import novak_oracle as O


def _mk(lib, params, **kw):
    return O.Oracle(O.Config(**kw), params, lib=lib)


def _close(a, b, rtol=1e-12, atol=1e-15, what=""):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    err = np.abs(a - b)
    tol = atol + rtol * np.abs(b)
    assert np.all(err <= tol), f"{what}: max err {err.max():.3e} (tol {tol.min():.3e})"


_C = np.array([0.3, -0.02, 1e-4, -7.0, 0.0, 2.5e-3])
_TH0 = np.array([0.05, -0.4, 1.0, 0.0, 0.7, -1e-3])


# --------------------------------------------------------------------------
# Moments and update under a constant gradient (Eq. 1-2, 5, 17, 18, 24)
# --------------------------------------------------------------------------
def pin_constant_grad_none(lib):
    """g == c for all t  =>  m_T = c(1-b1^T), v_T = c^2(1-b2^T), so m_hat = c,
    v_hat = c^2, u = c/(|c|+eps) and, with r_t = 1,
    theta_T = theta_0 d^T - alpha u (1-d^T)/(1-d),  d = 1-alpha*lambda."""
    b1, b2, lr, wd, eps, T = 0.9, 0.999, 1e-3, 1e-2, 1e-8, 37
    o = _mk(lib, [_TH0], lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd,
            nesterov_variant=O.NESTEROV_NONE, lookahead_k=0, rectified=False)
    for _ in range(T):
        o.step([_C])
    _close(o.m[0], _C * (1 - b1 ** T), what="m_T")
    _close(o.v[0], _C ** 2 * (1 - b2 ** T), what="v_T")
    d = 1 - lr * wd
    u = _C / (np.abs(_C) + eps)
    geo = (1 - d ** T) / (1 - d)
    _close(o.theta[0], _TH0 * d ** T - lr * u * geo, rtol=1e-11, what="theta_T")


def pin_constant_grad_approx(lib):
    """Eq. 13 feeding both moments.  With b = b1 - (1-b1) bN:
    m_t = c (1 - b^t),  g~_t = c (1 + bN b^(t-1)),
    v_T = (1-b2) sum_i b2^(T-i) g~_i^2   (explicit sum, no recurrence)."""
    b1, b2, bN, T = 0.9, 0.999, 0.7, 23
    o = _mk(lib, [_TH0], beta1=b1, beta2=b2, nesterov_variant=O.NESTEROV_APPROX,
            nesterov_beta=bN, lookahead_k=0, rectified=False)
    for _ in range(T):
        o.step([_C])
    b = b1 - (1 - b1) * bN
    _close(o.m[0], _C * (1 - b ** T), what="m_T approx")
    gt = [_C * (1 + bN * b ** (i - 1)) for i in range(1, T + 1)]
    v = sum((1 - b2) * b2 ** (T - i) * gt[i - 1] ** 2 for i in range(1, T + 1))
    _close(o.v[0], v, what="v_T approx")


def pin_constant_grad_classical(lib):
    """Eq. 16 literal under constant c: u = b1 c + (1-b1) c/(|c|+eps)."""
    b1, lr, wd, eps, T = 0.8, 2e-3, 0.05, 1e-8, 11
    o = _mk(lib, [_TH0], lr=lr, beta1=b1, eps=eps, weight_decay=wd,
            nesterov_variant=O.NESTEROV_CLASSICAL, lookahead_k=0, rectified=False)
    for _ in range(T):
        o.step([_C])
    d = 1 - lr * wd
    u = b1 * _C + (1 - b1) * _C / (np.abs(_C) + eps)
    _close(o.theta[0], _TH0 * d ** T - lr * u * (1 - d ** T) / (1 - d),
           rtol=1e-11, what="theta_T classical")


# --------------------------------------------------------------------------
# Unrolled-sum brute force with random gradients (no recurrence anywhere)
# --------------------------------------------------------------------------
def _unrolled(th0, G, lr, b1, b2, eps, wd, variant, bN, r):
    """theta_T from explicit sums.  G: (T, n) gradients; r: (T,) step factors."""
    T = G.shape[0]
    if variant == O.NESTEROV_APPROX:
        b = b1 - (1 - b1) * bN
        w = (1 - b1) * (1 + bN)
        M = [sum(w * b ** (t - i) * G[i - 1] for i in range(1, t + 1))
             for t in range(0, T + 1)]                      # M[t] = m_t, M[0] = 0
        Gt = [(1 + bN) * G[t - 1] - bN * M[t - 1] for t in range(1, T + 1)]
    else:
        M = [sum((1 - b1) * b1 ** (t - i) * G[i - 1] for i in range(1, t + 1))
             for t in range(0, T + 1)]
        Gt = [G[t - 1] for t in range(1, T + 1)]
    d = 1 - lr * wd
    total = th0 * d ** T
    us = []
    for t in range(1, T + 1):
        v = sum((1 - b2) * b2 ** (t - i) * Gt[i - 1] ** 2 for i in range(1, t + 1))
        mh = M[t] / (1 - b1 ** t)
        vh = v / (1 - b2 ** t)
        u = mh / (np.sqrt(vh) + eps)
        if variant == O.NESTEROV_CLASSICAL:
            u = b1 * mh + (1 - b1) * u
        us.append(u)
        total = total - d ** (T - t) * lr * r[t - 1] * u
    return total, M[T], us


def pin_unrolled_random(lib):
    rng = np.random.default_rng(7)
    T, n = 14, 9
    G = rng.normal(0, 1e-2, size=(T, n))
    G[3, 2] = 0.0
    th0 = rng.normal(0, 0.05, size=n)
    lr, b1, b2, eps, wd, bN = 3e-3, 0.85, 0.98, 1e-8, 0.02, 0.6
    for variant in (O.NESTEROV_NONE, O.NESTEROV_APPROX, O.NESTEROV_CLASSICAL):
        o = _mk(lib, [th0], lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd,
                nesterov_variant=variant, nesterov_beta=bN, lookahead_k=0,
                rectified=False)
        for t in range(T):
            o.step([G[t]])
        th, mT, _ = _unrolled(th0, G, lr, b1, b2, eps, wd, variant, bN, np.ones(T))
        _close(o.m[0], mT, rtol=1e-11, atol=1e-16, what=f"m unrolled v{variant}")
        _close(o.theta[0], th, rtol=1e-10, atol=1e-14, what=f"theta unrolled v{variant}")


# --------------------------------------------------------------------------
# Library special cases
# --------------------------------------------------------------------------
def pin_adamw_library(lib):
    """rectified off, Nesterov none, no lookahead == torch.optim.AdamW (fp64),
    step for step (same eps placement: sqrt(v_hat)+eps)."""
    g = torch.Generator().manual_seed(11)
    T, n = 25, 33
    th0 = torch.randn(n, generator=g, dtype=torch.float64) * 0.05
    G = torch.randn(T, n, generator=g, dtype=torch.float64) * 1e-2
    lr, b1, b2, eps, wd = 1e-3, 0.9, 0.999, 1e-8, 1e-2
    p = th0.clone().requires_grad_(True)
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd,
                            foreach=False)
    o = _mk(lib, [th0.numpy()], lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd,
            nesterov_variant=O.NESTEROV_NONE, lookahead_k=0, rectified=False)
    for t in range(T):
        p.grad = G[t].clone()
        opt.step()
        o.step([G[t].numpy()])
        _close(o.theta[0], p.detach().numpy(), rtol=1e-12, atol=1e-16,
               what=f"AdamW step {t + 1}")


def pin_radam_library(lib):
    """On rectified steps the per-step change theta_t - d*theta_{t-1} equals
    torch.optim.RAdam's (decoupled decay, fp64) when eps is negligible; this
    fixes r_t (Eq. 6-9), both bias corrections and the decay factor.  The
    earlier steps differ by design (the paper keeps the denominator there)."""
    g = torch.Generator().manual_seed(5)
    T, n = 40, 17
    th0 = torch.randn(n, generator=g, dtype=torch.float64) * 0.05
    G = torch.randn(T, n, generator=g, dtype=torch.float64) * 1e-2
    lr, wd, eps = 1e-3, 1e-2, 1e-30
    for b1, b2 in ((0.9, 0.999), (0.8, 0.99)):
        p = th0.clone().requires_grad_(True)
        opt = torch.optim.RAdam([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd,
                                decoupled_weight_decay=True, foreach=False)
        o = _mk(lib, [th0.numpy()], lr=lr, beta1=b1, beta2=b2, eps=eps,
                weight_decay=wd, nesterov_variant=O.NESTEROV_NONE, lookahead_k=0,
                rectified=True)
        d = 1 - lr * wd
        n_rect = 0
        for t in range(1, T + 1):
            p_prev = p.detach().clone().numpy()
            o_prev = o.theta[0].copy()
            p.grad = G[t - 1].clone()
            opt.step()
            o.step([G[t - 1].numpy()])
            if o.rect_flags[-1]:
                n_rect += 1
                _close(o.theta[0] - d * o_prev, p.detach().numpy() - d * p_prev,
                       rtol=1e-9, atol=1e-18, what=f"RAdam delta t={t} b2={b2}")
        assert n_rect >= T - 6


# --------------------------------------------------------------------------
# Host scalars (Eq. 5-9)
# --------------------------------------------------------------------------
def _scalars(lib, t, **kw):
    o = _mk(lib, [np.zeros(1)], **kw)
    return o.scalars(t)


def pin_scalars(lib):
    # rho_1 == 1 for every beta2: rho_inf - 2 b/(1-b) = (1+b)/(1-b) - 2b/(1-b).
    for b2 in (0.5, 0.9, 0.99, 0.999, 0.9999):
        s = _scalars(lib, 1, beta2=b2)
        assert abs(s.rho_t - 1.0) < 1e-9 * s.rho_inf, (b2, s.rho_t)
        assert abs(s.rho_inf - (1 + b2) / (1 - b2)) < 1e-9 * s.rho_inf
    # beta2 = 0.999: rho_inf = 1999; first rectified step is t = 6.
    flags = [_scalars(lib, t, beta2=0.999).rect_branch for t in range(1, 12)]
    assert flags == [0] * 5 + [1] * 6, flags
    assert abs(_scalars(lib, 1, beta2=0.999).rho_inf - 1999.0) < 1e-9
    # rho_t increases towards rho_inf; r_t in (0,1] and -> 1 (Prop. 6.4).
    prev_rho, prev_r = -1.0, 0.0
    for t in (1, 2, 5, 6, 7, 20, 100, 1000, 10 ** 4, 10 ** 5, 10 ** 6):
        s = _scalars(lib, t, beta2=0.999)
        # strictly increasing until beta2^t underflows against rho_inf
        assert s.rho_t <= s.rho_inf
        assert s.rho_t > prev_rho or (t >= 10 ** 5 and s.rho_t == prev_rho)
        prev_rho = s.rho_t
        if s.rect_branch:
            assert 0.0 < s.r_t <= 1.0
            assert s.r_t > prev_r or (t >= 10 ** 5 and s.r_t == prev_r)
            prev_r = s.r_t
        else:
            assert s.r_t == 1.0
    assert _scalars(lib, 10 ** 6, beta2=0.999).r_t > 0.9999
    # r_t at the threshold rho_t = 5 in closed form: with rho_t -> 5 exactly,
    # r^2 = 3*rho_inf / (5 (rho_inf-4)(rho_inf-2)); r_6 must sit just above it.
    s6 = _scalars(lib, 6, beta2=0.999)
    r5 = math.sqrt(3 * 1999.0 / (5 * 1995.0 * 1997.0))
    assert r5 < s6.r_t < 2 * r5, (s6.r_t, r5)
    # bias corrections against the log form 1 - exp(t log beta) (Section 5.8).
    for t in (1, 3, 10, 1000, 123456):
        s = _scalars(lib, t, beta1=0.9, beta2=0.999)
        assert abs(s.bc1 + math.expm1(t * math.log(0.9))) < 1e-15
        assert abs(s.bc2 + math.expm1(t * math.log(0.999))) < 1e-15
    # rectified = False never takes the first case of Eq. 8.
    assert _scalars(lib, 50, beta2=0.999, rectified=False).rect_branch == 0
    # rho_inf <= 5 (beta2 <= 2/3): never rectified, nothing undefined.
    for t in (1, 10, 1000):
        s = _scalars(lib, t, beta2=0.6)
        assert s.rect_branch == 0 and s.r_t == 1.0
    # decay uses the base rate alpha (Eq. 18), sync flags follow t mod k.
    s = _scalars(lib, 10, lr=0.25, weight_decay=0.5, lookahead_k=5)
    assert s.decay == 1 - 0.125 and s.is_sync == 1
    assert _scalars(lib, 11, lookahead_k=5).is_sync == 0
    assert _scalars(lib, 10, lookahead_k=0).is_sync == 0


def pin_rectified_step_scaling(lib):
    """On a rectified step the change is r_t times the un-rectified one, and
    r_t is the same number the scalar routine reports (Eq. 8 first case)."""
    rng = np.random.default_rng(3)
    th0, G = rng.normal(0, 0.05, 5), rng.normal(0, 1e-2, (9, 5))
    a = _mk(lib, [th0], weight_decay=0.0, lookahead_k=0, rectified=True,
            nesterov_variant=O.NESTEROV_NONE)
    b = _mk(lib, [th0], weight_decay=0.0, lookahead_k=0, rectified=False,
            nesterov_variant=O.NESTEROV_NONE)
    for t in range(1, 10):
        pa, pb = a.theta[0].copy(), b.theta[0].copy()
        a.step([G[t - 1]])
        b.step([G[t - 1]])
        r = a.scalars(t).r_t
        _close(a.theta[0] - pa, r * (b.theta[0] - pb), rtol=1e-9, atol=1e-18,
               what=f"r_t scaling t={t}")
        if t <= 5:
            assert r == 1.0
        else:
            assert r < 0.1


# --------------------------------------------------------------------------
# Decoupled decay (Prop. 6.5) and lookahead (Eq. 28-31, Thm 6.2)
# --------------------------------------------------------------------------
def pin_pure_decay(lib):
    """g == 0: m = v = 0, u = 0/(0+eps) = 0, theta_t = theta_0 (1-alpha*lambda)^t
    for every variant; with LAST lookahead each window maps S to
    S (1 + a (d^k - 1))."""
    lr, wd, T = 0.05, 0.3, 17
    d = 1 - lr * wd
    z = np.zeros_like(_TH0)
    for variant in (0, 1, 2):
        o = _mk(lib, [_TH0], lr=lr, weight_decay=wd, nesterov_variant=variant,
                lookahead_k=0)
        for _ in range(T):
            o.step([z])
        _close(o.theta[0], _TH0 * d ** T, what=f"pure decay v{variant}")
        assert not o.m[0].any() and not o.v[0].any()
    k, a = 5, 0.5
    o = _mk(lib, [_TH0], lr=lr, weight_decay=wd, lookahead_k=k, lookahead_alpha=a)
    for _ in range(T):
        o.step([z])
    w = (1 + a * (d ** k - 1)) ** (T // k)
    _close(o.theta[0], _TH0 * w * d ** (T % k), what="decay with LAST lookahead")
    _close(o.slow[0], _TH0 * w, what="slow after decay windows")
    assert o.sync_steps == [5, 10, 15]


def pin_lookahead_last(lib):
    """After k steps slow <- slow + a (fast - slow), where fast is what k plain
    steps (no lookahead) produce from the same start; moments are untouched;
    the second window starts from the synchronised point."""
    rng = np.random.default_rng(2)
    k, a, n = 4, 0.3, 7
    th0, G = rng.normal(0, 0.05, n), rng.normal(0, 1e-2, (2 * k, n))
    la = _mk(lib, [th0], lookahead_k=k, lookahead_alpha=a)
    pl = _mk(lib, [th0], lookahead_k=0)
    for t in range(k):
        la.step([G[t]])
        pl.step([G[t]])
        if t < k - 1:
            _close(la.theta[0], pl.theta[0], what="fast weights before sync")
            _close(la.slow[0], th0, what="slow untouched before sync")
    want = th0 + a * (pl.theta[0] - th0)
    _close(la.theta[0], want, what="theta at sync")
    _close(la.slow[0], want, what="slow at sync")
    _close(la.m[0], pl.m[0], what="m untouched by sync")
    _close(la.v[0], pl.v[0], what="v untouched by sync")
    # Second window: continue the plain run from the synchronised point.
    pl.theta[0][:] = want
    for t in range(k, 2 * k):
        la.step([G[t]])
        pl.step([G[t]])
    _close(la.theta[0], want + a * (pl.theta[0] - want), what="second sync")
    assert la.sync_steps == [k, 2 * k] and la.t == 2 * k


def pin_lookahead_traj_mean(lib):
    """TRAJ_MEAN: slow <- slow + a (mean of the window's k fast iterates - slow)
    (proof of Thm 6.2); k = 1 coincides with LAST; a constant displacement d per
    step gives slow + a d (k+1)/2."""
    rng = np.random.default_rng(4)
    k, a, n = 5, 0.6, 6
    th0, G = rng.normal(0, 0.05, n), rng.normal(0, 1e-2, (2 * k, n))
    tm = _mk(lib, [th0], lookahead_k=k, lookahead_alpha=a,
             lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN)
    pl = _mk(lib, [th0], lookahead_k=0)
    start = th0.copy()
    for w in range(2):
        its = []
        for t in range(w * k, (w + 1) * k):
            tm.step([G[t]])
            pl.step([G[t]])
            its.append(pl.theta[0].copy())
        want = start + a * (np.mean(its, axis=0) - start)
        _close(tm.theta[0], want, what=f"traj-mean sync {w}")
        _close(tm.slow[0], want, what=f"traj-mean slow {w}")
        assert not tm.acc[0].any()
        pl.theta[0][:] = want
        start = want
    # k = 1
    x = _mk(lib, [th0], lookahead_k=1, lookahead_alpha=a,
            lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN)
    y = _mk(lib, [th0], lookahead_k=1, lookahead_alpha=a)
    for t in range(4):
        x.step([G[t]])
        y.step([G[t]])
    _close(x.theta[0], y.theta[0], what="traj-mean k=1 == last")
    # constant displacement: constant g, no decay, r=1 -> each step moves by
    # dlt = -lr * c/(|c|+eps);  mean of iterates = S + dlt (k+1)/2.
    lr, eps = 1e-2, 1e-8
    o = _mk(lib, [_TH0], lr=lr, eps=eps, weight_decay=0.0, rectified=False,
            nesterov_variant=O.NESTEROV_NONE, lookahead_k=k, lookahead_alpha=a,
            lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN)
    for _ in range(k):
        o.step([_C])
    dlt = -lr * _C / (np.abs(_C) + eps)
    _close(o.theta[0], _TH0 + a * dlt * (k + 1) / 2, rtol=1e-11, what="const displacement")


def pin_bias1_power(lib):
    """bias1_power = 2 divides the step by (1 - beta1^t) once more (Eq. 8 used
    together with Eq. 24); nothing else changes."""
    rng = np.random.default_rng(9)
    th0, G = rng.normal(0, 0.05, 4), rng.normal(0, 1e-2, (8, 4))
    a = _mk(lib, [th0], weight_decay=0.0, lookahead_k=0, bias1_power=1)
    b = _mk(lib, [th0], weight_decay=0.0, lookahead_k=0, bias1_power=2)
    for t in range(1, 9):
        pa, pb = a.theta[0].copy(), b.theta[0].copy()
        a.step([G[t - 1]])
        b.step([G[t - 1]])
        _close((b.theta[0] - pb) * (1 - 0.9 ** t), a.theta[0] - pa, rtol=1e-9,
               atol=1e-18, what=f"bias1_power t={t}")
        _close(a.m[0], b.m[0])


# --------------------------------------------------------------------------
# Invariants (Prop. 6.3) and structure
# --------------------------------------------------------------------------
def pin_moment_bounds(lib):
    """|m_t| <= max_i |g~_i| and v_t <= max_i g~_i^2 element-wise (Prop. 6.3),
    v_t >= 0; g~ = g for variants none/classical."""
    rng = np.random.default_rng(1)
    T, n = 60, 50
    G = rng.normal(0, 1e-2, (T, n)) * rng.integers(0, 2, (T, n))
    for variant in (O.NESTEROV_NONE, O.NESTEROV_CLASSICAL):
        o = _mk(lib, [rng.normal(0, 0.05, n)], nesterov_variant=variant)
        for t in range(T):
            o.step([G[t]])
            gmax = np.abs(G[: t + 1]).max(axis=0)
            assert np.all(np.abs(o.m[0]) <= gmax + 1e-18)
            assert np.all(o.v[0] <= gmax ** 2 + 1e-24) and np.all(o.v[0] >= 0)


def pin_elements_independent(lib):
    """Splitting a tensor, permuting tensors or threading the element ranges
    does not change any element (the step has no cross-element term)."""
    rng = np.random.default_rng(8)
    n, T = 200_000, 7
    th0 = rng.normal(0, 0.05, n)
    G = rng.normal(0, 1e-2, (T, n))
    whole = _mk(lib, [th0], lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN, lookahead_k=3)
    parts = _mk(lib, [th0[:77], th0[77:1000], th0[1000:]],
                lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN, lookahead_k=3)
    thr = _mk(lib, [th0], lookahead_mode=O.LOOKAHEAD_TRAJ_MEAN, lookahead_k=3)
    for t in range(T):
        whole.step([G[t]])
        parts.step([G[t][:77], G[t][77:1000], G[t][1000:]])
        thr.step([G[t]], threads=3)
    assert np.array_equal(np.concatenate(parts.theta), whole.theta[0])
    assert np.array_equal(thr.theta[0], whole.theta[0])
    assert np.array_equal(np.concatenate(parts.slow), whole.slow[0])


# --------------------------------------------------------------------------
# Phase 2: global-norm clipping (Table 2, Section 5.8) and centralization (Eq. 26)
# --------------------------------------------------------------------------
def _prep(lib, grads, rows=None, **kw):
    o = O.Oracle(O.Config(lookahead_k=0, **kw), [np.zeros(g.size) for g in grads], lib=lib,
                 rows=rows)
    out = o.process_gradients([np.asarray(g, np.float64).reshape(-1).copy() for g in grads])
    return o, out


def pin_clip_closed_forms(lib):
    """3-4-5 and constant-vector norms; a clipped gradient has norm exactly c_clip and
    keeps its direction; a gradient inside the ball is returned bit for bit."""
    g = [np.array([3.0, 0.0]), np.array([0.0, -4.0, 0.0])]
    o, out = _prep(lib, g, clip_threshold=1.0)
    _close(o.grad_norms[0], 5.0, what="3-4-5 norm")
    _close(o.clip_factors[0], 0.2, what="3-4-5 factor")
    _close(np.concatenate(out), [0.6, 0.0, 0.0, -0.8, 0.0], what="3-4-5 clipped")
    # n equal entries a: ||g|| = |a| sqrt(n), spread over tensors of different sizes
    a, sizes = -0.37, [7, 1, 92]
    o, out = _prep(lib, [np.full(n, a) for n in sizes], clip_threshold=0.5)
    _close(o.grad_norms[0], abs(a) * math.sqrt(sum(sizes)), what="constant-vector norm")
    flat = np.concatenate(out)
    _close(math.sqrt(math.fsum(flat * flat)), 0.5, what="norm after clipping")
    _close(flat, np.full(sum(sizes), -0.5 / math.sqrt(sum(sizes))), what="direction kept")
    # inside the ball, and exactly on it: untouched
    rng = np.random.default_rng(3)
    g = [rng.normal(0, 1e-3, 50), rng.normal(0, 1e-3, 9)]
    o, out = _prep(lib, g, clip_threshold=1.0)
    assert o.clip_factors[0] == 1.0
    assert all(np.array_equal(x, y) for x, y in zip(out, g))
    o, out = _prep(lib, [np.array([0.6, 0.8])], clip_threshold=1.0)
    assert o.clip_factors[0] == 1.0 or abs(o.clip_factors[0] - 1.0) < 1e-15


def pin_clip_library(lib):
    """torch.nn.utils.clip_grad_norm_ (whose factor is c/(norm + 1e-6), clamped to 1)
    on random multi-tensor gradients: norm identical, gradients equal to ~1e-6."""
    rng = np.random.default_rng(11)
    shapes = [(5, 3), (17,), (2, 3, 2, 2), (1,)]
    g = [rng.normal(0, 2.0, s) for s in shapes]
    ps = [torch.zeros(s, dtype=torch.float64, requires_grad=True) for s in shapes]
    for p, x in zip(ps, g):
        p.grad = torch.tensor(x)
    total = torch.nn.utils.clip_grad_norm_(ps, max_norm=1.5)
    o, out = _prep(lib, g, clip_threshold=1.5)
    _close(o.grad_norms[0], float(total), rtol=1e-13, what="norm vs torch")
    for x, p in zip(out, ps):
        _close(x, p.grad.numpy().reshape(-1), rtol=2e-6, what="clipped vs torch")


def pin_centralize_library_and_invariants(lib):
    """Eq. 26 against torch's g - g.mean(dim=(1..d)); rows sum to zero; applying it
    twice changes nothing; tensors given with rows = 0 (one dimension) are untouched;
    a row of equal entries becomes zero."""
    rng = np.random.default_rng(5)
    shapes = [(4, 3, 2, 2), (6, 5), (7,), (3, 1)]
    g = [rng.normal(0.3, 1.0, s) for s in shapes]
    rows = [4, 6, 0, 3]
    _, out = _prep(lib, g, rows=rows, centralize=True)
    for x, y, s in zip(out, g, shapes):
        t = torch.tensor(y)
        if len(s) > 1:
            want = t - t.mean(dim=tuple(range(1, len(s))), keepdim=True)
        else:
            want = t
        _close(x, want.numpy().reshape(-1), rtol=1e-12, atol=1e-15, what=f"GC {s}")
        if len(s) > 1:
            _close(x.reshape(s[0], -1).sum(axis=1), 0.0, atol=1e-14, what="row sums")
    assert np.array_equal(out[2], g[2].reshape(-1))
    _close(out[3], 0.0, atol=0.0, what="rows of one element")
    _, twice = _prep(lib, out, rows=rows, centralize=True)
    for x, y in zip(twice, out):
        _close(x, y, atol=1e-15, what="idempotent")
    # not the mean over dimension 0 (columns) and not the tensor's overall mean
    gm = np.array([[1.0, 2.0, 6.0], [10.0, 20.0, 30.0]])
    _, out = _prep(lib, [gm], rows=[2], centralize=True)
    _close(out[0], [-2.0, -1.0, 3.0, -10.0, 0.0, 10.0], what="worked 2x3 example")


def pin_clip_then_centralize_then_step(lib):
    """Order inside phase 2 and its hand-over to the moments.  The clip factor comes
    from the RAW norm (a gradient whose centralized norm is below c_clip but whose raw
    norm is above is still scaled); the processed gradient is what Eq. 1-2 see: one
    step from m = v = 0 with no Nesterov term gives m_1 = (1-b1) g', v_1 = (1-b2) g'^2."""
    g = np.array([[10.0, 10.2], [-10.0, -9.8]])          # raw norm ~20, centralized ~0.2
    b1, b2 = 0.9, 0.99
    o = O.Oracle(O.Config(beta1=b1, beta2=b2, nesterov_variant=O.NESTEROV_NONE, lookahead_k=0,
                          clip_threshold=1.0, centralize=True), [np.zeros(4)], lib=lib, rows=[2])
    o.step([g.reshape(-1)])
    raw = math.sqrt(10.0 ** 2 + 10.2 ** 2 + 10.0 ** 2 + 9.8 ** 2)
    gp = (g - g.mean(axis=1, keepdims=True)).reshape(-1) / raw
    _close(o.grad_norms[0], raw, what="raw norm")
    _close(o.m[0], (1 - b1) * gp, rtol=1e-10, what="m_1 from processed gradient")
    _close(o.v[0], (1 - b2) * gp ** 2, rtol=1e-10, what="v_1 from processed gradient")
    # and with the library: clip + centralize by hand, then torch.optim.AdamW
    rng = np.random.default_rng(21)
    th0 = rng.normal(0, 0.1, (3, 4))
    G = rng.normal(0, 1.0, (6, 3, 4))
    p = torch.tensor(th0.copy(), requires_grad=True)
    opt = torch.optim.AdamW([p], lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.1)
    o = O.Oracle(O.Config(lr=1e-2, weight_decay=0.1, nesterov_variant=O.NESTEROV_NONE,
                          lookahead_k=0, rectified=False, clip_threshold=0.7, centralize=True),
                 [th0], lib=lib, rows=[3])
    for t in range(6):
        gt = torch.tensor(G[t])
        n = float(gt.norm())
        gt = gt * (0.7 / n if n > 0.7 else 1.0)
        p.grad = gt - gt.mean(dim=1, keepdim=True)
        opt.step()
        o.step([G[t]])
    # torch's AdamW puts eps before the bias scaling of the root: agree to ~1e-7 relative
    _close(o.theta[0], p.detach().numpy().reshape(-1), rtol=1e-6, what="AdamW after clip + GC")


# --------------------------------------------------------------------------
# Phase 3: adaptive beta (Eq. 3-4)
# --------------------------------------------------------------------------
def pin_adaptive_beta(lib):
    """beta(t) = beta (1 - exp(-t/tau)) in Eq. 1-2 only.  Moments as explicit sums of
    products (no recurrence); the schedule's own values; bias corrections, rho_t, r_t
    and the classical blend unchanged; a vanishing tau gives the constant-beta run."""
    b1, b2, t1, t2, T = 0.9, 0.999, 7.0, 20.0, 25
    rng = np.random.default_rng(13)
    G = rng.normal(0, 1.0, (T, 5))
    th0 = rng.normal(0, 0.1, 5)
    kw = dict(beta1=b1, beta2=b2, lookahead_k=0, nesterov_variant=O.NESTEROV_NONE)
    o = _mk(lib, [th0], adaptive_beta=True, tau1=t1, tau2=t2, **kw)
    ref = _mk(lib, [th0], **kw)
    B1 = [b1 * (1 - math.exp(-t / t1)) for t in range(1, T + 1)]
    B2 = [b2 * (1 - math.exp(-t / t2)) for t in range(1, T + 1)]
    assert B1[0] < 0.15 * b1 and abs(B1[-1] - b1) < 0.03 * b1     # warms up from near 0 to beta
    for t in range(1, T + 1):
        o.step([G[t - 1]])
        ref.step([G[t - 1]])
        s, sr = o.scalars(t), ref.scalars(t)
        _close(s.beta1_t, B1[t - 1], what="beta1(t)")
        _close(s.beta2_t, B2[t - 1], what="beta2(t)")
        for name in ("bc1", "bc2", "rho_inf", "rho_t", "r_t", "step_size", "decay"):
            assert getattr(s, name) == getattr(sr, name), name      # base betas everywhere else
        assert s.rect_branch == sr.rect_branch
    m = sum((1 - B1[i]) * math.prod(B1[i + 1:]) * G[i] for i in range(T))
    v = sum((1 - B2[i]) * math.prod(B2[i + 1:]) * G[i] ** 2 for i in range(T))
    _close(o.m[0], m, rtol=1e-11, what="m_T under Eq. 3")
    _close(o.v[0], v, rtol=1e-11, what="v_T under Eq. 4")
    # half way: beta(tau ln 2) = beta / 2
    h = _mk(lib, [th0], adaptive_beta=True, tau1=10 / math.log(2), tau2=10 / math.log(2), **kw)
    _close(h.scalars(10).beta1_t, b1 / 2, what="beta1 at tau ln 2")
    _close(h.scalars(10).beta2_t, b2 / 2, what="beta2 at tau ln 2")
    # tau -> 0: the schedule is at its limit from the first step on
    z = _mk(lib, [th0], adaptive_beta=True, tau1=1e-3, tau2=1e-3, **kw)
    for t in range(T):
        z.step([G[t]])
    _close(z.theta[0], ref.theta[0], rtol=1e-14, what="tau -> 0 equals constant beta")
    assert not np.allclose(o.theta[0], ref.theta[0], rtol=1e-6)    # and the warm-up matters
    # the classical blend keeps the base beta1: one step from m = v = 0
    c = _mk(lib, [np.zeros(1)], lr=1.0, weight_decay=0.0, eps=1e-8, beta1=b1, beta2=b2,
            lookahead_k=0, nesterov_variant=O.NESTEROV_CLASSICAL, rectified=False,
            adaptive_beta=True, tau1=t1, tau2=t2)
    c.step([np.array([2.0])])
    mh = (1 - B1[0]) * 2.0 / (1 - b1)
    vh = (1 - B2[0]) * 4.0 / (1 - b2)
    _close(c.theta[0], -(b1 * mh + (1 - b1) * mh / (math.sqrt(vh) + 1e-8)), rtol=1e-12,
           what="classical blend with base beta1")


# --------------------------------------------------------------------------
# Phase 7: layer-wise adaptation (Eq. 19 / 25)
# --------------------------------------------------------------------------
def pin_trust_ratio(lib):
    """lambda_trust = clip(||theta_t|| / ||u_t||, 0.1, 10) per tensor, multiplying the
    gradient part of the step only.  u_t is recovered from a run WITHOUT layer adaptation
    (whose step is pinned by the closed forms and library optimizers above), the norms are
    numpy's: the adapted step must be the plain one stretched by that ratio."""
    rng = np.random.default_rng(31)
    lr, wd = 1e-2, 0.1
    kw = dict(lr=lr, weight_decay=wd, lookahead_k=0, nesterov_variant=O.NESTEROV_APPROX)
    th = [rng.normal(0, 0.3, 40), rng.normal(0, 3.0, 7), rng.normal(0, 0.02, 300)]
    d = 1 - lr * wd
    plain = _mk(lib, th, **kw)
    adapt = _mk(lib, th, layer_adaptation=True, **kw)
    for t in range(1, 9):
        G = [rng.normal(0, 1.0, x.size) for x in th]
        # both runs start the step from the adapted run's state
        for i in range(3):
            plain.theta[i][:] = adapt.theta[i]
            plain.m[i][:] = adapt.m[i]
            plain.v[i][:] = adapt.v[i]
        before = [x.copy() for x in adapt.theta]
        plain.t = adapt.t
        plain.step(G)
        adapt.step(G)
        step = plain.scalars(t).step_size
        for i in range(3):
            u = -(plain.theta[i] - before[i] * d) / step              # Eq. 24 solved for u_t
            want = np.linalg.norm(before[i]) / np.linalg.norm(u)
            want = min(max(want, 0.1), 10.0)
            _close(adapt.trust[-1][i], want, rtol=1e-9, what=f"lambda_trust t={t} tensor {i}")
            _close(adapt.theta[i] - before[i] * d, want * (plain.theta[i] - before[i] * d),
                   rtol=1e-9, atol=1e-15, what="only the gradient part is stretched")
            _close(adapt.m[i], plain.m[i], rtol=0, atol=0, what="moments untouched")
    ratios = np.array(adapt.trust)
    assert ratios[:, 0].max() < 10 and ratios[:, 0].min() > 0.1      # tensor 0 unclipped ...
    assert len({round(float(x), 6) for x in ratios[0]}) == 3          # ... and one ratio per tensor
    # closed form at t = 1 (variant none): u = g/(|g|+eps), so ||u|| = sqrt(n) |g|/(|g|+eps)
    n, g0, eps = 16, 0.25, 1e-8
    o = _mk(lib, [np.full(n, 0.5)], layer_adaptation=True, lr=lr, weight_decay=wd, eps=eps,
            lookahead_k=0, nesterov_variant=O.NESTEROV_NONE)
    o.step([np.full(n, -g0)])
    lam = (0.5 * math.sqrt(n)) / (math.sqrt(n) * g0 / (g0 + eps))
    _close(o.trust[0][0], lam, what="closed form lambda")
    _close(o.theta[0], 0.5 * d + lr * lam * g0 / (g0 + eps), what="closed form step")
    # the clip bounds, and theta -> a theta scales the ratio by a inside them
    for scale, want in ((1e-4, 0.1), (1e4, 10.0)):
        o = _mk(lib, [np.full(n, 0.5 * scale)], layer_adaptation=True, lookahead_k=0, **{})
        o.step([np.full(n, g0)])
        assert o.trust[0][0] == want
    a = _mk(lib, [th[0]], layer_adaptation=True, **kw)
    b = _mk(lib, [3.0 * th[0]], layer_adaptation=True, **kw)
    G = rng.normal(0, 1.0, 40)
    a.step([G]); b.step([G])
    _close(b.trust[0][0], 3.0 * a.trust[0][0], what="scale equivariance")
    # the ratio uses the base direction of Eq. 17, not the blended one of Eq. 16
    c = _mk(lib, [th[0]], layer_adaptation=True, **dict(kw, nesterov_variant=O.NESTEROV_CLASSICAL))
    e = _mk(lib, [th[0]], layer_adaptation=True, **dict(kw, nesterov_variant=O.NESTEROV_NONE))
    c.step([G]); e.step([G])
    _close(c.trust[0][0], e.trust[0][0], what="base direction in the ratio")
    # zero gradient from zero moments: u = 0, ratio taken as 1, pure decay
    z = _mk(lib, [th[1]], layer_adaptation=True, **kw)
    z.step([np.zeros(7)])
    assert z.trust[0][0] == 1.0
    _close(z.theta[0], th[1] * d, what="pure decay with u = 0")


# --------------------------------------------------------------------------
# Phase 8: sparse updates (Eq. 27)
# --------------------------------------------------------------------------
def pin_sparse_mask(lib):
    """u <- u 1{|u| > tau}.  At t = 1 from zero moments (variant none) u = g/(|g|+eps), so
    whether an element moves is known in closed form; masked elements only decay; the
    classical blend still adds beta1 m_hat to a masked u; tau = 0 is the plain run."""
    lr, wd, eps, tau = 1e-2, 0.1, 0.5, 0.4
    g = np.array([1.0, 0.5, 0.35, -0.2, -2.0, 1e-3, 0.0])        # u = g/(|g|+0.5)
    u = g / (np.abs(g) + eps)                                    # .667 .5 .412 -.286 -.8 .002 0
    th = np.linspace(-1, 1, g.size)
    d = 1 - lr * wd
    kw = dict(lr=lr, weight_decay=wd, eps=eps, lookahead_k=0, rectified=False)
    o = _mk(lib, [th], sparse_threshold=tau, nesterov_variant=O.NESTEROV_NONE, **kw)
    o.step([g])
    keep = np.abs(u) > tau
    assert keep.tolist() == [True, True, True, False, True, False, False]   # |g| = .35 < tau < |u|
    _close(o.theta[0], th * d - lr * np.where(keep, u, 0.0), what="masked step")
    _close(o.m[0], 0.1 * g, what="moments ignore the mask")
    # |u| == tau exactly is NOT kept (strict inequality): g = 2 eps/3... use tau = 0.5, g = 0.5
    e = _mk(lib, [np.zeros(1)], sparse_threshold=0.5, nesterov_variant=O.NESTEROV_NONE, **kw)
    e.step([np.array([0.5])])
    assert e.theta[0][0] == 0.0
    # classical: Eq. 16 blends the masked u with m_hat
    b1 = 0.9
    c = _mk(lib, [th], sparse_threshold=tau, nesterov_variant=O.NESTEROV_CLASSICAL, **kw)
    c.step([g])
    _close(c.theta[0], th * d - lr * (b1 * g + (1 - b1) * np.where(keep, u, 0.0)),
           what="blend after the mask")
    # tau = 0: off, identical to a run that never heard of the mask
    rng = np.random.default_rng(2)
    a = _mk(lib, [th], sparse_threshold=0.0, **kw)
    b = _mk(lib, [th], **kw)
    for _ in range(5):
        G = rng.normal(0, 1, g.size)
        a.step([G]); b.step([G])
    assert np.array_equal(a.theta[0], b.theta[0])
    # the trust ratio (phase 7) sees the unmasked direction
    t1 = _mk(lib, [th], sparse_threshold=tau, layer_adaptation=True,
             nesterov_variant=O.NESTEROV_NONE, **kw)
    t0 = _mk(lib, [th], layer_adaptation=True, nesterov_variant=O.NESTEROV_NONE, **kw)
    t1.step([g]); t0.step([g])
    assert t1.trust[0][0] == t0.trust[0][0]


def _direction(lib, o, g):
    """novak_oracle_direction for the step the oracle object `o` would take next."""
    u = np.empty_like(g)
    lib.novak_oracle_direction(ctypes.byref(o.h), o.t + 1, g.size, O._dptr(g), O._dptr(o.m[0]),
                               O._dptr(o.v[0]), O._dptr(u))
    return u


def pin_direction(lib):
    """novak_oracle_direction (the base direction of Eq. 17 that the next step would
    produce, used to see how close |u| comes to Eq. 27's threshold) against the step itself,
    which the pins above fix: with no weight decay, rectification off and alpha = 1 the step
    of Eq. 24 moves every parameter by exactly -u, so theta_before - theta_after = u.  Runs
    from non-zero moments, for the plain and the approximation variant and under the warm-up
    of Eq. 3-4; at t = 1 from zero moments u is known in closed form."""
    rng = np.random.default_rng(77)
    n = 64
    for kw in (dict(nesterov_variant=O.NESTEROV_NONE),
               dict(nesterov_variant=O.NESTEROV_APPROX, nesterov_beta=0.7),
               dict(nesterov_variant=O.NESTEROV_APPROX, adaptive_beta=True, tau1=3.0, tau2=11.0),
               dict(nesterov_variant=O.NESTEROV_TRUE, true_steps=2, nesterov_beta=0.6)):
        o = _mk(lib, [rng.normal(0, 0.5, n)], lr=1.0, weight_decay=0.0, rectified=False,
                lookahead_k=0, eps=1e-3, **kw)
        for t in range(1, 7):
            g = rng.normal(0, 1.0, n) * 10.0 ** rng.integers(-4, 1, n)
            m0, v0 = o.m[0].copy(), o.v[0].copy()
            u = _direction(lib, o, g)
            assert np.array_equal(o.m[0], m0) and np.array_equal(o.v[0], v0), "nothing is written"
            before = o.theta[0].copy()
            o.step([g])
            # theta_after = theta_before - u: recover u to the rounding of that subtraction
            _close(u, before - o.theta[0], rtol=1e-9, atol=4e-16 * np.abs(before).max(),
                   what=f"direction against the step, t={t} {kw}")
    # closed forms at t = 1 from zero moments: m_hat = g~, v_hat = g~^2, u = g~/(|g~|+eps)
    g = np.array([0.3, -0.02, 1e-4, -7.0, 0.0, 2.5e-3])
    eps = 1e-2
    o = _mk(lib, [np.zeros(g.size)], eps=eps, nesterov_variant=O.NESTEROV_NONE)
    _close(_direction(lib, o, g), g / (np.abs(g) + eps), what="u_1, variant none")
    bn = 0.5
    o = _mk(lib, [np.zeros(g.size)], eps=eps, nesterov_variant=O.NESTEROV_APPROX, nesterov_beta=bn)
    gt = g * (1 + bn)                                        # Eq. 13 with m_0 = 0
    _close(_direction(lib, o, g), gt / (np.abs(gt) + eps), what="u_1, approximation")
    # eps sits outside the root: with v_hat = g^2 = 1e-12 and eps = 1e-3, u = g/(1e-6+1e-3)
    o = _mk(lib, [np.zeros(1)], eps=1e-3, nesterov_variant=O.NESTEROV_NONE)
    _close(_direction(lib, o, np.array([1e-6])), [1e-6 / (1e-6 + 1e-3)], what="eps outside the root")
    # the classical blend and the mask come after Eq. 17: the base direction ignores both
    a = _mk(lib, [np.zeros(g.size)], eps=eps, nesterov_variant=O.NESTEROV_CLASSICAL,
            sparse_threshold=0.4)
    _close(_direction(lib, a, g), g / (np.abs(g) + eps), what="before blend and mask")


# --------------------------------------------------------------------------
# Phase 7: automatic learning-rate scaling (Eq. 20-22)
# --------------------------------------------------------------------------
def pin_auto_lr(lib):
    """The averages as explicit sums of numpy norms, the clipped ratio, and the adapted
    step as the plain (pinned) step stretched by it; raw-gradient norm even when the
    gradient is clipped afterwards; both clip bounds; one scale for every tensor."""
    rng = np.random.default_rng(41)
    lr, wd, gam = 1e-2, 0.1, 0.1
    kw = dict(lr=lr, weight_decay=wd, lookahead_k=0, nesterov_variant=O.NESTEROV_APPROX)
    th = [rng.normal(0, 0.3, 40), rng.normal(0, 0.5, 7)]
    d = 1 - lr * wd
    plain = _mk(lib, th, **kw)
    auto = _mk(lib, th, auto_lr=True, clip_threshold=0.5, **kw)
    plain.cfg.clip_threshold = 0.5
    gn, pn = [], []
    for t in range(1, 8):
        G = [rng.normal(0, 0.1 * t, x.size) for x in th]
        for i in range(2):
            plain.theta[i][:] = auto.theta[i]
            plain.m[i][:] = auto.m[i]
            plain.v[i][:] = auto.v[i]
        before = [x.copy() for x in auto.theta]
        plain.t = auto.t
        gn.append(np.linalg.norm(np.concatenate(G)))
        pn.append(np.linalg.norm(np.concatenate(before)))
        plain.step(G)
        auto.step(G)
        g_bar = sum(gam * (1 - gam) ** (t - i) * gn[i - 1] for i in range(1, t + 1))
        p_bar = sum(gam * (1 - gam) ** (t - i) * pn[i - 1] for i in range(1, t + 1))
        want = min(max(g_bar / p_bar, 0.1), 2.0)
        _close(auto.g_bar.value, g_bar, what="Eq. 20")
        _close(auto.theta_bar.value, p_bar, what="Eq. 21")
        _close(auto.auto_scales[-1], want, what="Eq. 22")
        for i in range(2):
            _close(auto.theta[i] - before[i] * d, want * (plain.theta[i] - before[i] * d),
                   rtol=1e-9, atol=1e-15, what="step stretched by alpha_auto")
    seen = np.array(auto.auto_scales)
    assert seen.min() > 0.1 and seen.max() < 2.0 and seen.max() > 1.5 * seen.min()
    assert max(gn) > 0.5                       # the clipping was active: raw norm in Eq. 20
    for scale, want in ((1e-3, 0.1), (1e3, 2.0)):
        o = _mk(lib, [np.ones(10)], auto_lr=True, **kw)
        o.step([np.full(10, scale)])
        assert o.auto_scales[0] == want
    # with layer adaptation both factors multiply the step (Eq. 24a)
    both = _mk(lib, th, auto_lr=True, layer_adaptation=True, **kw)
    only = _mk(lib, th, layer_adaptation=True, **kw)
    G = [rng.normal(0, 0.3, x.size) for x in th]
    both.step(G); only.step(G)
    for i in range(2):
        _close(both.theta[i] - th[i] * d, both.auto_scales[0] * (only.theta[i] - th[i] * d),
               rtol=1e-9, atol=1e-15, what="alpha_auto times lambda_trust")


# --------------------------------------------------------------------------
# True Nesterov (Eq. 10-12, Section 5.8) and its fallback (Section 5.2)
# --------------------------------------------------------------------------
def pin_true_nesterov(lib):
    """Eq. 10 in closed form (hand values; after one step from zero moments), the
    closed loop on a quadratic against a scalar loop written here, the switch to
    Eq. 13 after exactly N_taylor steps, and that looking ahead moves nothing."""
    lr, b1, b2, eps, wd, bN = 1e-2, 0.9, 0.999, 0.5, 0.1, 0.8
    kw = dict(lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd, lookahead_k=0,
              rectified=False, nesterov_beta=bN)
    # hand values of theta + beta_N m
    out = np.empty(3)
    th = np.array([1.0, -2.0, 0.5]); m = np.array([0.5, 0.25, -1.0])   # named: _dptr keeps no reference
    lib.novak_oracle_extrapolate(bN, 3, O._dptr(th), O._dptr(m), O._dptr(out))
    _close(out, np.array([1.4, -1.8, -0.3]), what="Eq. 10 by hand")
    # after one step from zero moments: theta_1 = theta_0 d - lr g/(|g|+eps), m_1 = (1-b1) g
    g = np.array([1.0, -0.25, 2.0])
    o = _mk(lib, [th], nesterov_variant=O.NESTEROV_TRUE, true_steps=5, **kw)
    assert o.wants_extrapolation()
    _close(o.extrapolated()[0], th, what="m_0 = 0: the first look-ahead is the identity")
    o.step([g])
    before = o.theta[0].copy()
    _close(o.extrapolated()[0],
           th * (1 - lr * wd) - lr * g / (np.abs(g) + eps) + bN * (1 - b1) * g,
           what="Eq. 10 at t = 2 (beta_N, not beta1)")
    assert np.array_equal(o.theta[0], before), "looking ahead must not move theta"
    # closed loop on L = a theta^2 / 2: g~ = a (theta + beta_N m), Adam with no correction
    a, T = 3.0, 12
    q = _mk(lib, [np.array([0.7])], nesterov_variant=O.NESTEROV_TRUE, true_steps=T, **kw)
    x, mm, vv = 0.7, 0.0, 0.0
    for t in range(1, T + 1):
        q.step([a * q.extrapolated()[0]])
        gt = a * (x + bN * mm)
        mm = b1 * mm + (1 - b1) * gt
        vv = b2 * vv + (1 - b2) * gt * gt
        x = x * (1 - lr * wd) - lr * (mm / (1 - b1 ** t)) / (np.sqrt(vv / (1 - b2 ** t)) + eps)
        _close(q.theta[0], np.array([x]), rtol=1e-11, what=f"quadratic, step {t}")
    # N_taylor = 0: the approximation from the first step, bit for bit
    rng = np.random.default_rng(7)
    G = [rng.normal(0, 1, 5) for _ in range(8)]
    th5 = rng.normal(0, 1, 5)
    z = _mk(lib, [th5], nesterov_variant=O.NESTEROV_TRUE, true_steps=0, **kw)
    ap = _mk(lib, [th5], nesterov_variant=O.NESTEROV_APPROX, **kw)
    for gg in G:
        assert not z.wants_extrapolation()
        z.step([gg]); ap.step([gg])
    assert np.array_equal(z.theta[0], ap.theta[0])
    # N_taylor = 3: steps 1-3 as variant none, steps 4-8 as the approximation on that state
    N = 3
    tr = _mk(lib, [th5], nesterov_variant=O.NESTEROV_TRUE, true_steps=N, **kw)
    no = _mk(lib, [th5], nesterov_variant=O.NESTEROV_NONE, **kw)
    wants = []
    for t, gg in enumerate(G, start=1):
        wants.append(tr.wants_extrapolation())
        tr.step([gg])
        if t <= N:
            no.step([gg])
            assert np.array_equal(tr.theta[0], no.theta[0]), f"step {t}: no correction yet"
        if t == N:
            ap = _mk(lib, [no.theta[0]], nesterov_variant=O.NESTEROV_APPROX, **kw)
            ap.m[0][:] = no.m[0]; ap.v[0][:] = no.v[0]; ap.t = N
        if t > N:
            ap.step([gg])
            assert np.array_equal(tr.theta[0], ap.theta[0]), f"step {t}: Eq. 13 from N+1 on"
    assert wants == [t <= N for t in range(1, len(G) + 1)]
    assert not np.array_equal(tr.theta[0], z.theta[0])


# --------------------------------------------------------------------------
# Moments stored in bfloat16 (Section 10)
# --------------------------------------------------------------------------
def pin_bf16_moment_storage(lib):
    """The rounding against torch's fp32 -> bfloat16 conversion (random values, exact
    ties, subnormals, overflow); the stored moments are the roundings of what the plain
    step computes; the step itself uses the unrounded values; a second moment that
    cannot move under round-to-nearest (beta2 = 0.999 changes v by less than half a
    step of its 8-bit grid) stays put."""
    rnd = lambda a: np.array([lib.novak_oracle_round_bf16(float(x)) for x in a])
    rng = np.random.default_rng(11)
    x = (rng.normal(0, 1, 4000) * 10.0 ** rng.uniform(-30, 30, 4000)).astype(np.float32)
    ties = (1.0 + np.arange(0, 64) * 2.0 ** -8).astype(np.float32)          # odd multiples: ties
    sub = (np.arange(1, 300) * 2.0 ** -140).astype(np.float32)             # below 2^-126
    big = np.array([3.38e38, 3.39e38, 3.4e38, -3.4e38, 2.0 ** 127, 1.5 * 2.0 ** 127], np.float32)
    for arr in (x, ties, -ties, sub, -sub, big, np.array([0.0, -0.0], np.float32)):
        want = torch.from_numpy(arr).to(torch.bfloat16).to(torch.float64).numpy()
        got = rnd(arr.astype(np.float64))
        assert np.array_equal(got, want), "round_bf16 differs from torch"
    assert rnd([1.0 + 2.0 ** -8])[0] == 1.0 and rnd([1.0 + 3 * 2.0 ** -8])[0] == 1.0 + 2.0 ** -6
    assert rnd([1.0 + 2.0 ** -8 + 2.0 ** -40])[0] == 1.0 + 2.0 ** -7      # just above a tie
    # one step from a bf16-representable state: same theta as the plain step (the update
    # sees the unrounded moments), stored moments = roundings of the plain step's moments
    kw = dict(lr=1e-2, weight_decay=0.1, eps=1e-3, lookahead_k=0, rectified=False)
    th = rng.normal(0, 1, 64)
    g1, g2 = rng.normal(0, 1, 64), rng.normal(0, 1, 64)
    a = _mk(lib, [th], moment_bf16=True, **kw)
    b = _mk(lib, [th], **kw)
    a.step([g1]); b.step([g1])
    assert np.array_equal(a.theta[0], b.theta[0])
    assert np.array_equal(a.m[0], rnd(b.m[0])) and np.array_equal(a.v[0], rnd(b.v[0]))
    assert not np.array_equal(a.m[0], b.m[0])
    # second step: reads the ROUNDED moments back (a plain run started from them agrees)
    c = _mk(lib, [a.theta[0]], **kw)
    c.m[0][:] = a.m[0]; c.v[0][:] = a.v[0]; c.t = 1
    a.step([g2]); c.step([g2])
    assert np.array_equal(a.theta[0], c.theta[0])
    assert np.array_equal(a.m[0], rnd(c.m[0])) and np.array_equal(a.v[0], rnd(c.v[0]))
    assert not np.array_equal(a.theta[0], _two_plain_steps(lib, th, g1, g2, kw))
    # every stored value has at most 8 significant bits and lies within half a grid step
    for arr, ref in ((a.m[0], c.m[0]), (a.v[0], c.v[0])):
        mant, _ = np.frexp(arr)
        assert np.array_equal(mant * 256, np.round(mant * 256))
        assert np.all(np.abs(arr - ref) <= np.abs(ref) * 2.0 ** -8)
    # stagnation: v = 1, g = 0: 0.999 rounds back to 1 (grid step 2^-8 below 1), m decays
    z = _mk(lib, [np.ones(1)], moment_bf16=True, nesterov_variant=O.NESTEROV_NONE, **kw)
    z.v[0][:] = 1.0; z.m[0][:] = 1.0
    for _ in range(10):
        z.step([np.zeros(1)])
    assert z.v[0][0] == 1.0
    mm = 1.0
    for _ in range(10):
        mm = lib.novak_oracle_round_bf16(0.9 * mm)
    assert z.m[0][0] == mm and 0.3 < mm < 0.4
    # the margin helper: distance to the nearest midpoint over the sum of the terms
    mg = np.empty(1)
    hp = O.Config(moment_bf16=True, nesterov_variant=O.NESTEROV_NONE, beta1=0.5, beta2=0.5).to_c()
    # m_new = 0.5*1 + 0.5*(1 + 2^-6) = 1 + 2^-7: on the grid, 2^-8 from both midpoints
    # v_new = 0.5*v + 0.5*g^2 with v chosen so that v_new = 1 + 2^-8 (a midpoint) -> margin 0
    gq = 1.0 + 2.0 ** -6
    vq = 2.0 * (1.0 + 2.0 ** -8) - gq * gq
    ga, ma, va, vb = np.array([gq]), np.array([1.0]), np.array([vq]), np.array([gq * gq])
    lib.novak_oracle_rounding_margin(ctypes.byref(hp), 1, 1, O._dptr(ga), O._dptr(ma), O._dptr(va),
                                     O._dptr(mg))
    assert mg[0] == 0.0
    lib.novak_oracle_rounding_margin(ctypes.byref(hp), 1, 1, O._dptr(ga), O._dptr(ma), O._dptr(vb),
                                     O._dptr(mg))
    # m_new = 1 + 2^-7 sits 2^-8 from its midpoints; v_new = gq^2 = 1 + 2^-5 + 2^-12 sits
    # 2^-8 - 2^-12 from one: the smaller ratio is reported
    _close(mg, np.array([min(2.0 ** -8 / (1.0 + 2.0 ** -7), (2.0 ** -8 - 2.0 ** -12) / (gq * gq))]),
           what="margin at step 1")
    assert (2.0 ** -8 - 2.0 ** -12) / (gq * gq) < 2.0 ** -8 / (1.0 + 2.0 ** -7)


def _two_plain_steps(lib, th, g1, g2, kw):
    o = _mk(lib, [th], **kw)
    o.step([g1]); o.step([g2])
    return o.theta[0]


# --------------------------------------------------------------------------
# Everything at once against 40-digit arithmetic
# --------------------------------------------------------------------------
def pin_high_precision_all_variants(lib):
    """Every Nesterov variant x lookahead mode x rectification on/off, 30 steps on 12
    elements, against a reference in 40-digit arithmetic (mpmath) that forms the moments
    as explicit sums over the gradient history and the step scalars from Eq. 5-9 as
    printed.  Agreement to 1e-11 also bounds the oracle's own rounding (the
    cancellation in rho_t, the long powers)."""
    import mpmath as mp
    mp.mp.dps = 40
    rng = np.random.default_rng(23)
    T, n = 30, 12
    G = rng.normal(0, 1e-2, size=(T, n)); G[4, 1] = 0.0
    th0 = rng.normal(0, 0.05, size=n)
    lr, b1, b2, eps, wd, bN, aLA = 2e-3, 0.9, 0.999, 1e-8, 0.03, 0.7, 0.4
    F = mp.mpf
    for variant in (O.NESTEROV_NONE, O.NESTEROV_APPROX, O.NESTEROV_CLASSICAL):
        for k, mode in ((0, O.LOOKAHEAD_LAST), (4, O.LOOKAHEAD_LAST), (4, O.LOOKAHEAD_TRAJ_MEAN),
                        (1, O.LOOKAHEAD_TRAJ_MEAN)):
            for rect in (True, False):
                o = _mk(lib, [th0], lr=lr, beta1=b1, beta2=b2, eps=eps, weight_decay=wd,
                        nesterov_variant=variant, nesterov_beta=bN, lookahead_k=k,
                        lookahead_alpha=aLA, lookahead_mode=mode, rectified=rect)
                for t in range(T):
                    o.step([G[t]])
                for e in range(n):
                    g = [F(float(G[t, e])) for t in range(T)]
                    theta = F(float(th0[e])); slow = theta; acc = F(0)
                    gt = []                      # the gradients the moments see
                    for t in range(1, T + 1):
                        m_prev = sum((1 - F(b1)) * F(b1) ** (t - 1 - i) * gt[i - 1]
                                     for i in range(1, t)) if t > 1 else F(0)
                        cur = g[t - 1]
                        if variant == O.NESTEROV_APPROX:
                            cur = cur + F(bN) * (cur - m_prev)
                        gt.append(cur)
                        m = sum((1 - F(b1)) * F(b1) ** (t - i) * gt[i - 1] for i in range(1, t + 1))
                        v = sum((1 - F(b2)) * F(b2) ** (t - i) * gt[i - 1] ** 2 for i in range(1, t + 1))
                        mh = m / (1 - F(b1) ** t); vh = v / (1 - F(b2) ** t)
                        u = mh / (mp.sqrt(vh) + F(eps))
                        if variant == O.NESTEROV_CLASSICAL:
                            u = F(b1) * mh + (1 - F(b1)) * u
                        rho_inf = 2 / (1 - F(b2)) - 1
                        rho = rho_inf - 2 * t * F(b2) ** t / (1 - F(b2) ** t)
                        r = F(1)
                        if rect and rho >= 5:
                            r = mp.sqrt((rho - 4) * (rho - 2) * rho_inf / ((rho_inf - 4) * (rho_inf - 2) * rho))
                        fast = theta * (1 - F(lr) * F(wd)) - F(lr) * r * u
                        theta = fast
                        if k > 0:
                            acc += fast
                            if t % k == 0:
                                target = acc / k if mode == O.LOOKAHEAD_TRAJ_MEAN else fast
                                theta = slow + F(aLA) * (target - slow)
                                slow = theta
                                acc = F(0)
                    ref = float(theta)
                    assert abs(o.theta[0][e] - ref) <= 1e-11 * abs(ref) + 1e-15, \
                        (variant, k, mode, rect, e, o.theta[0][e], ref)


ALL_PINS = [
    pin_constant_grad_none,
    pin_constant_grad_approx,
    pin_constant_grad_classical,
    pin_unrolled_random,
    pin_adamw_library,
    pin_radam_library,
    pin_scalars,
    pin_rectified_step_scaling,
    pin_pure_decay,
    pin_lookahead_last,
    pin_lookahead_traj_mean,
    pin_bias1_power,
    pin_moment_bounds,
    pin_elements_independent,
    pin_clip_closed_forms,
    pin_clip_library,
    pin_centralize_library_and_invariants,
    pin_clip_then_centralize_then_step,
    pin_adaptive_beta,
    pin_trust_ratio,
    pin_sparse_mask,
    pin_direction,
    pin_auto_lr,
    pin_true_nesterov,
    pin_bf16_moment_storage,
    pin_high_precision_all_variants,
]
