// The per-step scalar plan (Eq. 3-9, 18 and the lookahead action of Eq. 28-31)
// as code that runs on the host and on the device alike: novak_step computes
// it on the host in double and passes the result by value; the graph-capturable
// step computes the same thing in a one-thread kernel from a step counter that
// lives in device memory.  Private to the library.
#pragma once

#include "novak.h"
#include "novak_step_types.h"

#include <math.h>
#include <stdint.h>

#ifdef __CUDACC__
#define NOVAK_HD __host__ __device__
#else
#define NOVAK_HD
#endif

namespace novak_host {

struct Hyper {
    double lr, beta1, beta2, eps, wd, beta_n, la_alpha;
    double clip;            // c_clip of the global-norm clipping, 0: off
    int nesterov, la_k, la_mode, rectified, bias1_power;
    int centralize;         // Eq. 26 on tensors that were given rows
    int layer_adapt;        // Eq. 19 / 25: one trust ratio per tensor
    int adaptive_beta;      // Eq. 3-4
    double tau1, tau2;      // warm-up time scales of beta1, beta2
    double sparse_tau;      // tau of Eq. 27, 0: no mask
    int auto_lr;            // Eq. 20-22
    double auto_gamma;      // gamma of Eq. 20-21
    int true_requested;     // the caller asked for the true variant (Eq. 10-12)
    int true_steps;         // N_taylor: steps 1..N_taylor take Eq. 11's gradient as given
    int mom16;              // m and v stored as bf16 (fixed at attach: it sets the layout)
};

struct Plan {
    double bc1, bc2, rho_inf, rho_t, r_t, step_size, decay;
    double beta1_t, beta2_t;   // coefficients of Eq. 1-2 at this step (Eq. 3-4 when warmed up)
    int rect_branch, is_sync;
    int nesterov;              // variant of this step: TRUE while t <= N_taylor, else the configured one
};

// Eq. 5-9 and 18 for the 1-based step index t.  1 - beta^t is evaluated as
// -expm1(t log beta) for every t (Section 5.8 gives the log form for large t).
NOVAK_HD inline Plan make_plan(const Hyper &h, int64_t t)
{
    Plan p;
    const double td = static_cast<double>(t);
    const double l1 = h.beta1 > 0.0 ? td * log(h.beta1) : -INFINITY;
    const double l2 = h.beta2 > 0.0 ? td * log(h.beta2) : -INFINITY;
    p.bc1 = -expm1(l1);
    p.bc2 = -expm1(l2);
    const double b2t = exp(l2);
    p.rho_inf = 2.0 / (1.0 - h.beta2) - 1.0;
    p.rho_t = p.rho_inf - 2.0 * td * b2t / p.bc2;
    p.rect_branch = (h.rectified && p.rho_t >= 5.0) ? 1 : 0;
    p.r_t = 1.0;
    if (p.rect_branch) {
        const double a = (p.rho_t - 4.0) / (p.rho_inf - 4.0);
        const double b = (p.rho_t - 2.0) / (p.rho_inf - 2.0);
        p.r_t = sqrt(a * b * (p.rho_inf / p.rho_t));
    }
    p.step_size = h.lr * p.r_t;
    if (h.bias1_power == 2) p.step_size /= p.bc1;
    p.decay = 1.0 - h.lr * h.wd;
    p.is_sync = (h.la_k > 0 && t % h.la_k == 0) ? 1 : 0;
    // Phase 3, Eq. 3-4: only the moment updates see the warmed-up coefficients.
    p.beta1_t = h.beta1;
    p.beta2_t = h.beta2;
    if (h.adaptive_beta) {
        p.beta1_t = h.beta1 * -expm1(-td / h.tau1);
        p.beta2_t = h.beta2 * -expm1(-td / h.tau2);
    }
    // Section 5.2: the true variant (the gradient is already Eq. 11's) for the
    // first N_taylor steps, the approximation of Eq. 13 afterwards.
    p.nesterov = (h.true_requested && t <= h.true_steps) ? NOVAK_NESTEROV_TRUE : h.nesterov;
    return p;
}

NOVAK_HD inline int lookahead_action(const Hyper &h, int64_t t)
{
    using namespace novak;
    if (h.la_k <= 0) return LA_NONE;
    const bool first_step = (t == 1);
    const bool sync = (t % h.la_k == 0);
    const bool first_of_window = ((t - 1) % h.la_k == 0);
    const bool traj = (h.la_mode == NOVAK_LOOKAHEAD_TRAJ_MEAN && h.la_k > 1);
    int la = 0;
    if (first_step) la |= LA_S_INIT | LA_S_WRITE;
    if (sync) {
        la |= LA_SYNC | LA_S_WRITE;
        if (!first_step) la |= LA_S_READ;
    }
    if (traj) {
        if (!first_of_window) la |= LA_A_READ;
        if (sync) la |= LA_TRAJ; else la |= LA_A_WRITE;
    }
    return la;
}

// The plan rounded once to what the kernels take (Section 8.1).
NOVAK_HD inline novak::StepScalars make_scalars(const Hyper &h, const Plan &p)
{
    novak::StepScalars s;
    s.beta1 = static_cast<float>(p.beta1_t);
    s.omb1 = static_cast<float>(1.0 - p.beta1_t);
    s.beta2 = static_cast<float>(p.beta2_t);
    s.omb2 = static_cast<float>(1.0 - p.beta2_t);
    s.blend_b1 = static_cast<float>(h.beta1);
    s.blend_omb1 = static_cast<float>(1.0 - h.beta1);
    s.beta_n = static_cast<float>(h.beta_n);
    s.inv_bc1 = static_cast<float>(1.0 / p.bc1);
    s.inv_bc2 = static_cast<float>(1.0 / p.bc2);
    s.eps = static_cast<float>(h.eps);
    s.decay = static_cast<float>(p.decay);
    s.step = static_cast<float>(p.step_size);
    s.la_alpha = static_cast<float>(h.la_alpha);
    s.k = static_cast<float>(h.la_k > 0 ? h.la_k : 1);
    s.sparse_tau = h.sparse_tau > 0.0 ? static_cast<float>(h.sparse_tau) : -1.0f;
    return s;
}

}  // namespace novak_host
