/*
 * NOVAK per-parameter optimizer step -- CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the definition the CUDA library is
 * checked against.  It is plain scalar C in double precision, one element at a
 * time, in the order the paper gives its phases (Section 5.1: Nesterov
 * approximation -> moments -> bias correction -> rectification -> direction
 * -> decoupled decay and update -> lookahead).  It shares no code, header,
 * table or constant with the CUDA library and is never called by it; only the
 * tests, the smoke check and the benchmark's CPU-baseline leg load it.
 *
 * Readings taken where the paper is ambiguous (each is also listed in the
 * design notes of the repository):
 *   - The first-moment bias correction is applied once: the parameter change
 *     is  -alpha * r_t * m_hat / (sqrt(v_hat) + eps)  (Eq. 24 with Eq. 24a).
 *     bias1_power = 2 reproduces the literal pairing of Eq. 8 with Eq. 24
 *     (1/(1-beta1^t) applied twice).                      [parity unpinned]
 *   - Eq. 13's g~ replaces g in BOTH moment updates (Table 2 lists it under
 *     gradient processing; the proof of Thm 6.1 writes g_t <- g_t + ...).
 *   - Eq. 16 is taken literally: beta1*m_hat + (1-beta1)*u.   [parity unpinned]
 *   - The branch of Eq. 8 is "rho_t >= 5"; the other branch keeps the
 *     adaptive denominator and sets r_t = 1.
 *   - Lookahead has two modes.  LAST: slow += alpha_LA*(fast - slow) on steps
 *     with t mod k == 0.  TRAJ_MEAN: the rule in the proof of Thm 6.2,
 *     slow += alpha_LA*(mean of the k fast iterates of the window - slow).
 *     Which of the two is "the" method is a reading.          [parity unpinned]
 *   - Moments are not touched by a synchronisation.
 *   - Phase 2 (gradient processing) runs clipping first, on the norm of the
 *     raw gradient (Section 7.3: before any other processing), then
 *     centralization, then the Nesterov approximation.  Table 2 lists
 *     centralization above clipping; the two steps are linear and commute, so
 *     the only difference is which norm is compared with c_clip.
 *     Clipping scales by c_clip/||g|| when ||g|| > c_clip (Table 2's activation
 *     condition), with no epsilon in the denominator.
 *   - Adaptive beta (Eq. 3-4): beta1(t), beta2(t) replace beta1, beta2 in the
 *     moment updates (Eq. 1-2) only.  The bias corrections (Eq. 5), rho_inf
 *     (set once at initialisation in Algorithm 1), rho_t, r_t and the classical
 *     blend (Eq. 16) keep the base values, as those equations are written.
 *                                                              [parity unpinned]
 *   - Layer-wise adaptation (Eq. 19, 25): one trust ratio per tensor,
 *     clip(||theta_t||_2 / ||u_t||_2, 0.1, 10), theta_t the parameters before
 *     the step, u_t the base direction of Eq. 17 (before the classical blend),
 *     multiplying the step size of Eq. 24a; where ||u_t|| = 0 the ratio is
 *     undefined and taken as 1 (the update is zero there anyway).
 *   - Sparse updates (Eq. 27): u <- u * 1{|u| > tau} on the base direction of
 *     Eq. 17, before the classical blend (the order of Table 2, phase 8); the
 *     trust ratio (phase 7) sees the unmasked direction.  tau = 0 switches the
 *     mask off (Table 2: active when sparse_threshold > 0).
 *   - Automatic learning-rate scaling: Eq. 20-22 (two moving averages of the
 *     global norms of gradient and parameters, gamma = 0.1, ratio clipped to
 *     [0.1, 2]), the form Tables 2 and 3 describe (two norm computations, two
 *     scalars of state).  Eq. 23, which Eq. 24a cites, is a different and
 *     incompatible definition (one average, a pole at EMA = 1/e) and is not
 *     used.  ||g_t|| is the norm of the gradient as given (the norm clipping
 *     uses), ||theta_t|| that of the parameters before the step, both over
 *     every tensor of the group; the averages start at 0.   [parity unpinned]
 *
 *   - True Nesterov (Eq. 10-12, Section 5.8): the caller saves theta_{t-1},
 *     sets the model to theta~ = theta_{t-1} + beta_N m_{t-1} (Eq. 10), obtains
 *     g~ there (Eq. 11), restores theta_{t-1}, and g~ then stands where g_t
 *     stands in every later phase: both moments, the direction and the update
 *     (Section 5.8, point 5).  Eq. 12 prints only g~ over a v~ it does not
 *     define and leaves m_t open; it is read as shorthand for that.  While
 *     t <= N_taylor the step applies no Eq. 13 correction to g~; from step
 *     N_taylor + 1 on the variant is the approximation of Eq. 13 (Section 5.2's
 *     automatic fallback).                                 [parity unpinned]
 *
 *   - Moments stored in bfloat16 (Section 10 names bfloat16 storage of the
 *     moments, with the arithmetic kept in float32, as future work): m_{t-1}
 *     and v_{t-1} are read back as stored, the step's own arithmetic (Eq. 1-2,
 *     5, 17) runs on the unrounded m_t, v_t, and what is stored for the next
 *     step is each of them rounded to the nearest bfloat16 (8 significant
 *     bits, fp32's exponent range, ties to even).  The paper fixes neither the
 *     rounding nor whether the step sees rounded values.   [parity unpinned]
 *
 * Pinned by tests/test_oracle_pins.py (closed forms, torch.optim.AdamW/RAdam
 * special cases, unrolled-sum brute force, invariants of Prop. 6.3-6.5); every
 * function of this file has a pin, novak_oracle_direction included (against the
 * pinned step: with alpha = 1, no decay and no rectification the step moves
 * every parameter by exactly -u).
 */
#include <math.h>
#include <stdint.h>

typedef struct {
    double lr;               /* alpha  > 0                                  */
    double beta1;            /* [0,1)                                       */
    double beta2;            /* [0,1)                                       */
    double eps;              /* > 0                                         */
    double weight_decay;     /* lambda >= 0                                 */
    double nesterov_beta;    /* beta_N in [0,1)                             */
    double lookahead_alpha;  /* alpha_LA in (0,1), used when lookahead_k>0  */
    int32_t nesterov_variant;/* 0 none, 1 approximation (Eq.13), 2 classical (Eq.16),
                                3 true (Eq. 10-12) for the first true_steps steps   */
    int32_t lookahead_k;     /* 0 = lookahead off                           */
    int32_t lookahead_mode;  /* 0 LAST, 1 TRAJ_MEAN                         */
    int32_t rectified;       /* 1: Eq. 8-9, 0: r_t = 1 on every step        */
    int32_t bias1_power;     /* 1 (default reading) or 2                    */
    int32_t adaptive_beta;   /* 1: Eq. 3-4 warm-up of beta1, beta2 in Eq. 1-2 */
    double tau1;             /* warm-up time scale of beta1 (paper: 1000)   */
    double tau2;             /* warm-up time scale of beta2 (paper: 5000)   */
    double sparse_threshold; /* tau of Eq. 27; 0 = no mask                  */
    int32_t true_steps;      /* N_taylor: steps 1..N_taylor of variant 3 take g~ */
    int32_t moment_bf16;     /* 1: m and v are stored rounded to bfloat16        */
} novak_oracle_hparams;

/* Nearest bfloat16 to x, ties to even: 1 sign bit, 8 exponent bits (fp32's
 * range: normal numbers from 2^-126, subnormals in steps of 2^-133, overflow
 * to infinity) and 8 significant bits (7 stored). */
double novak_oracle_round_bf16(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x))
        return x;
    int e;
    (void)frexp(x, &e);              /* |x| = f 2^e with f in [0.5, 1) */
    int q = e - 8;                   /* quantum 2^q leaves 8 significant bits */
    if (q < -133)
        q = -133;                    /* subnormal range: fixed quantum */
    const double r = ldexp(rint(ldexp(x, -q)), q);   /* rint: to nearest, ties to even */
    if (fabs(r) >= ldexp(1.0, 128))
        return x > 0.0 ? INFINITY : -INFINITY;
    return r;
}

/* Whether step t applies the correction of Eq. 13 to the gradient it is given:
 * always for the approximation variant; for the true variant only once the
 * first N_taylor steps, whose gradient already is Eq. 11's g~, are over. */
static int approximation_active(const novak_oracle_hparams *h, int64_t t)
{
    if (h->nesterov_variant == 3)
        return t > (int64_t)h->true_steps;
    return h->nesterov_variant == 1;
}

/* Eq. 10: the position the true variant evaluates the gradient at,
 * theta~ = theta_{t-1} + beta_N m_{t-1}, element by element. */
void novak_oracle_extrapolate(double beta_n, int64_t n, const double *theta,
                              const double *m, double *theta_tilde)
{
    for (int64_t i = 0; i < n; ++i)
        theta_tilde[i] = theta[i] + beta_n * m[i];
}

/* 1 when step t of these hyperparameters expects Eq. 11's gradient. */
int32_t novak_oracle_wants_extrapolation(const novak_oracle_hparams *h, int64_t t)
{
    return (h->nesterov_variant == 3 && t <= (int64_t)h->true_steps) ? 1 : 0;
}

typedef struct {
    double bc1;       /* 1 - beta1^t                        (Eq. 5) */
    double bc2;       /* 1 - beta2^t                        (Eq. 5) */
    double rho_inf;   /* Eq. 6 */
    double rho_t;     /* Eq. 7 */
    double r_t;       /* Eq. 9, or 1 on the un-rectified branch     */
    double step_size; /* alpha * r_t / bc1^(bias1_power-1)          */
    double decay;     /* 1 - alpha*lambda                   (Eq. 18) */
    int32_t rect_branch; /* 1 when Eq. 8's first case was taken      */
    int32_t is_sync;     /* 1 when lookahead_k>0 and t mod k == 0    */
    double beta1_t;   /* coefficient of Eq. 1 at this step: beta1, or Eq. 3 */
    double beta2_t;   /* coefficient of Eq. 2 at this step: beta2, or Eq. 4 */
} novak_oracle_scalars;

/* Per-step scalars for the 1-based step index t (Eq. 5-9, 18). */
void novak_oracle_scalars_at(const novak_oracle_hparams *h, int64_t t,
                             novak_oracle_scalars *s)
{
    long double b1t = powl((long double)h->beta1, (long double)t);
    long double b2t = powl((long double)h->beta2, (long double)t);
    s->bc1 = (double)(1.0L - b1t);
    s->bc2 = (double)(1.0L - b2t);
    s->rho_inf = 2.0 / (1.0 - h->beta2) - 1.0;
    s->rho_t = (double)((long double)s->rho_inf
                        - 2.0L * (long double)t * b2t / (1.0L - b2t));
    s->rect_branch = 0;
    s->r_t = 1.0;
    if (h->rectified && s->rho_t >= 5.0) {
        double num = (s->rho_t - 4.0) * (s->rho_t - 2.0) * s->rho_inf;
        double den = (s->rho_inf - 4.0) * (s->rho_inf - 2.0) * s->rho_t;
        s->r_t = sqrt(num / den);
        s->rect_branch = 1;
    }
    s->step_size = h->lr * s->r_t;
    if (h->bias1_power == 2)
        s->step_size /= s->bc1;
    s->decay = 1.0 - h->lr * h->weight_decay;
    s->is_sync = (h->lookahead_k > 0 && (t % h->lookahead_k) == 0) ? 1 : 0;
    /* Phase 3, Eq. 3-4: momentum coefficients warmed up over tau1, tau2 steps. */
    s->beta1_t = h->beta1;
    s->beta2_t = h->beta2;
    if (h->adaptive_beta) {
        s->beta1_t = h->beta1 * (1.0 - exp(-(double)t / h->tau1));
        s->beta2_t = h->beta2 * (1.0 - exp(-(double)t / h->tau2));
    }
}

/*
 * Layer-wise adaptation, Eq. 19 / 25, for ONE tensor of n elements at step t:
 * clip(||theta_t||_2 / ||u_t||_2, 0.1, 10), where u_t is the base direction of
 * Eq. 17 that this step's gradient produces (the moments are advanced in local
 * variables only; nothing is written).  1 when ||u_t|| = 0.
 */
double novak_oracle_trust_ratio(const novak_oracle_hparams *h, int64_t t, int64_t n,
                                const double *theta, const double *g,
                                const double *m, const double *v)
{
    novak_oracle_scalars s;
    novak_oracle_scalars_at(h, t, &s);
    double sum_theta = 0.0, sum_u = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double gt = g[i];
        if (approximation_active(h, t))
            gt = g[i] + h->nesterov_beta * (g[i] - m[i]);
        const double m_new = s.beta1_t * m[i] + (1.0 - s.beta1_t) * gt;
        const double v_new = s.beta2_t * v[i] + (1.0 - s.beta2_t) * gt * gt;
        const double u = (m_new / s.bc1) / (sqrt(v_new / s.bc2) + h->eps);   /* Eq. 5, 17 */
        sum_theta += theta[i] * theta[i];
        sum_u += u * u;
    }
    if (sum_u == 0.0)
        return 1.0;
    double eta = sqrt(sum_theta) / sqrt(sum_u);
    if (eta < 0.1) eta = 0.1;
    if (eta > 10.0) eta = 10.0;
    return eta;
}

/*
 * One step (index t, 1-based, i.e. after the counter was incremented) over n
 * independent elements.  theta, m, v are updated in place; g is read only.
 * slow is used when lookahead_k > 0 (caller sets slow = theta_0 before the
 * first step, Eq. 28); acc when lookahead_mode == 1 (caller zeroes it).
 * trust is the tensor's lambda_trust of Eq. 24a (1 without layer adaptation).
 */
void novak_oracle_step(const novak_oracle_hparams *h, int64_t t, int64_t n,
                       double *theta, const double *g, double *m, double *v,
                       double *slow, double *acc, double trust)
{
    novak_oracle_scalars s;
    novak_oracle_scalars_at(h, t, &s);
    const int k = h->lookahead_k;

    for (int64_t i = 0; i < n; ++i) {
        /* Phase 2: Nesterov approximation, Eq. 13 (m[i] is m_{t-1}). */
        double gt = g[i];
        if (approximation_active(h, t))
            gt = g[i] + h->nesterov_beta * (g[i] - m[i]);

        /* Phase 4: Eq. 1-2 (with the coefficients of Eq. 3-4 when warmed up). */
        m[i] = s.beta1_t * m[i] + (1.0 - s.beta1_t) * gt;
        v[i] = s.beta2_t * v[i] + (1.0 - s.beta2_t) * gt * gt;

        /* Phase 5: Eq. 5. */
        double m_hat = m[i] / s.bc1;
        double v_hat = v[i] / s.bc2;

        /* Phase 8: Eq. 17, the mask of Eq. 27, then Eq. 16 for the classical variant. */
        double u = m_hat / (sqrt(v_hat) + h->eps);
        if (h->sparse_threshold > 0.0 && !(fabs(u) > h->sparse_threshold))
            u = 0.0;
        if (h->nesterov_variant == 2)
            u = h->beta1 * m_hat + (1.0 - h->beta1) * u;

        /* Phase 9: Eq. 18 then Eq. 24 (decay with the base rate alpha). */
        double theta_fast = theta[i] * s.decay - s.step_size * trust * u;

        /* Reduced-precision storage: the step above used the unrounded moments;
         * the next step reads back their bfloat16 roundings. */
        if (h->moment_bf16) {
            m[i] = novak_oracle_round_bf16(m[i]);
            v[i] = novak_oracle_round_bf16(v[i]);
        }

        /* Phase 10: lookahead. */
        if (k <= 0) {
            theta[i] = theta_fast;
        } else if (h->lookahead_mode == 0) {
            if (s.is_sync) {
                theta[i] = slow[i] + h->lookahead_alpha * (theta_fast - slow[i]);
                slow[i] = theta[i];
            } else {
                theta[i] = theta_fast;
            }
        } else {
            acc[i] += theta_fast;
            if (s.is_sync) {
                theta[i] = slow[i]
                         + h->lookahead_alpha * (acc[i] / (double)k - slow[i]);
                slow[i] = theta[i];
                acc[i] = 0.0;
            } else {
                theta[i] = theta_fast;
            }
        }
    }
}

/* ------------------------------------------------------------------------
 * Phase 2, gradient processing (Section 5.1; Table 2; Section 5.8).
 * ---------------------------------------------------------------------- */

/* Global L2 norm of the gradient: every element of every tensor of the group
 * (Section 5.8: the threshold applies to the global gradient norm). */
double novak_oracle_global_norm(int32_t n_tensors, const int64_t *numel,
                                const double *const *g)
{
    double sum = 0.0;
    for (int32_t k = 0; k < n_tensors; ++k)
        for (int64_t i = 0; i < numel[k]; ++i)
            sum += g[k][i] * g[k][i];
    return sqrt(sum);
}

/* Gradient clipping (Table 2: active when ||g_t|| > c_clip; norm computation
 * and scaling): the factor that brings the norm down to c_clip, else 1. */
double novak_oracle_clip_factor(double norm, double c_clip)
{
    if (norm > c_clip)
        return c_clip / norm;
    return 1.0;
}

/* g <- factor * g */
void novak_oracle_scale(int64_t n, double factor, double *g)
{
    for (int64_t i = 0; i < n; ++i)
        g[i] = factor * g[i];
}

/* Gradient centralization, Eq. 26, for a tensor of dimension > 1 stored
 * contiguously as rows x row_len (row = one index of dimension 0, row_len =
 * the product of dimensions 1..d): subtract from every element the mean over
 * dimensions 1..d of its row. */
void novak_oracle_centralize(int64_t rows, int64_t row_len, double *g)
{
    for (int64_t r = 0; r < rows; ++r) {
        double *row = g + r * row_len;
        double sum = 0.0;
        for (int64_t j = 0; j < row_len; ++j)
            sum += row[j];
        const double mean = sum / (double)row_len;
        for (int64_t j = 0; j < row_len; ++j)
            row[j] = row[j] - mean;
    }
}

/* The base direction u_t of Eq. 17 that step t would produce for each of n
 * elements (moments advanced in local variables; nothing is written).  Lets a
 * test see how close |u| comes to the threshold of Eq. 27. */
void novak_oracle_direction(const novak_oracle_hparams *h, int64_t t, int64_t n,
                            const double *g, const double *m, const double *v,
                            double *u_out)
{
    novak_oracle_scalars s;
    novak_oracle_scalars_at(h, t, &s);
    for (int64_t i = 0; i < n; ++i) {
        double gt = g[i];
        if (approximation_active(h, t))
            gt = g[i] + h->nesterov_beta * (g[i] - m[i]);
        const double m_new = s.beta1_t * m[i] + (1.0 - s.beta1_t) * gt;
        const double v_new = s.beta2_t * v[i] + (1.0 - s.beta2_t) * gt * gt;
        u_out[i] = (m_new / s.bc1) / (sqrt(v_new / s.bc2) + h->eps);
    }
}

/* Distance from x to the nearest point where bfloat16 rounding changes its
 * answer (the midpoint between two neighbouring bfloat16 values). */
static double bf16_boundary_distance(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x))
        return INFINITY;
    int e;
    (void)frexp(x, &e);
    int q = e - 8;
    if (q < -133)
        q = -133;
    const double y = ldexp(fabs(x), -q);
    return ldexp(fabs(y - floor(y) - 0.5), q);
}

/* For tests of the bfloat16 storage: how close the unrounded m_t and v_t that
 * step t would produce come to a rounding boundary, relative to the size of
 * the terms they are summed from (so that cancellation is accounted for), the
 * smaller of the two per element.  An implementation in lower precision can
 * round an element differently only where this is of the order of its own
 * rounding error.  Nothing is written but margin_out. */
void novak_oracle_rounding_margin(const novak_oracle_hparams *h, int64_t t, int64_t n,
                                  const double *g, const double *m, const double *v,
                                  double *margin_out)
{
    novak_oracle_scalars s;
    novak_oracle_scalars_at(h, t, &s);
    for (int64_t i = 0; i < n; ++i) {
        double gt = g[i], g_scale = fabs(g[i]);
        if (approximation_active(h, t)) {
            gt = g[i] + h->nesterov_beta * (g[i] - m[i]);
            g_scale = fabs(g[i]) + h->nesterov_beta * (fabs(g[i]) + fabs(m[i]));
        }
        const double m_new = s.beta1_t * m[i] + (1.0 - s.beta1_t) * gt;
        const double v_new = s.beta2_t * v[i] + (1.0 - s.beta2_t) * gt * gt;
        const double m_scale = s.beta1_t * fabs(m[i]) + (1.0 - s.beta1_t) * g_scale;
        const double v_scale = s.beta2_t * v[i] + (1.0 - s.beta2_t) * g_scale * g_scale;
        double a = m_scale > 0.0 ? bf16_boundary_distance(m_new) / m_scale : INFINITY;
        double b = v_scale > 0.0 ? bf16_boundary_distance(v_new) / v_scale : INFINITY;
        margin_out[i] = a < b ? a : b;
    }
}

/* ------------------------------------------------------------------------
 * Phase 7, automatic learning-rate scaling (Eq. 20-22).
 * ---------------------------------------------------------------------- */

/* Advances the two moving averages (Eq. 20, 21) with this step's global norms
 * and returns alpha_auto = clip(g_bar / theta_bar, 0.1, 2) (Eq. 22).  The ratio
 * of two zero averages is undefined and taken as 1. */
double novak_oracle_auto_lr(double gamma, double grad_norm, double param_norm,
                            double *g_bar, double *theta_bar)
{
    *g_bar = gamma * grad_norm + (1.0 - gamma) * *g_bar;
    *theta_bar = gamma * param_norm + (1.0 - gamma) * *theta_bar;
    if (*g_bar == 0.0 && *theta_bar == 0.0)
        return 1.0;
    double a = *g_bar / *theta_bar;
    if (a < 0.1) a = 0.1;
    if (a > 2.0) a = 2.0;
    return a;
}
