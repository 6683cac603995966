"""Each plausible mistake planted in the oracle must trip at least one pin.

The mistake is planted in a copy of the oracle's C source (text replacement),
compiled on the CPU into a temporary library and run through the same pins as
the real oracle.  A mutant that passes every pin would mean the pins cannot
tell the oracle from a wrong one.
"""
import os

import pytest

from oracle import novak_oracle as O
from oracle_pins import ALL_PINS

SRC = os.path.join(os.path.dirname(O.__file__), "novak_oracle.c")

# (name, text in the oracle, replacement)
MUTANTS = [
    ("m_sign", "(1.0 - s.beta1_t) * gt;", "(1.0 + s.beta1_t) * gt;"),
    ("v_not_squared", "(1.0 - s.beta2_t) * gt * gt;", "(1.0 - s.beta2_t) * gt;"),
    ("v_uses_beta1", "s.beta2_t * v[i]", "s.beta1_t * v[i]"),
    ("approx_sign", "h->nesterov_beta * (g[i] - m[i]);", "h->nesterov_beta * (m[i] - g[i]);"),
    ("approx_uses_new_m_only_first_moment",
     "(1.0 - s.beta2_t) * gt * gt;", "(1.0 - s.beta2_t) * g[i] * g[i];"),
    ("vhat_uses_bc1", "double v_hat = v[i] / s.bc2;", "double v_hat = v[i] / s.bc1;"),
    ("mhat_uses_bc2", "double m_hat = m[i] / s.bc1;", "double m_hat = m[i] / s.bc2;"),
    ("mhat_uncorrected", "double m_hat = m[i] / s.bc1;", "double m_hat = m[i];"),
    ("eps_inside_root", "(sqrt(v_hat) + h->eps)", "sqrt(v_hat + h->eps)"),
    ("update_sign", "theta[i] * s.decay - s.step_size * trust * u;", "theta[i] * s.decay + s.step_size * trust * u;"),
    ("decay_without_lr", "1.0 - h->lr * h->weight_decay;", "1.0 - h->weight_decay;"),
    ("decay_with_rectified_rate", "1.0 - h->lr * h->weight_decay;",
     "1.0 - h->lr * s->r_t * h->weight_decay;"),
    ("classical_swapped", "u = h->beta1 * m_hat + (1.0 - h->beta1) * u;",
     "u = (1.0 - h->beta1) * m_hat + h->beta1 * u;"),
    ("last_sync_sign", "h->lookahead_alpha * (theta_fast - slow[i]);",
     "h->lookahead_alpha * (slow[i] - theta_fast);"),
    ("sync_off_by_one", "(t % h->lookahead_k) == 0", "(t % h->lookahead_k) == 1"),
    ("rho_drops_t", "2.0L * (long double)t * b2t", "2.0L * b2t"),
    ("rho_uses_beta1", "- 2.0L * (long double)t * b2t / (1.0L - b2t)",
     "- 2.0L * (long double)t * b1t / (1.0L - b1t)"),
    ("threshold_textbook", "s->rho_t >= 5.0", "s->rho_t > 4.0"),
    ("r_inverted", "sqrt(num / den)", "sqrt(den / num)"),
    ("r_not_rooted", "sqrt(num / den)", "(num / den)"),
    ("traj_mean_not_divided", "acc[i] / (double)k", "acc[i]"),
    ("traj_acc_not_reset", "acc[i] = 0.0;", ";"),
    ("bias1_power_ignored", "if (h->bias1_power == 2)", "if (0)"),
    ("rectified_flag_ignored", "if (h->rectified && s->rho_t >= 5.0)", "if (s->rho_t >= 5.0)"),
    # phase 3: adaptive beta
    ("warmup_sign", "exp(-(double)t / h->tau1)", "exp((double)t / h->tau1)"),
    ("warmup_beta2_uses_tau1", "exp(-(double)t / h->tau2)", "exp(-(double)t / h->tau1)"),
    ("warmup_not_complemented", "h->beta2 * (1.0 - exp(-(double)t / h->tau2));",
     "h->beta2 * exp(-(double)t / h->tau2);"),
    ("warmup_in_bias_correction", "s->bc1 = (double)(1.0L - b1t);",
     "s->bc1 = (double)(1.0L - b1t); if (h->adaptive_beta) s->bc1 = 1.0 - pow(h->beta1 * (1.0 - exp(-(double)t / h->tau1)), (double)t);"),
    ("warmup_in_classical_blend", "u = h->beta1 * m_hat + (1.0 - h->beta1) * u;",
     "u = s.beta1_t * m_hat + (1.0 - s.beta1_t) * u;"),
    ("warmup_flag_ignored", "if (h->adaptive_beta) {", "if (1) {"),
    # true Nesterov (Eq. 10) and its fallback
    ("extrapolate_sign", "theta_tilde[i] = theta[i] + beta_n * m[i];",
     "theta_tilde[i] = theta[i] - beta_n * m[i];"),
    ("extrapolate_drops_beta", "theta_tilde[i] = theta[i] + beta_n * m[i];",
     "theta_tilde[i] = theta[i] + m[i];"),
    ("fallback_off_by_one", "return t > (int64_t)h->true_steps;",
     "return t >= (int64_t)h->true_steps;"),
    ("fallback_never", "return t > (int64_t)h->true_steps;", "return 0;"),
    ("true_corrected_from_the_start", "return t > (int64_t)h->true_steps;", "return 1;"),
    ("wants_off_by_one", "t <= (int64_t)h->true_steps) ? 1 : 0", "t < (int64_t)h->true_steps) ? 1 : 0"),
    # moments stored in bfloat16
    ("bf16_truncates", "ldexp(rint(ldexp(x, -q)), q);", "ldexp(trunc(ldexp(x, -q)), q);"),
    ("bf16_ties_away", "ldexp(rint(ldexp(x, -q)), q);", "ldexp(round(ldexp(x, -q)), q);"),
    ("bf16_seven_bits", "int q = e - 8;                   /* quantum", "int q = e - 7;                   /* quantum"),
    ("bf16_no_subnormals", "if (q < -133)\n        q = -133;                    /* subnormal", "if (0)\n        q = -133;                    /* subnormal"),
    ("bf16_no_overflow", "if (fabs(r) >= ldexp(1.0, 128))", "if (0)"),
    ("bf16_step_sees_rounded_m", "double m_hat = m[i] / s.bc1;",
     "if (h->moment_bf16) m[i] = novak_oracle_round_bf16(m[i]); double m_hat = m[i] / s.bc1;"),
    ("bf16_step_sees_rounded_v", "double v_hat = v[i] / s.bc2;",
     "if (h->moment_bf16) v[i] = novak_oracle_round_bf16(v[i]); double v_hat = v[i] / s.bc2;"),
    ("bf16_v_kept_exact", "            v[i] = novak_oracle_round_bf16(v[i]);\n", ""),
    ("bf16_m_kept_exact", "            m[i] = novak_oracle_round_bf16(m[i]);\n", ""),
    ("bf16_margin_to_grid_point", "ldexp(fabs(y - floor(y) - 0.5), q);", "ldexp(fabs(y - floor(y)), q);"),
    ("bf16_margin_ignores_v", "margin_out[i] = a < b ? a : b;", "margin_out[i] = a;"),
    # phase 7: automatic learning-rate scaling
    ("auto_inverted", "double a = *g_bar / *theta_bar;", "double a = *theta_bar / *g_bar;"),
    ("auto_gamma_swapped", "*g_bar = gamma * grad_norm + (1.0 - gamma) * *g_bar;",
     "*g_bar = (1.0 - gamma) * grad_norm + gamma * *g_bar;"),
    ("auto_theta_not_averaged", "*theta_bar = gamma * param_norm + (1.0 - gamma) * *theta_bar;",
     "*theta_bar = param_norm;"),
    ("auto_upper_bound_10", "if (a > 2.0) a = 2.0;", "if (a > 10.0) a = 10.0;"),
    ("auto_lower_clip_missing", "if (a < 0.1) a = 0.1;", ";"),
    # phase 8: sparse updates
    ("mask_inverted", "!(fabs(u) > h->sparse_threshold))", "(fabs(u) > h->sparse_threshold))"),
    ("mask_signed", "!(fabs(u) > h->sparse_threshold))", "!(u > h->sparse_threshold))"),
    ("mask_not_strict", "!(fabs(u) > h->sparse_threshold))", "!(fabs(u) >= h->sparse_threshold))"),
    ("mask_after_blend", "if (h->sparse_threshold > 0.0 && !(fabs(u) > h->sparse_threshold))\n            u = 0.0;\n        if (h->nesterov_variant == 2)\n            u = h->beta1 * m_hat + (1.0 - h->beta1) * u;",
     "if (h->nesterov_variant == 2)\n            u = h->beta1 * m_hat + (1.0 - h->beta1) * u;\n        if (h->sparse_threshold > 0.0 && !(fabs(u) > h->sparse_threshold))\n            u = 0.0;"),
    ("mask_on_gradient", "!(fabs(u) > h->sparse_threshold))", "!(fabs(gt) > h->sparse_threshold))"),
    # the base direction on its own (novak_oracle_direction)
    ("direction_stale_moments", "u_out[i] = (m_new / s.bc1) / (sqrt(v_new / s.bc2) + h->eps);",
     "u_out[i] = (m[i] / s.bc1) / (sqrt(v[i] / s.bc2) + h->eps);"),
    ("direction_eps_inside_root", "u_out[i] = (m_new / s.bc1) / (sqrt(v_new / s.bc2) + h->eps);",
     "u_out[i] = (m_new / s.bc1) / sqrt(v_new / s.bc2 + h->eps);"),
    ("direction_without_nesterov_term",
     "gt = g[i] + h->nesterov_beta * (g[i] - m[i]);\n        const double m_new = s.beta1_t * m[i] + (1.0 - s.beta1_t) * gt;\n        const double v_new = s.beta2_t * v[i] + (1.0 - s.beta2_t) * gt * gt;\n        u_out",
     "gt = g[i];\n        const double m_new = s.beta1_t * m[i] + (1.0 - s.beta1_t) * gt;\n        const double v_new = s.beta2_t * v[i] + (1.0 - s.beta2_t) * gt * gt;\n        u_out"),
    ("direction_uncorrected_second_moment", "u_out[i] = (m_new / s.bc1) / (sqrt(v_new / s.bc2) + h->eps);",
     "u_out[i] = (m_new / s.bc1) / (sqrt(v_new) + h->eps);"),
    # phase 7: layer-wise adaptation
    ("trust_inverted", "double eta = sqrt(sum_theta) / sqrt(sum_u);", "double eta = sqrt(sum_u) / sqrt(sum_theta);"),
    ("trust_of_squared_norms", "double eta = sqrt(sum_theta) / sqrt(sum_u);", "double eta = sum_theta / sum_u;"),
    ("trust_l1", "sum_u += u * u;", "sum_u += fabs(u);"),
    ("trust_lower_clip_missing", "if (eta < 0.1) eta = 0.1;", ";"),
    ("trust_upper_clip_missing", "if (eta > 10.0) eta = 10.0;", ";"),
    ("trust_old_moments", "const double u = (m_new / s.bc1) / (sqrt(v_new / s.bc2) + h->eps);",
     "const double u = (m[i] / s.bc1) / (sqrt(v[i] / s.bc2) + h->eps);"),
    ("trust_without_nesterov_term", "gt = g[i] + h->nesterov_beta * (g[i] - m[i]);\n        const double m_new",
     "gt = g[i];\n        const double m_new"),
    ("trust_on_decay_too", "theta[i] * s.decay - s.step_size * trust * u;",
     "trust * (theta[i] * s.decay - s.step_size * u);"),
    ("trust_dropped", "s.step_size * trust * u;", "s.step_size * u;"),
    ("trust_zero_direction", "if (sum_u == 0.0)\n        return 1.0;", "if (sum_u == 0.0)\n        return 10.0;"),
    # phase 2: clipping and centralization
    ("norm_not_rooted", "return sqrt(sum);", "return sum;"),
    ("norm_l1", "sum += g[k][i] * g[k][i];", "sum += fabs(g[k][i]);"),
    ("norm_first_tensor_only", "for (int32_t k = 0; k < n_tensors; ++k)", "for (int32_t k = 0; k < 1; ++k)"),
    ("clip_inverted", "return c_clip / norm;", "return norm / c_clip;"),
    ("clip_always", "if (norm > c_clip)", "if (1)"),
    ("clip_when_small", "if (norm > c_clip)", "if (norm < c_clip)"),
    ("scale_dropped", "g[i] = factor * g[i];", "g[i] = g[i];"),
    ("gc_mean_over_rows", "const double mean = sum / (double)row_len;", "const double mean = sum / (double)rows;"),
    ("gc_added", "row[j] = row[j] - mean;", "row[j] = row[j] + mean;"),
    ("gc_sum_of_first_entries", "sum += row[j];", "sum += row[0];"),
    ("gc_mean_of_previous_row", "row[j] = row[j] - mean;", "row[j] = row[j] - (r ? prev : mean);\n        prev = mean;"),
    ("gc_first_row_only", "for (int64_t r = 0; r < rows; ++r) {", "for (int64_t r = 0; r < 1; ++r) {"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(name, old, new, tmp_path):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation site for {name} not found in the oracle"
    src = tmp_path / "mutant.c"
    src.write_text("static double prev;\n" + text.replace(old, new))
    lib = O.load_library(O.compile_oracle(str(src), str(tmp_path / "mutant.so"), force=True))
    caught = []
    for pin in ALL_PINS:
        try:
            pin(lib)
        except AssertionError:
            caught.append(pin.__name__)
            break
    assert caught, f"mutant {name} passed every pin"
