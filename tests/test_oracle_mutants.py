"""Each plausible mistake, planted in a copy of the oracle's source, must trip a pin.

The mutants are textual edits of oracle/ga_oracle.cpp compiled into a temporary library; the
committed oracle is never touched. A mutant that no pin catches means the pins are too weak.
"""
import os
import subprocess

import pytest

import oracle
from tests import oracle_pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "ga_oracle.cpp")

# (name, text in the oracle, replacement)
MUTANTS = [
    ("gap_without_plus_one", "const T G = dist / C + (T)1;", "const T G = dist / C;"),
    ("gap_multiplies_gradient", "const T inv_gap = (T)1 / G;", "const T inv_gap = G;"),
    ("gap_reciprocal_unused", "const T g_hat = inv_gap * g;", "const T g_hat = g;"),
    ("gap_divides_by_C_squared", "const T G = dist / C + (T)1;", "const T G = dist / C / C + (T)1;"),
    ("gap_uses_signed_distance", "const T dist = std::fabs(theta[j] - s[j]);\n                const T G",
     "const T dist = theta[j] - s[j];\n                const T G"),
    ("gap_against_master_itself", "const T dist = std::fabs(theta[j] - s[j]);\n                const T G",
     "const T dist = std::fabs(theta[j] - theta[j]);\n                const T G"),
    ("momentum_with_dampening", "v[j] = std::fma(gamma, v[j], g_hat);",
     "v[j] = std::fma(gamma, v[j], ((T)1 - gamma) * g_hat);"),
    ("momentum_dropped_in_ga", "v[j] = std::fma(gamma, v[j], g_hat);", "v[j] = g_hat;"),
    ("step_sign", "theta[j] = step(theta[j], v[j], g_hat, eta);\n                sum_gap",
     "theta[j] = step(theta[j], v[j], g_hat, -eta);\n                sum_gap"),
    ("step_uses_gradient_not_v", "theta[j] = step(theta[j], v[j], g_hat, eta);\n                sum_gap",
     "theta[j] = step(theta[j], g_hat, g_hat, eta);\n                sum_gap"),
    ("plain_step_is_nesterov", "if (!nesterov) return std::fma(-e, v_new, th);", "if (nesterov) return std::fma(-e, v_new, th);"),
    ("nesterov_without_gradient", "return std::fma(-e, std::fma(gamma, v_new, g_pen), th);",
     "return std::fma(-e, gamma * v_new, th);"),
    ("nesterov_lookahead_unscaled", "return std::fma(-e, std::fma(gamma, v_new, g_pen), th);",
     "return std::fma(-e, v_new + g_pen, th);"),
    ("sa_multiplies_by_tau", "const T eta_tau = eta / (T)tau;", "const T eta_tau = eta * (T)tau;"),
    ("sa_ignores_tau", "const T eta_tau = eta / (T)tau;", "const T eta_tau = eta;"),
    ("sa_divides_gradient_twice", "const T eta_tau = eta / (T)tau;", "const T eta_tau = eta / (T)tau / (T)tau;"),
    ("delay_off_by_one", "const int64_t tau = k - iter[i];", "const int64_t tau = k - iter[i] + 1;"),
    ("delay_of_wrong_worker", "const int64_t tau = k - iter[i];", "const int64_t tau = k - iter[0];"),
    ("pull_forgets_iteration", "iter[i] = k_done;\n", "\n"),
    ("pull_saves_wrong_row", "saved[(size_t)i * d + j] = theta[j];\n        iter[i]",
     "saved[(size_t)0 * d + j] = theta[j];\n        iter[i]"),
    ("c_without_sqrt", "return eta_max * (std::sqrt(m_hat) + eps);", "return eta_max * (m_hat + eps);"),
    ("c_without_eta_max", "return eta_max * (std::sqrt(m_hat) + eps);", "return (std::sqrt(m_hat) + eps);"),
    ("c_eps_inside_sqrt", "return eta_max * (std::sqrt(m_hat) + eps);", "return eta_max * std::sqrt(m_hat + eps);"),
    ("c_no_bias_correction", "const T m_hat = m_j * inv_bias_k;", "const T m_hat = m_j;"),
    ("c_bias_exponent_off_by_one", "std::pow((double)beta, (double)k_c)", "std::pow((double)beta, (double)(k_c + 1))"),
    ("c_bias_uses_beta_not_power", "std::pow((double)beta, (double)k_c)", "(double)beta"),
    ("m_first_moment", "m[j] = std::fma(beta, m[j], one_minus_beta * (v[j] * v[j]));",
     "m[j] = std::fma(beta, m[j], one_minus_beta * std::fabs(v[j]));"),
    ("m_weights_swapped", "m[j] = std::fma(beta, m[j], one_minus_beta * (v[j] * v[j]));",
     "m[j] = std::fma(one_minus_beta, m[j], beta * (v[j] * v[j]));"),
    ("m_from_raw_gradient", "m[j] = std::fma(beta, m[j], one_minus_beta * (v[j] * v[j]));",
     "m[j] = std::fma(beta, m[j], one_minus_beta * (gw(grad, j) * gw(grad, j)));"),
    ("asgd_dampened", "v[j] = std::fma(gamma, v[j], g);\n                theta[j] = step(theta[j], v[j], g, eta);",
     "v[j] = std::fma(gamma, v[j], ((T)1 - gamma) * g);\n                theta[j] = step(theta[j], v[j], g, eta);"),
    ("adam_order_uses_penalised_v", "const T u = std::fma(gamma, v[j], gw(grad, j));",
     "const T u = v[j];"),
    ("set_params_keeps_momentum", "v[j] = 0;\n            m[j] = 0;", "m[j] = 0;"),
    # SA-Gradient and the DANA masters
    ("sa_grad_multiplies", "const T g_tau = gw(grad, j) / (T)tau;", "const T g_tau = gw(grad, j) * (T)tau;"),
    ("sa_grad_ignores_tau", "const T g_tau = gw(grad, j) / (T)tau;", "const T g_tau = gw(grad, j);"),
    ("dana_estimate_sign", "saved[(size_t)i * d + j] = std::fma(-eta_gamma, total, theta[j]);",
     "saved[(size_t)i * d + j] = std::fma(eta_gamma, total, theta[j]);"),
    ("dana_estimate_without_gamma", "const T eta_gamma = eta * gamma;", "const T eta_gamma = eta;"),
    ("dana_estimate_own_momentum_only", "T total = vsum[j];", "T total = vw[(size_t)i * d + j];"),
    ("dana_sends_theta", "saved[(size_t)i * d + j] = std::fma(-eta_gamma, total, theta[j]);",
     "saved[(size_t)i * d + j] = theta[j];"),
    ("dana_shared_momentum", "T* vi = &vw[(size_t)i * d];", "T* vi = &vw[0];"),
    ("dana_sa_ignores_tau", "g_pen = g / (T)tau;                        // DANA-SA: g / tau", "g_pen = g;"),
    ("dana_master_uses_sum", "theta[j] = std::fma(-eta, v_new, theta[j]);    // master's weights",
     "theta[j] = std::fma(-eta, vsum[j], theta[j]);"),
    ("dana_sum_forgets_old", "vsum[j] = (vsum[j] - v_old) + v_new;", "vsum[j] = vsum[j] + v_new;"),
    ("dana_momentum_dampened", "const T v_new = std::fma(gamma, v_old, g_pen);",
     "const T v_new = std::fma(gamma, v_old, ((T)1 - gamma) * g_pen);"),
    ("dana_gap_against_theta0", "const T dist = std::fabs(theta[j] - s[j]); // s = the estimate saved when sent",
     "const T dist = std::fabs(theta[j] - theta[j]);"),
    ("dana_gap_without_one", "const T G = dist / C + (T)1;\n                const T inv_gap = (T)1 / G;\n                g_pen",
     "const T G = dist / C;\n                const T inv_gap = (T)1 / G;\n                g_pen"),
    ("dana_ga_m_from_sum", "m[j] = std::fma(beta, m[j], one_minus_beta * (vi[j] * vi[j]));",
     "m[j] = std::fma(beta, m[j], one_minus_beta * (vsum[j] * vsum[j]));"),
    # the Adam masters
    ("adam_first_moment_weight", "first = one_minus_beta1 * g;", "first = g;"),
    ("adam_second_moment_of_penalised", "v2[j] = std::fma(beta2, v2[j], one_minus_beta2 * (g * g));",
     "v2[j] = std::fma(beta2, v2[j], one_minus_beta2 * (first * first));"),
    ("adam_second_moment_unsquared", "v2[j] = std::fma(beta2, v2[j], one_minus_beta2 * (g * g));",
     "v2[j] = std::fma(beta2, v2[j], one_minus_beta2 * std::fabs(g));"),
    ("adam_no_bias_correction_1", "const T m_hat = v[j] * inv_bias1;", "const T m_hat = v[j];"),
    ("adam_no_bias_correction_2", "const T v_hat = v2[j] * inv_bias2;", "const T v_hat = v2[j];"),
    ("adam_bias_exponent", "std::pow((double)beta1, (double)k)", "std::pow((double)beta1, (double)(k + 1))"),
    ("adam_eps_inside_root", "(std::sqrt(v_hat) + adam_eps)", "std::sqrt(v_hat + adam_eps)"),
    ("adam_step_sign", "theta[j] = theta[j] - (eta * m_hat)", "theta[j] = theta[j] + (eta * m_hat)"),
    ("adam_sa_multiplies", "first = one_minus_beta1 * (g / (T)tau);", "first = one_minus_beta1 * (g * (T)tau);"),
    ("adam_ga_divides_twice", "first = (one_minus_beta1 / G) * g;", "first = (one_minus_beta1 / G / G) * g;"),
    ("adam_ga_unpenalised", "first = (one_minus_beta1 / G) * g;", "first = one_minus_beta1 * g;"),
    ("adam_ga_c_from_first_moment", "m[j] = std::fma(beta, m[j], one_minus_beta * (g * g));\n        }\n        if (variant == ADAM_GA && c_order == 0) k_c += 1;",
     "m[j] = std::fma(beta, m[j], one_minus_beta * (v[j] * v[j]));\n        }\n        if (variant == ADAM_GA && c_order == 0) k_c += 1;"),
    ("weight_decay_sign", "std::fma(wd, theta[j], (T)grad[j])", "std::fma(-wd, theta[j], (T)grad[j])"),
    ("weight_decay_on_saved_copy_scale", "std::fma(wd, theta[j], (T)grad[j])", "std::fma(wd * wd, theta[j], (T)grad[j])"),
    ("weight_decay_not_penalised", "const T g_hat = inv_gap * g;", "const T g_hat = inv_gap * (T)grad[j] + (g - (T)grad[j]);"),
    # layer-wise / global Gap
    ("layer_norm_is_l1", "dist2 += (double)diff * (double)diff;", "dist2 += std::fabs((double)diff);"),
    ("layer_norm_not_rooted", "const T dist = (T)std::sqrt(dist2);", "const T dist = (T)dist2;"),
    ("layer_gap_without_one", "const T G = dist / C + (T)1;\n            const T inv_gap = (T)1 / G;\n            last_layer_gap",
     "const T G = dist / C;\n            const T inv_gap = (T)1 / G;\n            last_layer_gap"),
    ("layer_c_of_wrong_layer", "const T C = coeff(m_layer[p], ib);", "const T C = coeff(m_layer[0], ib);"),
    ("layer_m_from_gradient", "norm2 += (double)v[j] * (double)v[j];", "norm2 += (double)grad[j] * (double)grad[j];"),
    ("layer_m_mean_not_sum", "m_layer[p] = std::fma(beta, m_layer[p], one_minus_beta * (T)norm2);",
     "m_layer[p] = std::fma(beta, m_layer[p], one_minus_beta * (T)(norm2 / (double)(hi - lo)));"),
    ("layer_whole_vector_norm", "for (int64_t j = lo; j < hi; ++j) {\n                const T diff",
     "for (int64_t j = 0; j < d; ++j) {\n                const T diff"),
    ("layer_unpenalised", "const T g_hat = inv_gap * gw(grad, j);\n                v[j]", "const T g_hat = gw(grad, j);\n                v[j]"),
    ("dana_pull_forgets_iteration", "saved[(size_t)i * d + j] = std::fma(-eta_gamma, total, theta[j]);\n        }\n        iter[i] = k_done;",
     "saved[(size_t)i * d + j] = std::fma(-eta_gamma, total, theta[j]);\n        }"),
]


def _build_mutant(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutant {name}: target text not found in the oracle"
    src = tmp_path / f"{name}.cpp"
    src.write_text(text.replace(old, new, 1))
    out = tmp_path / f"lib_{name}.so"
    subprocess.check_call(["g++", *oracle.CXXFLAGS, "-w", "-o", str(out), str(src)])
    return oracle._bind(str(out))


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(tmp_path, name, old, new):
    lib = _build_mutant(tmp_path, name, old, new)

    def make(*a, **kw):
        return oracle.Oracle(*a, _lib=lib, **kw)

    caught = []
    for pin in oracle_pins.ALL_PINS:
        try:
            pin(make)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, f"no pin notices the mistake '{name}'"
