"""Plausible mistakes planted in copies of the oracle (on the CPU) must each
trip at least one pin: a dropped term, a misplaced epsilon, a wrong index."""
import os
import subprocess

import pytest

import oracle_pins as pins
from oracle import build as obuild, step as ostep

MUTANTS = {
    "eps_inside_root": ("sqrt(v_hat) + eps", "sqrt(v_hat + eps)"),
    "sum_instead_of_mean": ("sum_sq / (double)L", "sum_sq"),
    "no_bias_correction_v": ("v[b] / bc2", "v[b]"),
    "no_bias_correction_m": ("m[k] / bc1", "m[k]"),
    "decay_uses_gradient": ("lr * wd * p[k]", "lr * wd * gi"),
    "decay_dropped": ("p[k] = p[k] - lr * wd * p[k];", ";"),
    "beta2_swapped": ("(1.0 - beta2) * mean_sq + beta2 * v[b]", "beta2 * mean_sq + (1.0 - beta2) * v[b]"),
    "m_gain_dropped": ("(1.0 - beta1) * gi + beta1 * m[k]", "gi + beta1 * m[k]"),
    "block_offset_lost": ("const int64_t lo = b * L;", "const int64_t lo = 0 * b * L;"),
    "step_off_by_one": ("pow(beta1, (double)t)", "pow(beta1, (double)(t + 1))"),
    "abs_instead_of_square": ("sum_sq = sum_sq + gi * gi;", "sum_sq = sum_sq + fabs(gi);"),
    "sum_not_accumulated": ("sum_sq = sum_sq + gi * gi;", "sum_sq = gi * gi;"),
    "update_uses_raw_gradient": ("lr * m_hat / denom", "lr * gi / denom"),
    "update_sign": ("p[k] = p[k] - lr * m_hat / denom;", "p[k] = p[k] + lr * m_hat / denom;"),
    "bf16_shift": ("((uint32_t)h) << 16", "((uint32_t)h) << 15"),
    "mean_over_tensor": ("sum_sq / (double)L", "sum_sq / (double)numel"),
    # second wave
    "decay_flag_ignored": ("if (apply_wd)", "if (1)"),
    # (p - lr*u) * (1 - lr*wd) instead of p * (1 - lr*wd) - lr*u
    "decay_after_the_adam_term": ("p[k] = p[k] - lr * m_hat / denom;",
                                  "p[k] = p[k] - lr * m_hat / denom * (apply_wd ? 1.0 - lr * wd : 1.0);"),
    "bias_corrections_swapped": ("const double bc1 = 1.0 - pow(beta1, (double)t);",
                                 "const double bc1 = 1.0 - pow(beta2, (double)t);"),
    "beta2_bias_uses_beta1": ("const double bc2 = 1.0 - pow(beta2, (double)t);",
                              "const double bc2 = 1.0 - pow(beta1, (double)t);"),
    "v_not_stored": ("v[b] = (1.0 - beta2) * mean_sq + beta2 * v[b];\n        const double v_hat = v[b] / bc2;",
                     "const double v_new = (1.0 - beta2) * mean_sq + beta2 * v[b];\n        const double v_hat = v_new / bc2;"),
    "v_hat_from_old_v": ("v[b] = (1.0 - beta2) * mean_sq + beta2 * v[b];\n        const double v_hat = v[b] / bc2;",
                         "const double v_hat = v[b] / bc2;\n        v[b] = (1.0 - beta2) * mean_sq + beta2 * v[b];"),
    "root_dropped": ("sqrt(v_hat) + eps", "v_hat + eps"),
    "eps_dropped": ("sqrt(v_hat) + eps", "sqrt(v_hat)"),
    "m_updated_after_use": ("const double m_hat = m[k] / bc1;", "const double m_hat = (m[k] - (1.0 - beta1) * gi) / (beta1 > 0 ? beta1 : 1.0) / bc1;"),
    "last_block_skipped": ("for (int64_t b = 0; b < n_blocks; ++b) {", "for (int64_t b = 0; b + 1 < n_blocks || b == 0; ++b) {"),
    "last_element_of_block_not_summed": ("for (int64_t i = 0; i < L; ++i) {\n            const double gi = grad_at(g, g_dtype, lo + i);\n            sum_sq",
                                         "for (int64_t i = 0; i + 1 < L || i == 0; ++i) {\n            const double gi = grad_at(g, g_dtype, lo + i);\n            sum_sq"),
    "gradient_index_shifted": ("const double gi = grad_at(g, g_dtype, k);", "const double gi = grad_at(g, g_dtype, k > 0 ? k - 1 : k);"),
    "f32_read_as_bf16_pairs": ("case ORACLE_G_F32:  return (double)((const float *)g)[i];",
                               "case ORACLE_G_F32:  return widen_bf16(((const uint16_t *)g)[2 * i + 1]);"),
    "lr_applied_twice": ("p[k] = p[k] - lr * m_hat / denom;", "p[k] = p[k] - lr * lr * m_hat / denom;"),
    "wd_not_scaled_by_lr": ("p[k] = p[k] - lr * wd * p[k];", "p[k] = p[k] - wd * p[k];"),
}


STAT_MUTANTS = {
    "max_is_min": ("(i == 0 || sq > acc) ? sq : acc", "(i == 0 || sq < acc) ? sq : acc"),
    "min_is_max": ("(i == 0 || sq < acc) ? sq : acc", "(i == 0 || sq > acc) ? sq : acc"),
    "two_norm_without_root": ("if (statistic == 4) stat = sqrt(acc);", ";"),
    "two_norm_of_g_not_gg": ("else acc = acc + sq * sq;", "else acc = acc + sq;"),
    "one_norm_divided": ("if (statistic == 0) stat = acc / (double)L;", "if (statistic == 0 || statistic == 3) stat = acc / (double)L;"),
    "stat_first_element_only": ("if (statistic == 0 || statistic == 3) acc = acc + sq;", "if (statistic == 0 || statistic == 3) acc = sq;"),
    "stat_v_not_averaged": ("v[b] = (1.0 - beta2) * stat + beta2 * v[b];", "v[b] = stat;"),
}


@pytest.mark.parametrize("name", sorted(STAT_MUTANTS))
def test_statistic_mutant_is_caught(tmp_path, name):
    old, new = STAT_MUTANTS[name]
    src = open(obuild.SOURCE).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique"
    cfile = tmp_path / "mutant.c"
    cfile.write_text(src.replace(old, new))
    so = tmp_path / f"mutant_{name}.so"
    subprocess.run(["gcc", *obuild.CFLAGS, "-o", str(so), str(cfile), "-lm"], check=True)
    lib = ostep.load(str(so))
    caught = []
    for check in pins.STAT_CHECKS:
        try:
            check(lib)
        except (AssertionError, ValueError, FloatingPointError):
            caught.append(check.__name__)
    assert caught, f"no pin noticed the mutant '{name}'"


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(tmp_path, name):
    old, new = MUTANTS[name]
    src = open(obuild.SOURCE).read()
    main_end = src.index("oracle_adammini_step_stat")       # mutate Algorithm 1's routine, which comes first
    assert src[:main_end].count(old) == 1, f"mutation site for {name} not unique"
    cfile = tmp_path / "mutant.c"
    cfile.write_text(src.replace(old, new, 1))
    so = tmp_path / f"mutant_{name}.so"
    subprocess.run(["gcc", *obuild.CFLAGS, "-o", str(so), str(cfile), "-lm"], check=True)
    lib = ostep.load(str(so))
    caught = []
    for check in pins.ALL_CHECKS:
        try:
            check(lib)
        except (AssertionError, ValueError, FloatingPointError):
            caught.append(check.__name__)
    assert caught, f"no pin noticed the mutant '{name}'"
