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
