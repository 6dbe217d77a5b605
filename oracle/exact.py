"""Exact-rational Adam-mini for tiny cases -- TEST INFRASTRUCTURE ONLY.

A literal, loop-by-loop transcription of Algorithm 1 (Adam-mini, general form)
over `fractions.Fraction`, so that every product, sum, mean and moving average
is exact.  The one irrational step, the square root of v_hat, is taken to
`SQRT_BITS` correct bits with integer arithmetic.  Brute-force tests compare
the float64 C oracle with this on all small cases they can enumerate.
"""
from __future__ import annotations

from fractions import Fraction
from math import isqrt
from typing import List, Sequence

SQRT_BITS = 256


def sqrt_fraction(x: Fraction, bits: int = SQRT_BITS) -> Fraction:
    """Square root of a non-negative rational, truncated to 2**-bits relative."""
    if x < 0:
        raise ValueError("negative radicand")
    if x == 0:
        return Fraction(0)
    # scale so the integer root carries `bits` significant bits
    shift = bits + max(0, x.denominator.bit_length() - x.numerator.bit_length())
    shift += shift & 1
    scaled = (x.numerator << shift) // x.denominator
    return Fraction(isqrt(scaled), 1 << (shift // 2))


def block_statistic(squares: Sequence[Fraction], statistic: int) -> Fraction:
    """mean (0), max (1), min (2), sum (3) or 2-norm (4) of a block's g*g values."""
    if statistic == 0:
        return sum(squares, Fraction(0)) / len(squares)
    if statistic == 1:
        return max(squares)
    if statistic == 2:
        return min(squares)
    if statistic == 3:
        return sum(squares, Fraction(0))
    if statistic == 4:
        return sqrt_fraction(sum((x * x for x in squares), Fraction(0)))
    raise ValueError("unknown statistic")


def adammini_exact(p: Sequence, g_steps: Sequence[Sequence], blocks: Sequence[Sequence[int]], *,
                   lr, beta1, beta2, eps, weight_decay,
                   statistic: int = 0) -> tuple[List[Fraction], List[Fraction], List[Fraction]]:
    """Run len(g_steps) Adam-mini steps exactly.

    p: initial parameters; g_steps[t-1][i]: gradient of element i at step t;
    blocks: a partition of range(len(p)) given as lists of element indices.
    Every number is converted with Fraction(), so floats are taken at their
    exact binary value.  Returns (p, m, v) with one v per block.
    """
    F = Fraction
    lr, beta1, beta2, eps, lam = F(lr), F(beta1), F(beta2), F(eps), F(weight_decay)
    p = [F(x) for x in p]
    m = [F(0)] * len(p)
    v = [F(0)] * len(blocks)
    for t, g in enumerate(g_steps, start=1):
        g = [F(x) for x in g]
        for b, idx in enumerate(blocks):
            mean_sq = block_statistic([g[i] * g[i] for i in idx], statistic)
            for i in idx:
                p[i] = p[i] - lr * lam * p[i]
                m[i] = (1 - beta1) * g[i] + beta1 * m[i]
            v[b] = (1 - beta2) * mean_sq + beta2 * v[b]
            v_hat = v[b] / (1 - beta2 ** t)
            root = sqrt_fraction(v_hat)
            for i in idx:
                m_hat = m[i] / (1 - beta1 ** t)
                p[i] = p[i] - lr * m_hat / (root + eps)
    return p, m, v
