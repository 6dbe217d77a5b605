"""Pin checks for the float64 oracle, each written against something other than
the oracle itself: a separately written AdamW, closed forms, invariants of the
update rule, exact rational arithmetic on tiny cases.

Every check takes the loaded oracle library, so the same checks can be pointed
at deliberately broken copies of the oracle (see test_oracle_mutants.py).
"""
from __future__ import annotations

import itertools
import math
from fractions import Fraction

import numpy as np

from oracle import adamw_ref, exact, partition_ref, step as ostep

HP = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


def run(lib, p0, g_steps, L, hp=HP, apply_wd=True):
    """Run the oracle over len(g_steps) steps; returns float64 p, m, v."""
    p = np.array(p0, dtype=np.float64)
    m = np.zeros_like(p)
    v = np.zeros(p.size // L, dtype=np.float64)
    for t, g in enumerate(g_steps, start=1):
        ostep.adammini_step(p, m, v, np.asarray(g, dtype=np.float64), L, step=t,
                            apply_wd=apply_wd, lib=lib, **hp)
    return p, m, v


def _rel(a, b, floor=1e-300):
    a, b = np.asarray(a, float), np.asarray(b, float)
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), floor))) if a.size else 0.0


# -- P1: block length 1 is AdamW, bit for bit (paper: Adam-mini "replaces g*g by
#    its mean"; the mean of one element is that element) -----------------------
def check_reduces_to_adamw(lib):
    rng = np.random.default_rng(11)
    n = 257
    p0 = rng.normal(0, 0.02, n)
    gs = [rng.normal(0, 1, n) * 10.0 ** rng.uniform(-4, 0, n) for _ in range(7)]
    gs[3][::5] = 0.0
    p, m, v = run(lib, p0, gs, 1)
    pa, ma, va = p0.copy(), np.zeros(n), np.zeros(n)
    for t, g in enumerate(gs, start=1):
        adamw_ref.adamw_step(pa, ma, va, g, step=t, **HP)
    assert np.array_equal(p.view(np.int64), pa.view(np.int64))
    assert np.array_equal(m.view(np.int64), ma.view(np.int64))
    assert np.array_equal(v.view(np.int64), va.view(np.int64))


# -- I1 / five-parameter example: v_b is the block mean of AdamW's v, m is
#    AdamW's m, and the step uses eta / sqrt(mean of Adam's v over the block) ---
def check_block_mean_of_adam_v(lib, blocks=((0, 1, 2), (3, 4))):
    rng = np.random.default_rng(5)
    n = sum(len(b) for b in blocks)
    p0 = rng.normal(0, 0.02, n)
    T = 6
    gs = [rng.normal(0, 1, n) * np.array([1e-3, 1.0, 30.0, 0.2, 5e-2][:n]) for _ in range(T)]
    # Adam-mini: every block is its own tensor (blocks here differ in length)
    state = []
    for idx in blocks:
        idx = list(idx)
        state.append([p0[idx].copy(), np.zeros(len(idx)), np.zeros(1)])
    pa, ma, va = p0.copy(), np.zeros(n), np.zeros(n)
    for t, g in enumerate(gs, start=1):
        p_before = [s[0].copy() for s in state]
        adamw_ref.adamw_step(pa, ma, va, g, step=t, **HP)
        for s, idx in zip(state, blocks):
            idx = list(idx)
            ostep.adammini_step(s[0], s[1], s[2], g[idx], len(idx), step=t, lib=lib, **HP)
        for s, idx, pb in zip(state, blocks, p_before):
            idx = list(idx)
            assert np.array_equal(s[1], ma[idx])                       # m is Adam's m
            assert _rel(s[2][0], va[idx].mean()) < 1e-13               # v_b = mean of Adam's v
            bc1 = 1 - HP["beta1"] ** t
            bc2 = 1 - HP["beta2"] ** t
            u_mini = HP["lr"] / (math.sqrt(va[idx].mean() / bc2) + HP["eps"])
            want = pb * (1 - HP["lr"] * HP["weight_decay"]) - u_mini * ma[idx] / bc1
            assert _rel(s[0], want) < 1e-12


# -- P2: constant gradient.  m_hat = g and v_hat = mean(g_b^2) at every step, so
#    with a = 1 - eta*lambda and c_i = g_i / (rms(g_b) + eps):
#    p_T = a^T p_0 - eta c_i (1 - a^T) / (1 - a) --------------------------------
def check_constant_gradient_closed_form(lib):
    rng = np.random.default_rng(3)
    L, nb, T = 6, 4, 25
    p0 = rng.normal(0, 0.02, L * nb)
    g = rng.normal(0, 1, L * nb) * np.repeat(10.0 ** rng.uniform(-3, 1, nb), L)
    p, m, v = run(lib, p0, [g] * T, L)
    ms = (g.reshape(nb, L) ** 2).mean(axis=1)
    a = 1 - HP["lr"] * HP["weight_decay"]
    c = g / (np.repeat(np.sqrt(ms), L) + HP["eps"])
    want = a ** T * p0 - HP["lr"] * c * (1 - a ** T) / (1 - a)
    assert _rel(p, want) < 1e-11
    assert _rel(m, g * (1 - HP["beta1"] ** T)) < 1e-12
    assert _rel(v, ms * (1 - HP["beta2"] ** T)) < 1e-12
    # lambda = 0: p_T = p_0 - T eta c_i
    hp0 = dict(HP, weight_decay=0.0)
    p, _, _ = run(lib, p0, [g] * T, L, hp=hp0)
    assert _rel(p, p0 - T * HP["lr"] * c) < 1e-11
    # decay switched off per tensor behaves like lambda = 0
    p2, _, _ = run(lib, p0, [g] * T, L, apply_wd=False)
    assert np.array_equal(p, p2)


# -- P2': zero gradient.  m = v = 0 and the Adam term is 0/(0+eps) = 0 ----------
def check_zero_gradient(lib):
    p0 = np.linspace(-1, 1, 12)
    T = 9
    p, m, v = run(lib, p0, [np.zeros(12)] * T, 4)
    assert not m.any() and not v.any()
    assert _rel(p, (1 - HP["lr"] * HP["weight_decay"]) ** T * p0) < 1e-14


# -- I2, I3: the first step, p_1 = a p_0 - eta g / (rms(g_b) + eps); if |g| = c on
#    the block the Adam term is eta sign(g) c / (c + eps) ------------------------
def check_first_step(lib):
    rng = np.random.default_rng(8)
    L, nb = 8, 3
    p0 = rng.normal(0, 0.02, L * nb)
    g = rng.normal(0, 2, L * nb)
    p, m, v = run(lib, p0, [g], L)
    rms = np.repeat(np.sqrt((g.reshape(nb, L) ** 2).mean(axis=1)), L)
    a = 1 - HP["lr"] * HP["weight_decay"]
    assert _rel(p, a * p0 - HP["lr"] * g / (rms + HP["eps"])) < 1e-12
    c = 0.37
    s = np.sign(rng.normal(size=L * nb))
    p, _, _ = run(lib, p0, [c * s], L)
    assert _rel(p, a * p0 - HP["lr"] * s * c / (c + HP["eps"])) < 1e-12
    # eps sits outside the root: with a large eps the step is eta g / (rms + eps)
    hp = dict(HP, eps=0.5)
    p, _, _ = run(lib, p0, [g], L, hp=hp)
    assert _rel(p, a * p0 - HP["lr"] * g / (rms + 0.5)) < 1e-12


# -- I4: scaling a block's gradients by k > 0 leaves p unchanged as eps -> 0 -----
def check_scale_invariance(lib):
    rng = np.random.default_rng(21)
    L, nb, T = 5, 3, 6
    hp = dict(HP, eps=1e-300)
    p0 = rng.normal(0, 0.02, L * nb)
    gs = [rng.normal(0, 1, L * nb) for _ in range(T)]
    k = np.repeat([1.0, 1024.0, 2.0 ** -20], L)          # powers of two: exact scaling
    p_a, _, _ = run(lib, p0, gs, L, hp=hp)
    p_b, _, _ = run(lib, p0, [g * k for g in gs], L, hp=hp)
    assert _rel(p_b, p_a) < 1e-13


# -- I5: permuting elements inside blocks permutes m and p and leaves v ---------
def check_permutation_invariance(lib):
    rng = np.random.default_rng(22)
    L, nb, T = 7, 4, 5
    p0 = rng.normal(0, 0.02, L * nb)
    gs = [rng.normal(0, 1, L * nb) for _ in range(T)]
    perm = np.concatenate([b * L + rng.permutation(L) for b in range(nb)])
    p_a, m_a, v_a = run(lib, p0, gs, L)
    p_b, m_b, v_b = run(lib, p0[perm], [g[perm] for g in gs], L)
    assert _rel(v_b, v_a) < 1e-14
    assert _rel(p_b, p_a[perm]) < 1e-12
    assert np.array_equal(m_b, m_a[perm])


# -- I6: blocks evolve independently ---------------------------------------------
def check_block_independence(lib):
    rng = np.random.default_rng(23)
    L, nb, T = 4, 5, 4
    p0 = rng.normal(0, 0.02, L * nb)
    gs = [rng.normal(0, 1, L * nb) for _ in range(T)]
    gs2 = [g.copy() for g in gs]
    for g in gs2:
        g[2 * L:3 * L] *= -3.0                              # disturb block 2 only
    a = run(lib, p0, gs, L)
    b = run(lib, p0, gs2, L)
    keep = np.ones(L * nb, bool)
    keep[2 * L:3 * L] = False
    assert np.array_equal(a[0][keep], b[0][keep]) and np.array_equal(a[1][keep], b[1][keep])
    assert np.array_equal(np.delete(a[2], 2), np.delete(b[2], 2))
    assert not np.array_equal(a[0][~keep], b[0][~keep])
    # a tensor run alone equals the same blocks run inside a longer tensor
    c = run(lib, p0[L:3 * L], [g[L:3 * L] for g in gs], L)
    assert np.array_equal(c[0], a[0][L:3 * L]) and np.array_equal(c[2], a[2][1:3])


# -- P4: brute force against exact rational arithmetic ---------------------------
GRAD_VALUES = (-2.0, -0.5, 0.0, 0.25, 1.5)


def _compare_exact(lib, p0, g_steps, L):
    n = len(p0)
    p, m, v = run(lib, p0, g_steps, L)
    descs = [partition_ref.TensorDesc(1, n, partition_ref.FIXED, fixed_block_len=L)]
    blocks = partition_ref.blocks_as_index_lists(descs)
    pe, me, ve = exact.adammini_exact(p0, g_steps, blocks, **HP)
    for got, want in ((p, pe), (m, me), (v, ve)):
        for x, y in zip(got, want):
            y = float(y)
            assert abs(x - y) <= 4e-15 * max(abs(y), 1e-3 if got is p else 0.0) + 1e-300, (x, y, L, g_steps)


def check_brute_force_exact(lib):
    # every gradient pattern on up to 4 elements, every divisor as block length
    for n in (1, 2, 3, 4):
        p0 = [0.02 * ((-1) ** i) * (i + 1) for i in range(n)]
        for L in [d for d in range(1, n + 1) if n % d == 0]:
            for g in itertools.product(GRAD_VALUES, repeat=n):
                _compare_exact(lib, p0, [list(g)], L)
    # three steps on up to 12 elements, every divisor, sampled patterns
    rng = np.random.default_rng(99)
    for n in (6, 8, 12):
        p0 = list(rng.normal(0, 0.02, n))
        for L in [d for d in range(1, n + 1) if n % d == 0]:
            for _ in range(6):
                gs = [list(rng.choice(GRAD_VALUES, n)) for _ in range(3)]
                _compare_exact(lib, p0, gs, L)


# -- widening: bfloat16 / float32 bits reach the oracle exactly ------------------
def check_widening(lib):
    import ctypes
    bits = np.arange(65536, dtype=np.uint16)
    out = np.empty(65536, dtype=np.float64)
    lib.oracle_widen_bf16(bits.ctypes.data, out.ctypes.data, 65536)
    with np.errstate(invalid="ignore"):
        want = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ok = ~np.isnan(want)
    assert np.array_equal(out[ok], want[ok]) and np.isnan(out[~ok]).all()
    # the step reads bf16 gradients as those values: 1.0 is 0x3F80, -2.5 is 0xC020
    p = np.zeros(2); m = np.zeros(2); v = np.zeros(1)
    g = np.array([0x3F80, 0xC020], dtype=np.uint16)
    ostep.adammini_step(p, m, v, g, 2, step=1, lib=lib, **HP)
    assert _rel(m, [0.1, -0.25]) < 1e-15 and _rel(v, [0.05 * (1 + 6.25) / 2]) < 1e-15
    g32 = np.array([1.0, -2.5], dtype=np.float32)
    p2 = np.zeros(2); m2 = np.zeros(2); v2 = np.zeros(1)
    ostep.adammini_step(p2, m2, v2, g32, 2, step=1, lib=lib, **HP)
    assert np.array_equal(p, p2) and np.array_equal(m, m2) and np.array_equal(v, v2)
    # float32 gradients keep all 24 significant bits: values bfloat16 cannot hold, a denormal,
    # the largest finite float; numpy's own conversion to float64 is the reference
    g32 = np.array([1.0 + 2.0 ** -23, np.pi, -1.0 / 3.0, 1e-30, 1.4e-45, 3.4028235e38, -7.0e-5, 123456.789],
                   dtype=np.float32)
    pa = np.linspace(-1.0, 1.0, 8); ma = np.zeros(8); va = np.zeros(2)
    pb = pa.copy(); mb = np.zeros(8); vb = np.zeros(2)
    for t in (1, 2):
        ostep.adammini_step(pa, ma, va, g32, 4, step=t, lib=lib, **HP)
        ostep.adammini_step(pb, mb, vb, g32.astype(np.float64), 4, step=t, lib=lib, **HP)
    assert np.array_equal(pa, pb) and np.array_equal(ma, mb) and np.array_equal(va, vb)
    assert ma[0] - 0.19 > 1e-8                                  # m = 0.19 * (1 + 2^-23): the last bit of g is there
    rng = np.random.default_rng(5)
    bits32 = rng.integers(0, 1 << 32, 4096, dtype=np.uint64).astype(np.uint32)
    src = bits32.view(np.float32)
    out32 = np.empty(4096, dtype=np.float64)
    lib.oracle_widen_f32(src.ctypes.data, out32.ctypes.data, 4096)
    with np.errstate(invalid="ignore"):
        want32 = src.astype(np.float64)
    ok = ~np.isnan(want32)
    assert np.array_equal(out32[ok], want32[ok]) and np.isnan(out32[~ok]).all()
    del ctypes


ALL_CHECKS = (
    check_reduces_to_adamw,
    check_block_mean_of_adam_v,
    check_constant_gradient_closed_form,
    check_zero_gradient,
    check_first_step,
    check_scale_invariance,
    check_permutation_invariance,
    check_block_independence,
    check_brute_force_exact,
    check_widening,
)


# =============================================================================
# The ablation variants of the block statistic (max, min, 1-norm, 2-norm of g*g)
# =============================================================================
STATS = (1, 2, 3, 4)


def run_stat(lib, p0, g_steps, L, statistic, hp=HP):
    p = np.array(p0, dtype=np.float64)
    m = np.zeros_like(p)
    v = np.zeros(p.size // L, dtype=np.float64)
    for t, g in enumerate(g_steps, start=1):
        ostep.adammini_step(p, m, v, np.asarray(g, dtype=np.float64), L, step=t, lib=lib,
                            statistic=statistic, **hp)
    return p, m, v


# -- with one element per block every statistic of {g*g} is g*g: AdamW again, bit for bit
#    (sqrt(x*x) = |x| exactly in IEEE arithmetic, so this holds for the 2-norm too) --------
def check_stat_reduces_to_adamw(lib):
    rng = np.random.default_rng(31)
    n = 129
    p0 = rng.normal(0, 0.02, n)
    gs = [rng.normal(0, 1, n) * 10.0 ** rng.uniform(-3, 0, n) for _ in range(5)]
    pa, ma, va = p0.copy(), np.zeros(n), np.zeros(n)
    for t, g in enumerate(gs, start=1):
        adamw_ref.adamw_step(pa, ma, va, g, step=t, **HP)
    for s in STATS:
        p, m, v = run_stat(lib, p0, gs, 1, s)
        assert np.array_equal(p, pa) and np.array_equal(m, ma) and np.array_equal(v, va), s


# -- |g| = c on a block: max = min = c^2, 1-norm = L c^2, 2-norm = sqrt(L) c^2, constant in t,
#    so v_hat = k c^2 and p_T = a^T p_0 - eta sign(g) c / (sqrt(k) c + eps) (1-a^T)/(1-a) -------
def check_stat_closed_form(lib):
    rng = np.random.default_rng(32)
    L, nb, T = 9, 3, 12
    p0 = rng.normal(0, 0.02, L * nb)
    c = np.repeat([0.5, 3e-3, 7.0], L)
    sgn = np.sign(rng.normal(size=L * nb))
    g = c * sgn
    a = 1 - HP["lr"] * HP["weight_decay"]
    for s, k in ((1, 1.0), (2, 1.0), (3, float(L)), (4, math.sqrt(L))):
        p, m, v = run_stat(lib, p0, [g] * T, L, s)
        assert _rel(v, k * c[::L] ** 2 * (1 - HP["beta2"] ** T)) < 1e-12, s
        want = a ** T * p0 - HP["lr"] * sgn * c / (math.sqrt(k) * c + HP["eps"]) * (1 - a ** T) / (1 - a)
        assert _rel(p, want) < 1e-11, s


# -- against numpy on random data: the EMA of numpy's own max / min / sum / 2-norm --------
def check_stat_against_numpy(lib):
    rng = np.random.default_rng(33)
    L, nb, T = 16, 5, 6
    p0 = rng.normal(0, 0.02, L * nb)
    gs = [rng.normal(0, 1, L * nb) for _ in range(T)]
    fns = {1: lambda q: q.max(axis=1), 2: lambda q: q.min(axis=1), 3: lambda q: q.sum(axis=1),
           4: lambda q: np.sqrt((q * q).sum(axis=1))}
    v_mean = run(lib, p0, gs, L)[2]
    for s in STATS:
        p, m, v = run_stat(lib, p0, gs, L, s)
        want = np.zeros(nb)
        for g in gs:
            want = (1 - HP["beta2"]) * fns[s]((g * g).reshape(nb, L)) + HP["beta2"] * want
        assert _rel(v, want) < 1e-13, s
        # the last step's parameter change uses eta m_hat / (sqrt(v_hat) + eps)
        p_prev, m_prev, _ = run_stat(lib, p0, gs[:-1], L, s)
        m_new = (1 - HP["beta1"]) * gs[-1] + HP["beta1"] * m_prev
        denom = np.repeat(np.sqrt(want / (1 - HP["beta2"] ** T)), L) + HP["eps"]
        expect = p_prev * (1 - HP["lr"] * HP["weight_decay"]) - HP["lr"] * (m_new / (1 - HP["beta1"] ** T)) / denom
        assert _rel(p, expect) < 1e-12, s
    v_max, v_min = run_stat(lib, p0, gs, L, 1)[2], run_stat(lib, p0, gs, L, 2)[2]
    assert (v_max >= v_mean).all() and (v_mean >= v_min).all()
    assert np.array_equal(run_stat(lib, p0, gs, L, 3)[2], L * v_mean)        # L = 16: scaling by L is exact


def check_stat_brute_force_exact(lib):
    rng = np.random.default_rng(34)
    for s in STATS:
        for n in (2, 3, 4, 6):
            p0 = list(rng.normal(0, 0.02, n))
            for L in [d for d in range(1, n + 1) if n % d == 0]:
                for _ in range(8):
                    gs = [list(rng.choice(GRAD_VALUES, n)) for _ in range(2)]
                    p, m, v = run_stat(lib, p0, gs, L, s)
                    blocks = [list(range(b * L, (b + 1) * L)) for b in range(n // L)]
                    pe, me, ve = exact.adammini_exact(p0, gs, blocks, statistic=s, **HP)
                    for got, want, floor in ((p, pe, 1e-3), (m, me, 0.0), (v, ve, 0.0)):
                        for x, y in zip(got, want):
                            y = float(y)
                            assert abs(x - y) <= 4e-15 * max(abs(y), floor) + 1e-300, (s, L, gs)


STAT_CHECKS = (check_stat_reduces_to_adamw, check_stat_closed_form, check_stat_against_numpy,
               check_stat_brute_force_exact)
