"""The acceptance metric itself (no GPU): an element is measured against its own
block and nothing else."""
import numpy as np
import pytest

import harness as H


def test_scale_is_the_elements_own_block():
    # two blocks of four: a quiet one (1e-4) next to a loud one (1e-1)
    want = np.array([1e-4, -1e-4, 1e-4, -1e-4, 1e-1, -1e-1, 1e-1, -1e-1])
    got = want.copy()
    got[0] += 1e-8                                   # 1e-4 of the quiet block's own scale
    assert H.block_relative_error(got, want, 4) == pytest.approx(1e-4, rel=1e-6)
    got = want.copy()
    got[4] += 1e-8                                   # the same absolute error in the loud block: 1e-7
    assert H.block_relative_error(got, want, 4) == pytest.approx(1e-7, rel=1e-6)


def test_an_element_near_zero_is_measured_against_its_blocks_rms():
    want = np.array([1e-12, 3.0, -4.0, 0.0])         # rms = 2.5
    got = want + np.array([2.5e-6, 0.0, 0.0, 2.5e-6])
    err, k, scale = H.block_error_detail(got, want, 4)
    assert err == pytest.approx(1e-6, rel=1e-6) and k in (0, 3) and scale == pytest.approx(2.5)


def test_non_finite_values_must_match():
    want = np.array([1.0, np.inf, np.nan, 2.0])
    assert H.block_relative_error(want.copy(), want, 4) == 0.0
    bad = want.copy()
    bad[1] = 1.0
    assert H.block_relative_error(bad, want, 4) == float("inf")
    bad = want.copy()
    bad[1] = -np.inf
    assert H.block_relative_error(bad, want, 4) == float("inf")


def test_floor_is_only_for_blocks_too_short_for_a_scale_of_their_own():
    want = np.array([1e-9, 2e-9])
    got = want + 1e-12
    floor = np.array([1e-3, 1e-3])
    assert H.block_relative_error(got, want, 1) > 1e-4              # pure ratio
    assert H.block_relative_error(got, want, 1, floor) == pytest.approx(1e-9, rel=1e-6)
    assert H.block_relative_error(got, want, 2, floor) == pytest.approx(1e-9, rel=1e-6)
    with pytest.raises(AssertionError):
        H.block_relative_error(np.zeros(8), np.zeros(8), 4, np.ones(8))


def test_short_block_scale_follows_one_elements_operands():
    s = H.ShortBlockScale(np.array([0.02, -0.5]))
    g = np.array([1.0, -2.0])
    m = 0.1 * g
    s.update(g, np.array([0.019, -0.49]), m, 0.9)
    assert np.allclose(s.m, [0.1, 0.2]) and np.allclose(s.p, [0.02, 0.5])
    # the next gradient cancels m exactly: the scale stays at the operands' size
    g2 = -0.9 * m / 0.1
    s.update(g2, np.array([1e-9, 0.6]), np.zeros(2), 0.9)
    assert np.allclose(s.m, 0.1 * np.abs(g2) + 0.9 * np.array([0.1, 0.2]))
    assert np.allclose(s.p, [0.02, 0.6])
