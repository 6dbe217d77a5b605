"""The oracle against what the paper and the mathematics fix (no GPU)."""
import os

import numpy as np
import pytest

import oracle_pins as pins
from oracle import step as ostep

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def lib():
    return ostep.load()


@pytest.mark.parametrize("check", pins.ALL_CHECKS, ids=lambda f: f.__name__)
def test_pin(lib, check):
    check(lib)


@pytest.mark.parametrize("check", pins.STAT_CHECKS, ids=lambda f: f.__name__)
def test_statistic_variant_pin(lib, check):
    """The ablation statistics (max, min, 1-norm, 2-norm of g*g) of the paper's appendix."""
    check(lib)


def test_five_parameter_example_from_paper(lib):
    """Section 2.1 example: partition (1,2,3),(4,5); the per-block step size is
    eta / sqrt(mean of Adam's v over the block)."""
    blocks = []
    for line in open(os.path.join(GOLDEN, "example_five_parameters.txt")):
        if line.strip() and not line.startswith("#"):
            blocks.append(tuple(int(x) - 1 for x in line.split()))
    assert blocks == [(0, 1, 2), (3, 4)]
    pins.check_block_mean_of_adam_v(lib, blocks=blocks)


def test_rejects_bad_arguments(lib):
    p = np.zeros(6); m = np.zeros(6); v = np.zeros(2); g = np.zeros(6)
    with pytest.raises(ValueError):
        ostep.adammini_step(p, m, v, g, 3, step=0, **pins.HP)          # t is 1-based
    with pytest.raises(ValueError):
        ostep.adammini_step(p, m, np.zeros(1), g, 4, step=1, **pins.HP)  # L must divide numel
