"""AdamW with a coordinate-wise second moment -- TEST INFRASTRUCTURE ONLY.

Written separately from the Adam-mini oracle, in numpy, after the paper's
appendix algorithm "AdamW in Pytorch style".  That listing prints the decay
line with the gradient in place of the parameter; decoupled weight decay acts
on the parameter (as the Adam-mini algorithm itself prints), and that is what
this file does.  Used to pin the Adam-mini oracle: with every block of length
one, mean(g*g) = g*g and the two methods coincide.
"""
from __future__ import annotations

import math

import numpy as np


def adamw_step(p: np.ndarray, m: np.ndarray, v: np.ndarray, g: np.ndarray, *,
               lr: float, beta1: float, beta2: float, eps: float,
               weight_decay: float, step: int, apply_wd: bool = True) -> None:
    """One AdamW step in place; p, m, v, g are float64 arrays of equal size."""
    if step < 1:
        raise ValueError("step is 1-based")
    g = np.asarray(g, dtype=np.float64)
    bc1 = 1.0 - math.pow(beta1, float(step))
    bc2 = 1.0 - math.pow(beta2, float(step))
    if apply_wd:
        p -= lr * weight_decay * p
    m[:] = (1.0 - beta1) * g + beta1 * m
    v[:] = (1.0 - beta2) * (g * g) + beta2 * v
    m_hat = m / bc1
    v_hat = v / bc2
    p -= lr * m_hat / (np.sqrt(v_hat) + eps)
