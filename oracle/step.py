"""ctypes front end of the C oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

`adammini_step` runs Algorithm 1 (Adam-mini, general form) for one tensor;
`OracleState` keeps the float64 state of a list of tensors across steps.
"""
from __future__ import annotations

import ctypes
from typing import Sequence

import numpy as np

from . import build as _build

G_F32, G_BF16, G_F64 = 0, 1, 2

_lib = None


def load(path: str | None = None) -> ctypes.CDLL:
    """Load (building if needed) the oracle's shared object."""
    global _lib
    if path is None and _lib is not None:
        return _lib
    lib = ctypes.CDLL(path or _build.build())
    lib.oracle_adammini_step.restype = ctypes.c_int
    lib.oracle_adammini_step.argtypes = [
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
        ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double,
        ctypes.c_double, ctypes.c_int, ctypes.c_int64,
    ]
    lib.oracle_adammini_step_stat.restype = ctypes.c_int
    lib.oracle_adammini_step_stat.argtypes = lib.oracle_adammini_step.argtypes + [ctypes.c_int]
    lib.oracle_widen_f32.restype = None
    lib.oracle_widen_f32.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]
    lib.oracle_widen_bf16.restype = None
    lib.oracle_widen_bf16.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]
    if path is None:
        _lib = lib
    return lib


def _grad_view(g) -> tuple[np.ndarray, int]:
    """Return (contiguous numpy array, dtype code) for a gradient.

    Accepts numpy float32/float64, numpy uint16 (bfloat16 bit patterns), or a
    CPU torch tensor of dtype float32/bfloat16/float64.
    """
    if not isinstance(g, np.ndarray):  # torch tensor, without importing torch here
        name = str(g.dtype)
        if name == "torch.bfloat16":
            import torch

            g = g.contiguous().view(torch.int16).numpy().view(np.uint16)
        else:
            g = g.contiguous().numpy()
    g = np.ascontiguousarray(g).reshape(-1)
    if g.dtype == np.float32:
        return g, G_F32
    if g.dtype == np.uint16:
        return g, G_BF16
    if g.dtype == np.float64:
        return g, G_F64
    raise TypeError(f"unsupported gradient dtype {g.dtype}")


def adammini_step(p: np.ndarray, m: np.ndarray, v: np.ndarray, g, block_len: int, *,
                  lr: float, beta1: float, beta2: float, eps: float,
                  weight_decay: float, step: int, apply_wd: bool = True,
                  lib: ctypes.CDLL | None = None, statistic: int = 0) -> None:
    """One Adam-mini step (Algorithm 1) on one tensor, in place, float64 state.

    statistic != 0 selects the ablation variants of the block statistic
    (1 max, 2 min, 3 one-norm, 4 two-norm of g*g), a separate C routine."""
    lib = lib or load()
    for a in (p, m, v):
        if a.dtype != np.float64 or not a.flags.c_contiguous:
            raise TypeError("oracle state must be contiguous float64")
    gv, code = _grad_view(g)
    n = p.size
    if m.size != n or gv.size != n or n % block_len or v.size != n // block_len:
        raise ValueError("shape mismatch")
    args = (p.ctypes.data, m.ctypes.data, v.ctypes.data, gv.ctypes.data, code, n,
            int(block_len), float(lr), float(beta1), float(beta2), float(eps),
            float(weight_decay), int(bool(apply_wd)), int(step))
    if statistic:
        rc = lib.oracle_adammini_step_stat(*args, int(statistic))
    else:
        rc = lib.oracle_adammini_step(*args)
    if rc != 0:
        raise ValueError(f"oracle_adammini_step rejected its arguments (rc={rc})")


def widen(x) -> np.ndarray:
    """Exact widening of float32 / bfloat16 data (numpy or CPU torch) to float64."""
    lib = load()
    xv, code = _grad_view(x)
    out = np.empty(xv.size, dtype=np.float64)
    if code == G_F32:
        lib.oracle_widen_f32(xv.ctypes.data, out.ctypes.data, xv.size)
    elif code == G_BF16:
        lib.oracle_widen_bf16(xv.ctypes.data, out.ctypes.data, xv.size)
    else:
        out[:] = xv
    return out


class OracleState:
    """Float64 state (p, m, v) of several tensors, stepped with the C oracle.

    `block_lens[i]` is the block length of tensor i; `wd_flags[i]` says whether
    the decay line applies to it.  m and v start at zero.
    """

    def __init__(self, params: Sequence, block_lens: Sequence[int],
                 wd_flags: Sequence[bool] | None = None):
        self.p = [widen(x) for x in params]
        self.block_lens = [int(b) for b in block_lens]
        self.wd_flags = list(wd_flags) if wd_flags is not None else [True] * len(self.p)
        self.m = [np.zeros_like(x) for x in self.p]
        self.v = [np.zeros(x.size // b, dtype=np.float64)
                  for x, b in zip(self.p, self.block_lens)]

    def step(self, grads: Sequence, step: int, **hp) -> None:
        for i, g in enumerate(grads):
            adammini_step(self.p[i], self.m[i], self.v[i], g, self.block_lens[i],
                          step=step, apply_wd=self.wd_flags[i], **hp)
