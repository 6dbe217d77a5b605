"""Shared test machinery: run a workload through the CUDA library and through
the float64 oracle on the same seeded inputs, and compare.

The comparison follows the acceptance rule for this library: for p and m the
error of element i is |gpu_i - oracle_i| / max(|oracle_i|, rms of the oracle's
values over i's block); for v it is the plain relative error with an absolute
floor.  The bound is 1e-5 (float32 arithmetic against float64; rounding errors
add up but do not feed back because the synthetic gradients do not depend on
the parameters).
"""
from __future__ import annotations

import concurrent.futures as cf
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

import paper_2406_16793_b200 as am
from oracle import step as ostep
from paper_2406_16793_b200 import build as _lib_build, workloads as W

_lib_build.build()      # compile the CUDA library if the shared object is missing or older than its sources

TOL = 1e-5
GUARD = 64          # float32 guard words either side of every test buffer
SENTINEL = -7.0e33


OWN_SCALE_MIN_L = 4     # blocks shorter than this also get the per-element floor of ShortBlockScale


def block_error_detail(got: np.ndarray, want: np.ndarray, L: int, floor: Optional[np.ndarray] = None):
    """(max_i |got_i - want_i| / max(|want_i|, rms of want over i's OWN block), index of that element,
    its scale); NaN/inf must match (else the error is inf).

    The scale of an element is taken from its own block only, never from a
    neighbouring block.  Blocks of fewer than OWN_SCALE_MIN_L elements have no
    dependable scale of their own (every element of such a block can come out of
    a cancellation at once, and a one-element block has nothing but the element
    itself); for those the caller passes `floor`, a per-element magnitude of the
    operands the entry was computed from (see ShortBlockScale), and the scale is
    max(|want_i|, block rms, floor_i)."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    if want.size == 0:
        return 0.0, -1, 0.0
    fin = np.isfinite(want)
    if not np.array_equal(fin, np.isfinite(got)):
        return float("inf"), int(np.argmax(fin != np.isfinite(got))), 0.0
    if not fin.all():
        same = np.where(fin, True, (np.isnan(want) & np.isnan(got)) | (want == got))
        if not same.all():
            return float("inf"), int(np.argmin(same)), 0.0
    w = np.where(fin, want, 0.0)
    assert w.size % L == 0
    if L == 1:
        scale = np.abs(w)
    else:
        rms = np.sqrt((w.reshape(-1, L) ** 2).mean(axis=1))
        scale = np.maximum(np.abs(w), np.repeat(rms, L))
    if floor is not None:
        assert L < OWN_SCALE_MIN_L, "the floor is for blocks too short to have a scale of their own"
        f = np.asarray(floor, dtype=np.float64).reshape(-1)
        scale = np.maximum(scale, np.where(np.isfinite(f), f, 0.0))
    scale = np.where(scale > 0, scale, 1.0)
    err = np.where(fin, np.abs(got - w) / scale, 0.0)
    k = int(err.argmax())
    return float(err[k]), k, float(scale[k])


def block_relative_error(got: np.ndarray, want: np.ndarray, L: int, floor: Optional[np.ndarray] = None) -> float:
    return block_error_detail(got, want, L, floor)[0]


class ShortBlockScale:
    """Error scale for the elements of blocks of fewer than OWN_SCALE_MIN_L
    elements, each element from its own history.

    An element's m (or p) can pass through zero: m_t = (1-beta1) g_t + beta1 m_{t-1}
    with operands of opposite sign.  float32 then carries an absolute error of the
    order of an ulp of the OPERANDS, so the ratio to |m_t| says nothing about the
    arithmetic; in a block of one, two or three elements all of them can do so at
    once (the seeded tests hold two-element blocks whose two entries of m are both below
    1e-2 of their operands), and the block's RMS is then no better a scale.  The scale kept here is the magnitude of those operands,
    followed along the oracle's own trajectory of that element:
        S_m(t) = max(|m_t|, (1-beta1)|g_t| + beta1 S_m(t-1)),  S_m(0) = 0
        S_p(t) = max(|p_t|, S_p(t-1)),                         S_p(0) = |p_0|
    (rounding errors of earlier steps stay in the state, scaled by beta1 for m
    and by 1 - eta*lambda, about one, for p).  No other element enters."""

    def __init__(self, p0: np.ndarray):
        self.p = np.abs(np.asarray(p0, dtype=np.float64)).copy()
        self.m = np.zeros_like(self.p)

    def update(self, g64: np.ndarray, p: np.ndarray, m: np.ndarray, beta1: float) -> None:
        with np.errstate(invalid="ignore"):
            self.m = np.maximum(np.abs(m), (1.0 - beta1) * np.abs(g64) + beta1 * self.m)
            self.p = np.maximum(self.p, np.abs(p))


def v_relative_error(got: np.ndarray, want: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    fin = np.isfinite(want)
    if not np.array_equal(fin, np.isfinite(got)):
        return float("inf")
    with np.errstate(invalid="ignore"):
        d = np.abs(got - want)[fin]
    return float((d / np.maximum(np.abs(want[fin]), 1e-30)).max()) if d.size else 0.0


class Guarded:
    """A device tensor with sentinel-filled guard zones before and after it."""

    def __init__(self, numel: int, dtype: torch.dtype, device):
        item = torch.empty((), dtype=dtype).element_size()
        self.guard = GUARD * 4 // item
        pad = (-numel) % (16 // item)          # keep the rear guard 16-byte aligned too
        self.raw = torch.full((numel + pad + 2 * self.guard,), SENTINEL, dtype=dtype, device=device)
        self.view = self.raw[self.guard:self.guard + numel]
        self.numel = numel

    def intact(self) -> bool:
        front = self.raw[:self.guard]
        back = self.raw[self.guard + self.numel:]
        ref = torch.full((1,), SENTINEL, dtype=self.raw.dtype, device=self.raw.device)
        return bool((front == ref).all() and (back == ref).all())


class DeviceState:
    """Parameters, moments and gradient buffers of a workload on the GPU."""

    def __init__(self, w: W.Workload, device="cuda", guarded: bool = True):
        self.w = w
        self.device = device
        self.guards: List[Guarded] = []

        def alloc(n, dtype):
            if guarded:
                g = Guarded(n, dtype, device)
                self.guards.append(g)
                return g.view
            return torch.empty(n, dtype=dtype, device=device)

        self.p, self.m, self.g = [], [], []
        for i, t in enumerate(w.tensors):
            p = alloc(t.numel, torch.float32)
            p.copy_(W.gen_param(w, i, device))
            m = alloc(t.numel, torch.float32)
            m.zero_()
            g = alloc(t.numel, W.torch_dtype(t.grad_dtype))
            g.zero_()
            self.p.append(p); self.m.append(m); self.g.append(g)
        self.v = alloc(max(w.n_blocks, 1), torch.float32)
        self.v.zero_()
        self.sigmas = [W.row_sigmas(w, i, device) for i in range(len(w.tensors))]

    def draw_grads(self, step: int) -> None:
        for i in range(len(self.w.tensors)):
            W.gen_grad(self.w, i, step, self.device, out=self.g[i], sigmas=self.sigmas[i])

    def guards_intact(self) -> bool:
        return all(g.intact() for g in self.guards)


def mixed_workload():
    """Every kernel family at once: tiny blocks, packed rows, long rows (aligned and not), a clustered head, a two-pass block."""
    T = W.TensorSpec
    bf = dict(grad_dtype=W.BF16)
    tensors = [
        T("tiny", 1, 4096, W.FIXED, fixed_block_len=1, **bf),
        T("rows", 96, 4096, W.ROWS, **bf),
        T("short", 300, 768, W.ROWS, **bf),
        T("long", 24, 11008, W.ROWS, **bf),
        T("head", 256, 4096, W.HEADS, n_heads=2, **bf),
        T("whole", 1, 3 << 20, W.WHOLE, **bf),
        T("odd", 5, 1001, W.ROWS, **bf),
        T("longodd", 6, 10007, W.ROWS, **bf),
        T("f32rows", 64, 512, W.ROWS, grad_dtype=W.F32),
    ]
    return W.Workload("mixed", 61, tensors, W.GradRecipe(-4.0, -1.0), steps=3)


def make_optimizer(w: W.Workload, options: Optional[Dict[int, int]] = None, **hp) -> am.AdamMini:
    part = am.Partition(w.tensors)
    opt = am.AdamMini(part, **{**w.hparams, **hp})
    for k, val in (options or {}).items():
        opt.set_option(k, val)
    return opt


def oracle_step_all(state: ostep.OracleState, grads_cpu: Sequence, step: int, hp: Dict[str, float],
                    pool: Optional[cf.ThreadPoolExecutor] = None, statistic: int = 0) -> None:
    """One oracle step over all tensors; tensors are independent, so they may
    run on several host threads (each call is the single-threaded C routine)."""
    def one(i):
        ostep.adammini_step(state.p[i], state.m[i], state.v[i], grads_cpu[i], state.block_lens[i],
                            step=step, apply_wd=state.wd_flags[i], statistic=statistic, **hp)
    if pool is None:
        for i in range(len(grads_cpu)):
            one(i)
    else:
        list(pool.map(one, range(len(grads_cpu))))


def run_parity(w: W.Workload, steps: Optional[int] = None, options: Optional[Dict[int, int]] = None,
               device="cuda", hp_override: Optional[Dict[str, float]] = None, mutate_grads=None,
               lr_schedule=None, statistic: int = 0, optimizer: Optional[am.AdamMini] = None) -> Dict[str, float]:
    """Run `steps` steps on the GPU and in the oracle; returns the worst errors.

    mutate_grads(step, list_of_device_grads) may edit the gradients in place
    (zero rows, infinities) before both sides consume them.  `optimizer`: step
    with this handle (made for `w`) instead of a new one; it is left open.
    """
    steps = steps or w.steps
    hp = {**w.hparams, **(hp_override or {})}
    dev = DeviceState(w, device)
    if statistic:
        options = {**(options or {}), am.binding.OPT_STATISTIC: statistic}
    opt = optimizer or make_optimizer(w, options, **(hp_override or {}))
    ora = ostep.OracleState([p.cpu() for p in dev.p], [t.block_len for t in w.tensors],
                            [bool(t.apply_weight_decay) for t in w.tensors])
    unit = {i: ShortBlockScale(ora.p[i]) for i, t in enumerate(w.tensors)
            if t.block_len < (2 if os.environ.get("ADAMMINI_FLOOR_ONLY_UNIT_BLOCKS") == "1" else OWN_SCALE_MIN_L)}
    pool = cf.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1))
    try:
        for t in range(1, steps + 1):
            dev.draw_grads(t)
            if mutate_grads is not None:
                mutate_grads(t, dev.g)
            hp_t = dict(hp)
            if lr_schedule is not None:
                hp_t["lr"] = lr_schedule(t)
                opt.set_lr(hp_t["lr"])
            opt.step(dev.p, dev.g, dev.m, dev.v, t)
            grads_cpu = [g.cpu() for g in dev.g]
            oracle_step_all(ora, grads_cpu, t, hp_t, pool, statistic)
            for i, u in unit.items():
                u.update(ostep.widen(grads_cpu[i]), ora.p[i], ora.m[i], hp_t["beta1"])
        opt.sync_status()
    finally:
        pool.shutdown()
    assert dev.guards_intact(), "a kernel wrote outside its buffers"
    worst = {"p": 0.0, "m": 0.0, "v": 0.0}
    v_gpu = dev.v.cpu().numpy()
    off = 0
    for i, t in enumerate(w.tensors):
        u = unit.get(i)
        for key, got, want, floor in (("p", dev.p[i], ora.p[i], u.p if u else None), ("m", dev.m[i], ora.m[i], u.m if u else None)):
            got = got.cpu().numpy()
            err, k, scale = block_error_detail(got, want, t.block_len, floor)
            if err > worst[key]:
                worst[key] = err
                # where the worst element is, for the failure message
                worst[key + "_at"] = (f"{t.name}[{k}] L={t.block_len} gpu={got[k]!r} oracle={want[k]!r} scale={scale:.3e}"
                                      f" g={float(ostep.widen(grads_cpu[i][k:k + 1])[0]):.3e}")
        worst["v"] = max(worst["v"], v_relative_error(v_gpu[off:off + t.n_blocks], ora.v[i]))
        off += t.n_blocks
    if optimizer is None:
        opt.close()
    return worst


def assert_parity(worst: Dict[str, float], tol: float = TOL) -> None:
    assert worst["p"] <= tol and worst["m"] <= tol and worst["v"] <= tol, worst


def run_sampled_parity(w: W.Workload, steps: int, tensor_indices: Sequence[int], blocks_per_tensor: int = 3,
                       device="cuda") -> Dict[str, float]:
    """Full-size run in the configuration the benchmark times (unguarded
    buffers, default options); the oracle recomputes a sample of blocks one by
    one: first, last and seeded-random blocks of the chosen tensors."""
    dev = DeviceState(w, device, guarded=False)
    opt = make_optimizer(w)
    rng = np.random.default_rng(W.mix_seed(W.BASE_SEED, w.config_id, 4242) % (1 << 32))
    samples = []            # (tensor, block, oracle p, m, v)
    for i in tensor_indices:
        t = w.tensors[i]
        picks = {0, t.n_blocks - 1} | {int(x) for x in rng.integers(0, t.n_blocks, max(0, blocks_per_tensor - 2))}
        for b in sorted(picks):
            sl = slice(b * t.block_len, (b + 1) * t.block_len)
            samples.append([i, b, sl, ostep.widen(dev.p[i][sl].cpu()), np.zeros(t.block_len), np.zeros(1)])
    for step in range(1, steps + 1):
        dev.draw_grads(step)
        opt.step(dev.p, dev.g, dev.m, dev.v, step)
        for s in samples:
            i, b, sl = s[0], s[1], s[2]
            t = w.tensors[i]
            ostep.adammini_step(s[3], s[4], s[5], dev.g[i][sl].cpu(), t.block_len, step=step,
                                apply_wd=bool(t.apply_weight_decay), **w.hparams)
    opt.sync_status()
    worst = {"p": 0.0, "m": 0.0, "v": 0.0, "blocks": len(samples)}
    v_off = np.cumsum([0] + [t.n_blocks for t in w.tensors])
    for i, b, sl, po, mo, vo in samples:
        L = w.tensors[i].block_len
        worst["p"] = max(worst["p"], block_relative_error(dev.p[i][sl].cpu().numpy(), po, L))
        worst["m"] = max(worst["m"], block_relative_error(dev.m[i][sl].cpu().numpy(), mo, L))
        worst["v"] = max(worst["v"], v_relative_error(dev.v[v_off[i] + b:v_off[i] + b + 1].cpu().numpy(), vo))
    opt.close()
    return worst


def run_sampled_runs(w: W.Workload, steps: int, run_elems: int, n_runs: int, device="cuda") -> Dict[str, float]:
    """Full-size run of a one-tensor workload with short blocks; the oracle
    recomputes `n_runs` aligned runs of `run_elems` elements (whole blocks):
    the first, the last and seeded-random ones."""
    t = w.tensors[0]
    L = t.block_len
    assert len(w.tensors) == 1 and run_elems % L == 0 and t.numel % run_elems == 0
    dev = DeviceState(w, device, guarded=False)
    opt = make_optimizer(w)
    rng = np.random.default_rng(W.mix_seed(W.BASE_SEED, w.config_id, L) % (1 << 32))
    n_slots = t.numel // run_elems
    picks = sorted({0, n_slots - 1} | {int(x) for x in rng.integers(0, n_slots, n_runs - 2)})
    samples = []
    for k in picks:
        sl = slice(k * run_elems, (k + 1) * run_elems)
        p0 = ostep.widen(dev.p[0][sl].cpu())
        samples.append([sl, p0, np.zeros(run_elems), np.zeros(run_elems // L), ShortBlockScale(p0) if L < OWN_SCALE_MIN_L else None])
    for step in range(1, steps + 1):
        dev.draw_grads(step)
        opt.step(dev.p, dev.g, dev.m, dev.v, step)
        for sl, po, mo, vo, unit in samples:
            g = dev.g[0][sl].cpu()
            ostep.adammini_step(po, mo, vo, g, L, step=step, **w.hparams)
            if unit is not None:
                unit.update(ostep.widen(g), po, mo, w.hparams["beta1"])
    opt.sync_status()
    worst = {"p": 0.0, "m": 0.0, "v": 0.0, "blocks": len(samples) * (run_elems // L)}
    for sl, po, mo, vo, unit in samples:
        worst["p"] = max(worst["p"], block_relative_error(dev.p[0][sl].cpu().numpy(), po, L, unit.p if unit else None))
        worst["m"] = max(worst["m"], block_relative_error(dev.m[0][sl].cpu().numpy(), mo, L, unit.m if unit else None))
        vs = slice(sl.start // L, sl.stop // L)
        worst["v"] = max(worst["v"], v_relative_error(dev.v[vs].cpu().numpy(), vo))
    opt.close()
    return worst
