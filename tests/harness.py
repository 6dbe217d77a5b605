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


MIN_SCALE_RUN = 64


def block_relative_error(got: np.ndarray, want: np.ndarray, L: int) -> float:
    """max_i |got-want| / max(|want_i|, rms(want over i's block)); NaN/inf must match.

    For blocks shorter than 64 elements the RMS is taken over the aligned run
    of 64 consecutive elements that holds the block (a one-element block has no
    scale of its own: an entry of m or p that crosses zero would otherwise make
    the ratio meaningless)."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    if want.size == 0:
        return 0.0
    fin = np.isfinite(want)
    if not np.array_equal(fin, np.isfinite(got)):
        return float("inf")
    if not fin.all():
        same = np.where(fin, True, (np.isnan(want) & np.isnan(got)) | (want == got))
        if not same.all():
            return float("inf")
    w = np.where(fin, want, 0.0)
    run = L if L >= MIN_SCALE_RUN else MIN_SCALE_RUN
    starts = np.arange(0, w.size, run)
    counts = np.diff(np.append(starts, w.size))
    rms = np.sqrt(np.add.reduceat(w * w, starts) / counts)
    scale = np.maximum(np.abs(w), np.repeat(rms, counts))
    scale = np.where(scale > 0, scale, 1.0)
    err = np.where(fin, np.abs(got - w) / scale, 0.0)
    return float(err.max())


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
               lr_schedule=None, statistic: int = 0) -> Dict[str, float]:
    """Run `steps` steps on the GPU and in the oracle; returns the worst errors.

    mutate_grads(step, list_of_device_grads) may edit the gradients in place
    (zero rows, infinities) before both sides consume them.
    """
    steps = steps or w.steps
    hp = {**w.hparams, **(hp_override or {})}
    dev = DeviceState(w, device)
    if statistic:
        options = {**(options or {}), am.binding.OPT_STATISTIC: statistic}
    opt = make_optimizer(w, options, **(hp_override or {}))
    ora = ostep.OracleState([p.cpu() for p in dev.p], [t.block_len for t in w.tensors],
                            [bool(t.apply_weight_decay) for t in w.tensors])
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
        opt.sync_status()
    finally:
        pool.shutdown()
    assert dev.guards_intact(), "a kernel wrote outside its buffers"
    worst = {"p": 0.0, "m": 0.0, "v": 0.0}
    v_gpu = dev.v.cpu().numpy()
    off = 0
    for i, t in enumerate(w.tensors):
        worst["p"] = max(worst["p"], block_relative_error(dev.p[i].cpu().numpy(), ora.p[i], t.block_len))
        worst["m"] = max(worst["m"], block_relative_error(dev.m[i].cpu().numpy(), ora.m[i], t.block_len))
        worst["v"] = max(worst["v"], v_relative_error(v_gpu[off:off + t.n_blocks], ora.v[i]))
        off += t.n_blocks
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
        samples.append([sl, ostep.widen(dev.p[0][sl].cpu()), np.zeros(run_elems), np.zeros(run_elems // L)])
    for step in range(1, steps + 1):
        dev.draw_grads(step)
        opt.step(dev.p, dev.g, dev.m, dev.v, step)
        for sl, po, mo, vo in samples:
            ostep.adammini_step(po, mo, vo, dev.g[0][sl].cpu(), L, step=step, **w.hparams)
    opt.sync_status()
    worst = {"p": 0.0, "m": 0.0, "v": 0.0, "blocks": len(samples) * (run_elems // L)}
    for sl, po, mo, vo in samples:
        worst["p"] = max(worst["p"], block_relative_error(dev.p[0][sl].cpu().numpy(), po, L))
        worst["m"] = max(worst["m"], block_relative_error(dev.m[0][sl].cpu().numpy(), mo, L))
        vs = slice(sl.start // L, sl.stop // L)
        worst["v"] = max(worst["v"], v_relative_error(dev.v[vs].cpu().numpy(), vo))
    opt.close()
    return worst
