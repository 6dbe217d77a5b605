#!/usr/bin/env python3
"""Benchmark of the Adam-mini optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one Adam-mini update (Algorithm 1 of the paper) over every tensor of
the workload; the default workload is the Llama-2-7B shape set (6.74 G
parameters, bf16 gradients, fp32 master parameters and moments).  One JSON
line is printed by rank 0.  With N > 1 (launched by torch.distributed.run)
every rank steps its own Llama-2-7B-sized shard of a model N times larger:
blocks are independent, so the step needs no collective (weak scaling).
`--shard blocks` / `--shard flat` make the ranks share ONE table instead
(whole-block shards without a collective / flat shards whose cut blocks get
their sums through one all-gather per step): strong scaling.

`--impl reference` times the float64 CPU checker from oracle/ on the host
cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "adam_mini_step_throughput"
UNIT = "Gparams/s"

NOMINAL_HBM_GBS = 8000.0      # HBM3e of a B200, nominal (quoted beside the measured-peak fraction)

# DRAM traffic per parameter (dram__bytes_read.sum + dram__bytes_write.sum) of each kernel
# family from the ncu captures summarised under profiles/.  An entry counts only while the
# sources its kernel is compiled from still have the digest they had at the capture.
NCU_TRAFFIC = [
    {"family": "stream_kernel<false>", "grad": "bf16", "block_lens": {4096, 11008}, "sources": "stream", "digest": "bb2178e8f2c7d6a3",
     "bytes_per_param": 17.909, "elements_query": lambda B: B.Q_ELEMENTS_STREAM,
     "capture": "profiles/stream_kernel_llama2_7b.md (2-layer case, scaled by parameters)"},
    {"family": "stream_kernel<true>", "grad": "bf16", "block_lens": {524288}, "sources": "stream", "digest": "bb2178e8f2c7d6a3",
     "bytes_per_param": 17.201, "elements_query": lambda B: B.Q_ELEMENTS_CLUSTER,
     "capture": "profiles/stream_kernel_llama2_7b.md (2-layer case, scaled by parameters)"},
    {"family": "stream_kernel<false>", "grad": "bf16", "block_lens": {10007}, "sources": "stream", "digest": "bb2178e8f2c7d6a3",
     "bytes_per_param": 17.595, "elements_query": lambda B: B.Q_ELEMENTS_STREAM,
     "capture": "profiles/stream_kernel_unaligned_rows_bf16_L10007.md (2^27 parameters, scaled)"},
    {"family": "short_block_kernels", "grad": "f32", "block_lens": {1}, "sources": "basic", "digest": "85b9245f3da5fdb0",
     "bytes_per_param": 27.587, "elements_query": lambda B: B.Q_ELEMENTS_SMALL,
     "capture": "profiles/small_and_twopass_kernels_flat_fp32.md (2^27 parameters, scaled)"},
    {"family": "short_block_kernels", "grad": "f32", "block_lens": {2}, "sources": "basic", "digest": "85b9245f3da5fdb0",
     "bytes_per_param": 23.597, "elements_query": lambda B: B.Q_ELEMENTS_SMALL,
     "capture": "profiles/small_and_twopass_kernels_flat_fp32.md (2^27 parameters, scaled)"},
    {"family": "twopass_kernels", "grad": "f32", "min_block_len": 1 << 22, "sources": "basic", "digest": "85b9245f3da5fdb0",
     "bytes_per_param": 23.650, "elements_query": lambda B: B.Q_ELEMENTS_TWOPASS,
     "capture": "profiles/small_and_twopass_kernels_flat_fp32.md (one block of 2^27 elements, scaled)"},
    {"family": "short_block_kernels", "grad": "f32", "block_lens": {32}, "sources": "tile", "digest": "c7d52bfd623def44",
     "bytes_per_param": 19.839, "elements_query": lambda B: B.Q_ELEMENTS_SMALL,
     "capture": "profiles/tile_kernel_flat_fp32_L32.md (2^27 parameters, scaled)"},
    {"family": "short_block_kernels", "grad": "bf16", "block_lens": {1001}, "sources": "tile", "digest": "c7d52bfd623def44",
     "bytes_per_param": 17.584, "elements_query": lambda B: B.Q_ELEMENTS_SMALL,
     "capture": "profiles/tile_kernel_rows_bf16_L1001.md (2^27 parameters, scaled)"},
]


def _stripped(text: str) -> bytes:
    import re
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    return "".join(text.split()).encode()


def kernel_digests() -> dict:
    """Digests of the sources each kernel family is compiled from, comments and
    whitespace removed: "stream" = the shared device helpers at the top of
    kernels_basic.cuh + the device code of kernels_stream.cuh; "tile" = those +
    kernels_tile.cuh; "basic" = all of kernels_basic.cuh (one-element blocks, two-pass)."""
    csrc = os.path.join(ROOT, "paper_2406_16793_b200", "csrc")
    basic = open(os.path.join(csrc, "kernels_basic.cuh")).read()
    stream = open(os.path.join(csrc, "kernels_stream.cuh")).read()
    tile = open(os.path.join(csrc, "kernels_tile.cuh")).read()
    helpers = basic[:basic.index("// Short blocks (L <= 64)")]
    stream_dev = stream[:stream.index("host-side planning")]
    out = {}
    for name, parts in (("stream", (helpers, stream_dev)), ("tile", (helpers, stream_dev, tile)), ("basic", (basic,))):
        h = hashlib.sha256()
        for part in parts:
            h.update(_stripped(part))
        out[name] = h.hexdigest()[:16]
    return out


def kernel_digest() -> str:
    """Digest of the streaming kernel's sources."""
    return kernel_digests()["stream"]


def ring_copy_ceiling(opt, dev, load_bytes: int, store_bytes: int, reps: int = 10):
    """What the device's memory gives a kernel that reads load_bytes and writes store_bytes per
    item and computes nothing: the library's copy through its ring of bulk loads and bulk stores
    (adammini_probe_ring_copy), timed here with events over 4 GiB of items."""
    import torch
    n_items = (4 << 30) // 40960
    try:
        src = torch.ones(max(n_items * load_bytes, 16), dtype=torch.uint8, device=dev)
        dst = torch.zeros(max(n_items * store_bytes, 16), dtype=torch.uint8, device=dev)
    except torch.OutOfMemoryError:
        return None
    for _ in range(3):
        opt.probe_ring_copy(src, dst, n_items, load_bytes, store_bytes)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        opt.probe_ring_copy(src, dst, n_items, load_bytes, store_bytes)
    e1.record()
    torch.cuda.synchronize(dev)
    opt.sync_status()
    ms = e0.elapsed_time(e1) / reps
    del src, dst
    return {"gbs": n_items * (load_bytes + store_bytes) / (ms * 1e-3) / 1e9, "ms_per_launch": ms,
            "read_bytes_per_item": load_bytes, "written_bytes_per_item": store_bytes, "items": n_items}


def update_mix(grad_f32: bool):
    """Bytes a stage of 4096 elements reads (g, m, p) and writes (m, p), scaled to a 40960-byte read."""
    return (40960, 27296) if grad_f32 else (40960, 32768)


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def pick_workload(name: str):
    from paper_2406_16793_b200 import workloads as W
    table = {
        "llama2-7b": W.llama2_7b, "llama3-8b": W.llama3_8b, "gpt2-small": W.gpt2_small,
        "tiny-gpt2": W.tiny_gpt2,
    }
    if name in table:
        return table[name]()
    if name.startswith("flat-L"):                      # flat-L<block length>[-n<log2 of the element count>]
        parts = name[6:].split("-n")
        L, numel = int(parts[0]), 1 << (int(parts[1]) if len(parts) > 1 else 30)
        import math
        unit = math.lcm(L, 64)                                         # whole blocks and whole 64-element chunks of one sigma
        return W.flat_sweep(L, numel=max(numel // unit, 1) * unit)
    if name.startswith("llama2-7b-layers"):
        return W.llama2_7b(n_layers=int(name[len("llama2-7b-layers"):]))
    if name.startswith("rows-"):                        # rows-<bf16|f32>-L<row length>-r<rows>: one matrix, a block per row
        dt, cols, rows = name[5:].split("-")
        spec = W.TensorSpec("mlp.rows", int(rows[1:]), int(cols[1:]), W.ROWS,
                            grad_dtype=W.BF16 if dt == "bf16" else W.F32)
        return W.Workload(name, 2, [spec], W.GradRecipe(-5.0, -1.0), steps=10)
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        clocks, powers, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.tmp:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) != 7:
                continue
            try:
                clocks.append(float(parts[0])); out["sm_max_mhz"] = float(parts[1]); powers.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:]):
                if val == "Active":
                    reasons.add(nm)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if clocks:
            out["sm_mhz"] = statistics.median(clocks)
            out["power_w_max"] = max(powers)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(clocks)
        return out


def oracle_sample(workload, budget_s: float = 12.0, max_steps: int = 40):
    """Time the float64 checker, as it stands and single-threaded, on the first
    transformer layer of the workload (all its tensors if it has no layers)."""
    import torch
    from oracle import step as ostep
    from paper_2406_16793_b200 import workloads as W
    idx = [i for i, t in enumerate(workload.tensors) if t.name.startswith(("layers.0.", "h.0."))]
    if not idx:
        idx = list(range(len(workload.tensors)))
        while sum(workload.tensors[i].numel for i in idx) > (1 << 28) and len(idx) > 1:
            idx.pop()
    specs = [workload.tensors[i] for i in idx]
    if sum(t.numel for t in specs) > (1 << 28):       # one huge flat tensor: take a prefix of whole blocks
        t = specs[0]
        L = min(t.block_len, 1 << 26)
        specs = [W.TensorSpec(t.name, 1, max(L, (1 << 26) // L * L), W.FIXED, fixed_block_len=L, grad_dtype=t.grad_dtype)]
        sub = W.Workload(workload.name, workload.config_id, specs, workload.recipe, workload.steps, workload.hparams)
        idx = [0]
    else:
        sub = workload
    params = [W.gen_param(sub, i) for i in idx]
    grads = [W.gen_grad(sub, i, 1) for i in idx]
    state = ostep.OracleState(params, [t.block_len for t in specs], [bool(t.apply_weight_decay) for t in specs])
    n = sum(t.numel for t in specs)
    ostep.load()
    done, t0 = 0, time.perf_counter()
    while done < max_steps and (done == 0 or time.perf_counter() - t0 < budget_s):
        state.step(grads, done + 1, **workload.hparams)
        done += 1
    dt = time.perf_counter() - t0
    return {"value": n * done / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{len(specs)} tensors ({n} params: first layer of {workload.name}), {done} steps, {dt:.1f} s",
            "seconds_per_step_extrapolated": workload.numel / (n * done / dt)}, n, done, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = pick_workload(args.workload)
    # each "step" of this arm is one oracle step over the bounded sample
    base, n, done, dt = oracle_sample(w, budget_s=max(4.0, 8.0 * args.steps / 10), max_steps=args.warmup + args.steps)
    value = base["value"]
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * n / (value * 1e9),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "params": w.numel, "sample_params": n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": base["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class PlainJob:
    """The whole table on this GPU: one handle, adammini_step."""

    def __init__(self, w, dev, world, rank):
        import torch
        import paper_2406_16793_b200 as am
        from paper_2406_16793_b200 import workloads as W
        n_t = len(w.tensors)
        self.specs = list(w.tensors)
        self.p = [W.gen_param(w, i, dev) for i in range(n_t)]
        self.m = [torch.zeros_like(x) for x in self.p]
        self.g = [W.gen_grad(w, i, 1, dev) for i in range(n_t)]
        self.part = am.Partition(w.tensors)
        self.v = torch.zeros(max(self.part.total_blocks, 1), dtype=torch.float32, device=dev)
        self.opt = am.AdamMini(self.part, **w.hparams)
        self.numel = w.numel                      # parameters this rank steps
        self.extra_launches = 0

    def step(self, t):
        self.opt.step(self.p, self.g, self.m, self.v, t)


class ShardedJob:
    """This rank's share of ONE table that all ranks step together (strong scaling).
    `blocks`: contiguous runs of whole blocks, no collective.  `flat`: equal ranges of
    the flat parameter space; blocks cut by a range boundary get their sum of g*g through
    one all-gather of part sums per step, inside the timed region."""

    def __init__(self, w, dev, world, rank, mode):
        import torch
        from paper_2406_16793_b200 import sharding, workloads as W
        self.mode = mode
        if mode == "blocks":
            self.sh = sharding.ShardedStep(w.tensors, world, rank, **w.hparams)
        else:
            self.sh = sharding.ShardedFlatStep(w.tensors, world, rank, device=dev, **w.hparams)
            self.exchange = sharding.all_gather_exchange if world > 1 else (lambda local: local.unsqueeze(0))
        self.opt, self.specs = self.sh.optimizer, self.sh.specs
        self.p, self.m, self.g = [], [], []
        cache = {}
        for piece in self.sh.pieces:              # this rank's slices of the full tensors' seeded inputs
            if piece.tensor not in cache:
                cache.clear()
                cache[piece.tensor] = (W.gen_param(w, piece.tensor, dev), W.gen_grad(w, piece.tensor, 1, dev))
            fp, fg = cache[piece.tensor]
            self.p.append(fp[piece.elem_begin:piece.elem_end].clone())
            self.g.append(fg[piece.elem_begin:piece.elem_end].clone())
            self.m.append(torch.zeros_like(self.p[-1]))
        cache.clear()
        self.v = torch.zeros(max(self.sh.local_blocks, 1), dtype=torch.float32, device=dev)
        self.numel = sum(x.numel() for x in self.p)
        # flat: two kernels for the part sums when this rank holds parts (torch's tiny index/copy kernels are not counted)
        self.extra_launches = 2 if mode == "flat" and self.sh.n_parts else 0

    def step(self, t):
        if self.mode == "blocks":
            self.sh.step_local(self.p, self.g, self.m, self.v, t)
        else:
            self.sh.step_local(self.p, self.g, self.m, self.v, t, self.exchange)


def family_of_specs(job, B):
    """The kernel family each tensor of the job runs on, by the library's routing rules as its
    element counts per family confirm them: short or tile-sized unaligned blocks -> short-block
    kernels; head-sized blocks -> the cluster kernel; blocks beyond 4 MB of gradients -> two-pass."""
    out = []
    for t in job.specs:
        gsz = 2 if t.grad_dtype == 1 else 4
        L = t.block_len
        if L <= 64 or (L <= 4096 and (L * gsz) % 16):
            out.append("short_block_kernels")
        elif L * gsz <= 256 * 1024:
            out.append("stream_kernel<false>")
        elif L * gsz <= 4 * 1024 * 1024 and L % (8 * 16 // gsz) == 0:
            out.append("stream_kernel<true>")
        else:
            out.append("twopass_kernels")
    counts = {"short_block_kernels": B.Q_ELEMENTS_SMALL, "stream_kernel<false>": B.Q_ELEMENTS_STREAM,
              "stream_kernel<true>": B.Q_ELEMENTS_CLUSTER, "twopass_kernels": B.Q_ELEMENTS_TWOPASS}
    for fam, q in counts.items():
        if sum(t.numel for t, f in zip(job.specs, out) if f == fam) != job.opt.query(q):
            return [None] * len(out)           # the routing differs (an option forces a path): no capture applies
    return out


def ncu_traffic(family: str, job, B):
    """DRAM bytes per launch of the dominant kernel family from the ncu captures
    summarised under profiles/, scaled by the parameters the family processes; None
    when the kernel sources have changed since the capture or no capture matches."""
    digests = kernel_digests()
    bf16 = all(t.grad_dtype == 1 for t in job.specs)
    f32 = all(t.grad_dtype == 0 for t in job.specs)
    for e in NCU_TRAFFIC:
        if e["family"] != family or digests.get(e["sources"]) != e["digest"]:
            continue
        if (e["grad"] == "bf16" and not bf16) or (e["grad"] == "f32" and not f32):
            continue
        # a capture speaks for the block lengths it ran: every tensor the family handles must have one of them
        fam_lens = {t.block_len for t, path in zip(job.specs, family_of_specs(job, B)) if path == family}
        if not fam_lens:
            continue
        if "min_block_len" in e:
            if min(fam_lens) < e["min_block_len"]:
                continue
        elif not fam_lens <= e["block_lens"]:
            continue
        return e["bytes_per_param"] * job.opt.query(e["elements_query"](B)), e["capture"]
    return None, None


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2406_16793_b200 import build as lib_build
    from paper_2406_16793_b200 import binding as B, workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()

    w = pick_workload(args.workload)
    job = PlainJob(w, dev, world, rank) if args.shard == "none" else ShardedJob(w, dev, world, rank, args.shard)
    opt = job.opt
    for key, val in ((B.OPT_STREAM_THREADS, args.stream_threads), (B.OPT_STREAM_CTAS, args.stream_ctas),
                     (B.OPT_CLUSTER_SIZE, args.cluster_size), (B.OPT_PATH, args.path),
                     (B.OPT_STREAM_CHUNK, args.stream_chunk), (B.OPT_CLUSTER_CHUNK, args.cluster_chunk),
                     (B.OPT_STREAM_GROUPS, args.stream_groups), (B.OPT_STATISTIC, args.statistic)):
        if val:
            opt.set_option(key, val)
    launches = opt.query(B.Q_LAUNCHES_PER_STEP) + job.extra_launches
    alg_bytes = opt.query(B.Q_ALGORITHMIC_BYTES)

    t = 0
    for _ in range(args.warmup):
        t += 1
        job.step(t)
    opt.sync_status()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler("GPU-" + str(props.uuid) if hasattr(props, "uuid") else str(local))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the library records CUDA events around each of its kernels on the launch stream, so the
    # per-kernel durations below come from the timed region itself
    opt.set_option(B.OPT_PROFILE, min(args.steps, 4096))
    time.sleep(0.3)
    barrier()
    e0.record()
    for _ in range(args.steps):
        t += 1
        job.step(t)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    opt.sync_status()
    if world > 1:
        tt = torch.tensor([ms_total], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_total = float(tt.item())
    ms_step = ms_total / args.steps
    # whole-job throughput: the parameters all ranks stepped (replicas: world x the table; shards: the table once)
    total_params = world * w.numel if args.shard == "none" else w.numel
    value = total_params / (ms_step * 1e-3) / 1e9
    fam_ms, prof_steps = opt.get_profile()
    opt.set_option(B.OPT_PROFILE, 0)
    fam_bytes = [opt.query(q) for q in (B.Q_BYTES_SMALL, B.Q_BYTES_STREAM, B.Q_BYTES_CLUSTER, B.Q_BYTES_TWOPASS)]
    fam_names = ["short_block_kernels", "stream_kernel<false>", "stream_kernel<true>", "twopass_kernels"]
    peak, peak_kind = measured_peak_gbs()
    kernels = {}
    for nme, ms_k, by in zip(fam_names, fam_ms, fam_bytes):
        if by:
            kernels[nme] = {"ms": ms_k, "algorithmic_bytes": by, "gbs": by / (ms_k * 1e-3) / 1e9,
                            "frac": by / (ms_k * 1e-3) / 1e9 / peak}
    top = max(range(4), key=lambda k: fam_ms[k] if fam_bytes[k] else -1.0)
    achieved = fam_bytes[top] / (fam_ms[top] * 1e-3) / 1e9
    traffic, capture = ncu_traffic(fam_names[top], job, B)
    whole_gbs = alg_bytes / (ms_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": fam_names[top], "achieved": achieved, "peak": peak,
                "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                "frac_of_nominal": achieved / NOMINAL_HBM_GBS, "nominal_peak": NOMINAL_HBM_GBS,
                "traffic": traffic, "traffic_capture": capture, "algorithmic_bytes_per_launch": fam_bytes[top],
                "whole_step_gbs": whole_gbs, "whole_step_frac": whole_gbs / peak,
                "whole_step_frac_of_nominal": whole_gbs / NOMINAL_HBM_GBS}

    if not args.no_ring_copy:
        # the ceiling for the update's own mix of reads and writes (and, on request, for other mixes)
        ring = ring_copy_ceiling(opt, dev, *update_mix(w.tensors[0].grad_dtype != W.BF16))
        if ring:
            ring["what"] = "bulk-load / bulk-store ring of this library with no arithmetic, the update's read:write mix"
            roofline["ring_copy"] = ring
            roofline["frac_of_ring_copy"] = achieved / ring["gbs"]
            roofline["whole_step_frac_of_ring_copy"] = whole_gbs / ring["gbs"]
        if args.ring_copy_modes:
            roofline["ring_copy_modes"] = [ring_copy_ceiling(opt, dev, *(int(x) for x in mode.split(":")))
                                           for mode in args.ring_copy_modes.split(",")]

    e2e = None
    if not args.no_e2e:
        if args.shard == "flat" and opt.query(B.Q_PART_TENSORS) > 0:
            e2e = {"value": None, "unit": UNIT, "skipped": "this rank holds parts of cut blocks: the host-buffer step has no exchange"}
        else:
            e2e = run_e2e(args, opt, job.specs, total_params / world, world, dev, job.p, job.g, job.m, job.v, w.name)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_sample(w)[0]

    if rank == 0:
        parallelism = {"none": f"dp{world} (independent replicas of the table, no collective)",
                       "blocks": f"dp{world} (whole-block shards of one table, no collective)",
                       "flat": f"dp{world} (flat shards of one table, one all-gather of part sums per step)"}[args.shard]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak" if args.shard == "none" else "strong",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "params": w.numel, "blocks": w.n_blocks, "tensors": len(w.tensors),
                       "grad_dtype": "bf16" if w.tensors[0].grad_dtype == W.BF16 else "f32",
                       "l2": "inputs larger than L2 (no flush needed)" if alg_bytes > (1 << 29) else "inputs fit L2",
                       "shard": args.shard, "statistic": args.statistic, "parallelism": parallelism},
            "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline, "e2e": e2e,
            "gpu_launches": launches * args.steps, "clocks": clocks,
            "gpu": {"name": props.name, "uuid_tail": str(getattr(props, "uuid", ""))[-8:]},
            "stream_ctas": opt.query(B.Q_STREAM_CTAS), "cluster": [opt.query(B.Q_CLUSTER_COUNT), opt.query(B.Q_CLUSTER_SIZE)],
        }
        print(json.dumps(line), flush=True)
    if args.shard == "none":
        opt.close()
    else:
        job.sh.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_e2e(args, opt, specs, params_per_rank, world, dev, p, g, m, v, workload_name):
    """The same step through adammini_step_host: parameters, moments, v and
    gradients in pinned host memory; host->device and device->host copies are
    inside the timed region (CUDA events cannot bracket a call that blocks on
    several internal streams, so this arm is timed with the host clock around
    the blocking C call, max over ranks)."""
    import torch
    import torch.distributed as dist
    need = sum(t.numel * (8 + (2 if t.grad_dtype else 4)) for t in specs)
    avail = 0
    for line in open("/proc/meminfo"):
        if line.startswith("MemAvailable"):
            avail = int(line.split()[1]) * 1024
    if avail < 1.5 * need * max(1, min(world, torch.cuda.device_count())):
        return {"value": None, "unit": UNIT, "skipped": f"host memory: need {need} B pinned per rank, {avail} B available"}
    def pinned_copy(x):                     # straight into pinned memory: no pageable intermediate
        out = torch.empty(x.shape, dtype=x.dtype, pin_memory=True)
        out.copy_(x)
        return out
    hp = [pinned_copy(x) for x in p]
    hm = [pinned_copy(x) for x in m]
    hg = [pinned_copy(x) for x in g]
    hv = pinned_copy(v)
    h2d = sum(x.numel() * x.element_size() for x in hp + hm + hg) + hv.numel() * 4
    d2h = sum(x.numel() * x.element_size() for x in hp + hm) + hv.numel() * 4
    steps = max(1, min(args.e2e_steps, args.steps))
    t = 1000
    opt.step_host(hp, hg, hm, hv, t)          # warm-up: builds the staging pipeline
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        t += 1
        opt.step_host(hp, hg, hm, hv, t)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    if world > 1:
        tt = torch.tensor([dt], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        dt = float(tt.item())
    return {"value": world * params_per_rank * steps / dt / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * dt / steps, "steps": steps,
            "h2d_plus_d2h_gbs": (h2d + d2h) * steps / dt / 1e9, "workload": workload_name,
            "api": "adammini_step_host (pinned host buffers, 3 staging slots)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--stream-threads", type=int, default=0, help="consumer threads per CTA (0 = library default)")
    ap.add_argument("--stream-groups", type=int, default=0, help="consumer groups per CTA (0 = library default)")
    ap.add_argument("--stream-ctas", type=int, default=0, help="persistent CTAs (0 = one per SM)")
    ap.add_argument("--cluster-size", type=int, default=0, help="CTAs per cluster for head-sized blocks (0 = default)")
    ap.add_argument("--stream-chunk", type=int, default=0, help="items per grab from the shared work counter (0 = automatic, 1000000 = static ranges)")
    ap.add_argument("--cluster-chunk", type=int, default=0, help="blocks per grab of a cluster (0 = automatic, 1000000 = static)")
    ap.add_argument("--path", type=int, default=0, help="1 = force the two-pass kernels")
    ap.add_argument("--statistic", type=int, default=0, help="block statistic: 0 mean (Algorithm 1); 1 max, 2 min, 3 one-norm, 4 two-norm (the paper's ablation)")
    ap.add_argument("--shard", default="none", choices=["none", "blocks", "flat"],
                    help="none: every rank steps its own copy of the table (weak scaling); blocks / flat: the ranks "
                         "share ONE table as whole-block shards / as flat shards with one exchange of part sums (strong scaling)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-ring-copy", action="store_true", help="skip the copy-through-the-ring ceiling measurement")
    ap.add_argument("--ring-copy-modes", default="", help="further read:write byte mixes per item to time through the ring, e.g. 40960:40960,40960:0,0:40960")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
