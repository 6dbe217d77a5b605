"""Whole-block sharding of an Adam-mini step over data-parallel ranks.

Blocks are independent (Algorithm 1 of the paper loops over blocks and nothing
crosses them), so a rank that owns a contiguous range of whole blocks can step
it with no collective inside the step: the optimizer-state sharding pattern of
ZeRO-1.  This module holds the host logic only: which blocks go to which rank,
and the tensor descriptors a rank hands to the library for its pieces.
"""
from __future__ import annotations

from dataclasses import dataclass
from math import gcd
from typing import List, Sequence

from .workloads import BF16, FIXED, TensorSpec


@dataclass(frozen=True)
class ShardPiece:
    """Blocks [block_begin, block_end) of tensor `tensor`, owned by one rank."""
    tensor: int
    block_begin: int
    block_end: int
    block_len: int
    v_begin: int            # index of the piece's first block in the unsharded v

    @property
    def elem_begin(self) -> int:
        return self.block_begin * self.block_len

    @property
    def elem_end(self) -> int:
        return self.block_end * self.block_len

    @property
    def numel(self) -> int:
        return self.elem_end - self.elem_begin

    def spec(self, parent: TensorSpec) -> TensorSpec:
        """Descriptor of the piece: a flat run of whole blocks of the parent."""
        return TensorSpec(f"{parent.name}[{self.block_begin}:{self.block_end}]", 1, self.numel, FIXED,
                          fixed_block_len=self.block_len, grad_dtype=parent.grad_dtype,
                          apply_weight_decay=parent.apply_weight_decay)


def shard_by_blocks(tensors: Sequence[TensorSpec], world_size: int) -> List[List[ShardPiece]]:
    """Cut the flat block table into `world_size` contiguous ranges of whole
    blocks with (nearly) equal element counts.  Rank r owns result[r]; the
    pieces of all ranks tile every tensor exactly once, in table order."""
    if world_size < 1:
        raise ValueError("world_size must be positive")
    total = sum(t.numel for t in tensors)
    out: List[List[ShardPiece]] = [[] for _ in range(world_size)]
    done = 0                 # elements assigned so far
    rank = 0
    v_off = 0
    for ti, t in enumerate(tensors):
        L, nb = t.block_len, t.n_blocks
        b = 0
        while b < nb:
            # this rank's quota ends at the block boundary nearest to its target
            target = total * (rank + 1) // world_size
            room = target - done
            take = nb - b if rank == world_size - 1 else min(nb - b, max(0, (room + L // 2) // L))
            if take < nb - b:
                # a cut inside a tensor must leave every piece 16-byte aligned (8 bf16 or 4 fp32 elements)
                step = 8 // gcd(L, 8)
                take = ((b + take) // step) * step - b
                take = max(take, 0)
            if take == 0:
                if rank < world_size - 1:
                    rank += 1
                    continue
                take = nb - b
            out[rank].append(ShardPiece(ti, b, b + take, L, v_off + b))
            done += take * L
            b += take
            if done >= target and rank < world_size - 1:
                rank += 1
        v_off += nb
    return out


class ShardedStep:
    """One rank's share of an Adam-mini step: the rank's pieces as a partition
    of their own, stepped through the library on views of the full tensors.

    Every rank holds (or can address) the full parameter, gradient and moment
    tensors and updates only its blocks; after the step a trainer all-gathers
    the updated parameters (outside this class).  v is sharded: the rank keeps
    only the second moments of its own blocks.
    """

    def __init__(self, tensors: Sequence[TensorSpec], world_size: int, rank: int, **hparams):
        from . import binding
        self.tensors = list(tensors)
        self.pieces = shard_by_blocks(self.tensors, world_size)[rank]
        self.specs = [p.spec(self.tensors[p.tensor]) for p in self.pieces]
        self.partition = binding.Partition(self.specs)
        self.optimizer = binding.AdamMini(self.partition, **hparams)
        self.local_blocks = sum(p.block_end - p.block_begin for p in self.pieces)

    def _views(self, full, grads: bool):
        out = []
        for p in self.pieces:
            t = self.tensors[p.tensor]
            item = (2 if t.grad_dtype == BF16 else 4) if grads else 4
            x = full[p.tensor]
            base = int(x.data_ptr()) if hasattr(x, "data_ptr") else int(x)
            out.append(base + p.elem_begin * item)
        return out

    def step(self, params, grads, m, v_local, step: int, stream: int = 0) -> None:
        """params/grads/m: the FULL tensors in table order (device tensors or raw
        addresses); v_local: float32[self.local_blocks] of this rank."""
        self.optimizer.step(self._views(params, False), self._views(grads, True), self._views(m, False),
                            v_local, step, stream)

    def step_local(self, params, grads, m, v_local, step: int, stream: int = 0) -> None:
        """The same for a rank that keeps only its own share: params/grads/m hold one
        buffer per piece of self.pieces (piece k: self.specs[k].numel elements)."""
        self.optimizer.step(params, grads, m, v_local, step, stream)

    def close(self) -> None:
        self.optimizer.close()
        self.partition.close()


# -----------------------------------------------------------------------------
# Flat shards that cut blocks (FSDP-style): one exchange per step
# -----------------------------------------------------------------------------
# A rank owns a contiguous range of the flat concatenation of all tensors.  The
# range can begin and end inside a block; such a block's mean of g*g needs the
# parts held by other ranks, so the step gets ONE exchange: every rank computes
# the sums of g*g of its parts (adammini_part_sums), the sums of each cut block
# are added over its holders (an all-gather of a few doubles per rank), and the
# step uses the totals (am_step_extras.part_sums).  Blocks that lie wholly
# inside a shard need nothing from outside.  The second moment of a cut block
# is kept, identically, by every rank that holds a part of it.

from .workloads import PART  # noqa: E402


@dataclass(frozen=True)
class FlatPiece:
    """Elements [elem_begin, elem_end) of tensor `tensor`, owned by one rank:
    either whole blocks, or (part=True) a piece of the single block `block`."""
    tensor: int
    elem_begin: int
    elem_end: int
    block_len: int
    part: bool
    block: int              # first block index (whole blocks) or the cut block's index (part)

    @property
    def numel(self) -> int:
        return self.elem_end - self.elem_begin

    @property
    def n_blocks(self) -> int:
        return 1 if self.part else self.numel // self.block_len

    def spec(self, parent: TensorSpec) -> TensorSpec:
        if self.part:
            return TensorSpec(f"{parent.name}[{self.elem_begin}:{self.elem_end}]part", 1, self.numel, PART,
                              fixed_block_len=self.block_len, grad_dtype=parent.grad_dtype,
                              apply_weight_decay=parent.apply_weight_decay)
        return TensorSpec(f"{parent.name}[{self.elem_begin}:{self.elem_end}]", 1, self.numel, FIXED,
                          fixed_block_len=self.block_len, grad_dtype=parent.grad_dtype,
                          apply_weight_decay=parent.apply_weight_decay)


def shard_flat(tensors: Sequence[TensorSpec], world_size: int, align: int = 8) -> List[List[FlatPiece]]:
    """Equal contiguous ranges of the flat concatenation of `tensors` (range
    boundaries at multiples of `align` elements of the flat space), expressed
    as pieces: whole blocks where a block lies inside the range, parts of a
    block where the range cuts it.  A run of whole blocks that would not start
    16-byte aligned is handed out block by block as parts that happen to be
    whole (their sums then come from the rank itself)."""
    total = sum(t.numel for t in tensors)
    bounds = [min(total, ((total * r // world_size) + align - 1) // align * align) for r in range(world_size)] + [total]
    bounds[0] = 0
    out: List[List[FlatPiece]] = [[] for _ in range(world_size)]
    base = 0
    for ti, t in enumerate(tensors):
        L = t.block_len
        step = 8 // gcd(L, 8)           # block indices at which a run of whole blocks is 16-byte aligned
        for r in range(world_size):
            a, b = max(bounds[r], base) - base, min(bounds[r + 1], base + t.numel) - base
            if a >= b:
                continue
            pieces = out[r]
            cur = a
            if cur % L:                                     # leading part of a cut block
                end = min(b, (cur // L + 1) * L)
                pieces.append(FlatPiece(ti, cur, end, L, True, cur // L))
                cur = end
            while cur < b and (cur // L) % step and cur + L <= b:      # unaligned whole blocks, one by one
                pieces.append(FlatPiece(ti, cur, cur + L, L, True, cur // L))
                cur += L
            whole_end = b // L * L
            if whole_end > cur:
                pieces.append(FlatPiece(ti, cur, whole_end, L, False, cur // L))
                cur = whole_end
            if cur < b:                                     # trailing part
                pieces.append(FlatPiece(ti, cur, b, L, True, cur // L))
        base += t.numel
    return out


class FlatExchangePlan:
    """Bookkeeping of the one exchange of a flat-sharded step, for one rank:
    which of the gathered part sums belong to each of this rank's cut blocks.
    Pure host logic (torch tensors on any device)."""

    def __init__(self, tensors: Sequence[TensorSpec], world_size: int, rank: int, device="cpu"):
        import torch
        self.tensors = list(tensors)
        self.world, self.rank = world_size, rank
        all_pieces = shard_flat(self.tensors, world_size)
        self.pieces = all_pieces[rank]
        self.local_blocks = sum(p.n_blocks for p in self.pieces)
        # who holds a part of which cut block, in rank order (identical on every rank)
        part_lists = [[(p.tensor, p.block) for p in ps if p.part] for ps in all_pieces]
        self.part_keys = part_lists[rank]
        self.max_parts = max(1, max(len(x) for x in part_lists))
        holders = {}
        for r, keys in enumerate(part_lists):
            for slot, key in enumerate(keys):
                holders.setdefault(key, []).append(r * self.max_parts + slot)
        self.n_parts = len(self.part_keys)
        width = max([len(holders[k]) for k in self.part_keys], default=1)
        idx = torch.zeros(max(self.n_parts, 1), width, dtype=torch.int64)
        mask = torch.zeros(max(self.n_parts, 1), width, dtype=torch.float64)
        for i, k in enumerate(self.part_keys):
            for j, pos in enumerate(holders[k]):
                idx[i, j] = pos
                mask[i, j] = 1.0
        self.idx, self.mask = idx.to(device), mask.to(device)

    def combine(self, gathered):
        """Whole-block sums of this rank's cut blocks from the [world, max_parts]
        tensor of every rank's part sums, added in rank order (so every holder
        of a block computes the same bits)."""
        vals = gathered.reshape(-1)[self.idx] * self.mask
        total = vals[:, 0].clone()
        for j in range(1, vals.shape[1]):
            total = total + vals[:, j]
        return total


class ShardedFlatStep:
    """One rank's share of a step under flat sharding.

    step() runs: local sums of the rank's parts -> `exchange` -> the library's
    step with the whole-block sums.  `exchange(local)` receives this rank's
    float64 device tensor of part sums (padded to `max_parts`) and must return
    the [world, max_parts] tensor of every rank's sums (an all-gather);
    `all_gather_exchange` does that with torch.distributed.
    """

    def __init__(self, tensors: Sequence[TensorSpec], world_size: int, rank: int, device="cuda", **hparams):
        import torch
        from . import binding
        self.plan = FlatExchangePlan(tensors, world_size, rank, device)
        self.tensors, self.pieces = self.plan.tensors, self.plan.pieces
        self.n_parts, self.max_parts, self.local_blocks = self.plan.n_parts, self.plan.max_parts, self.plan.local_blocks
        self.specs = [p.spec(self.tensors[p.tensor]) for p in self.pieces]
        self.partition = binding.Partition(self.specs)
        self.optimizer = binding.AdamMini(self.partition, **hparams)
        self.local = torch.zeros(self.max_parts, dtype=torch.float64, device=device)
        self.totals = torch.zeros(max(self.n_parts, 1), dtype=torch.float64, device=device)

    def _views(self, full, grads: bool):
        out = []
        for p in self.pieces:
            t = self.tensors[p.tensor]
            item = (2 if t.grad_dtype == BF16 else 4) if grads else 4
            x = full[p.tensor]
            base = int(x.data_ptr()) if hasattr(x, "data_ptr") else int(x)
            out.append(base + p.elem_begin * item)
        return out

    def local_sums(self, grads):
        """Phase 1: this rank's sums of g*g over its parts, padded to max_parts."""
        self.local.zero_()
        if self.n_parts:
            self.optimizer.part_sums(self._views(grads, True), self.local)
        return self.local

    def combine(self, gathered):
        self.totals.copy_(self.plan.combine(gathered))
        return self.totals

    def apply(self, params, grads, m, v_local, step: int, stream: int = 0) -> None:
        """Phase 2: the step proper, with the totals from combine()."""
        self.optimizer.step_ex(self._views(params, False), self._views(grads, True), self._views(m, False),
                               v_local, step, stream, part_sums=self.totals if self.n_parts else None)

    def step(self, params, grads, m, v_local, step: int, exchange) -> None:
        self.combine(exchange(self.local_sums(grads)))
        self.apply(params, grads, m, v_local, step)

    def step_local(self, params, grads, m, v_local, step: int, exchange) -> None:
        """step() for a rank that keeps only its own share: one buffer per piece of
        self.pieces (piece k: self.specs[k].numel elements)."""
        self.local.zero_()
        if self.n_parts:
            self.optimizer.part_sums(grads, self.local)
        self.combine(exchange(self.local))
        self.optimizer.step_ex(params, grads, m, v_local, step, part_sums=self.totals if self.n_parts else None)

    def close(self) -> None:
        self.optimizer.close()
        self.partition.close()


def all_gather_exchange(local, group=None):
    """The exchange of ShardedFlatStep over torch.distributed, whatever the
    backend of the process group (NCCL between GPUs, gloo between CPU ranks):
    returns the [world, len(local)] tensor of every rank's part sums, rank r's
    in row r.  A few doubles per rank: a latency-sized collective."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = torch.empty(world, local.numel(), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous(), group=group)
    return out


nccl_all_gather = all_gather_exchange
