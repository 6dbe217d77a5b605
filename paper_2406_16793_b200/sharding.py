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

    def close(self) -> None:
        self.optimizer.close()
        self.partition.close()
