"""Whole-block sharding of an Adam-mini step over data-parallel ranks.

Blocks are independent (Algorithm 1 of the paper loops over blocks and nothing
crosses them), so a rank that owns a contiguous range of whole blocks can step
it with no collective inside the step: the optimizer-state sharding pattern of
ZeRO-1.  This module holds the host logic only: which blocks go to which rank,
and the tensor descriptors a rank hands to the library for its pieces.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

from .workloads import FIXED, TensorSpec


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
