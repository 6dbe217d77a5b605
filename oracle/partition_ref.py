"""Partition rules of Adam-mini in plain Python -- TEST INFRASTRUCTURE ONLY.

Algorithm 2 ("Partition for non-Transformers": one block per named tensor) and
Algorithm 3 ("Partition for Transformers": embed/output by token, query/key by
head, value/attn.proj/mlp by output neuron, anything else whole).  Weights are
taken as [out_features, in_features], row-major, so a token row, an output
neuron and a head (head_dim consecutive rows) are all contiguous runs and a
tensor is n_blocks runs of one length.

The table produced here is compared bit for bit with the one the library's
host partitioner exports.  Kind and dtype codes are the library's ABI values.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterable, List, Sequence

WHOLE, ROWS, HEADS, TOKENS, FIXED, PART = 0, 1, 2, 3, 4, 5
F32, BF16 = 0, 1


@dataclass(frozen=True)
class TensorDesc:
    rows: int
    cols: int
    kind: int
    n_heads: int = 0
    fixed_block_len: int = 0
    grad_dtype: int = F32
    apply_weight_decay: int = 1


@dataclass(frozen=True)
class TableRow:
    numel: int
    block_len: int
    n_blocks: int
    v_offset: int
    kind: int
    grad_dtype: int
    wd: int
    mean_len: int = 0       # divisor of the block mean; differs from block_len only for PART


def block_len_of(d: TensorDesc) -> int:
    """Length of one block of tensor `d` under its kind (Algorithm 3 branches)."""
    numel = d.rows * d.cols
    if d.kind == WHOLE:                      # ELSE branch / Algorithm 2
        return numel
    if d.kind in (ROWS, TOKENS):             # one block per output neuron / token
        return d.cols
    if d.kind == HEADS:                      # one block per head
        if d.n_heads <= 0 or d.rows % d.n_heads:
            raise ValueError("rows must divide into n_heads heads")
        return (d.rows // d.n_heads) * d.cols
    if d.kind == FIXED:
        if d.fixed_block_len <= 0 or numel % d.fixed_block_len:
            raise ValueError("fixed block length must divide numel")
        return d.fixed_block_len
    if d.kind == PART:                       # a part of one block held elsewhere too: one local block
        if d.rows != 1 or d.fixed_block_len < numel:
            raise ValueError("a part cannot be longer than its block")
        return numel
    raise ValueError(f"unknown kind {d.kind}")


def build_table(descs: Sequence[TensorDesc]) -> tuple[List[TableRow], int]:
    """Flat block table in the caller's tensor order, and the total block count."""
    rows: List[TableRow] = []
    v_offset = 0
    for d in descs:
        if d.rows <= 0 or d.cols <= 0:
            raise ValueError("empty tensor")
        numel = d.rows * d.cols
        L = block_len_of(d)
        nb = numel // L
        rows.append(TableRow(numel, L, nb, v_offset, d.kind, d.grad_dtype,
                             1 if d.apply_weight_decay else 0,
                             d.fixed_block_len if d.kind == PART else L))
        v_offset += nb
    return rows, v_offset


def kind_from_name(name: str) -> int:
    """Algorithm 3's name tests, in its order of precedence."""
    if "embed" in name or "output" in name:
        return TOKENS
    if "query" in name or "key" in name:
        return HEADS
    if "value" in name or "attn.proj" in name or "mlp" in name:
        return ROWS
    return WHOLE


def blocks_as_index_lists(descs: Iterable[TensorDesc]) -> List[List[int]]:
    """Every block as an explicit list of flat element indices (tiny cases)."""
    out: List[List[int]] = []
    base = 0
    for d in descs:
        L = block_len_of(d)
        numel = d.rows * d.cols
        for b in range(numel // L):
            out.append(list(range(base + b * L, base + (b + 1) * L)))
        base += numel
    return out
