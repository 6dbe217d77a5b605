"""Front end of the partitioner: (name, shape) pairs -> tensor descriptors.

Algorithm 3 of the paper ("Partition for Transformers") chooses a tensor's
blocks from its name: "embed"/"output" by token, "query"/"key" by head,
"value"/"attn.proj"/"mlp" by output neuron, everything else as one block.
The name tests themselves run in the library (adammini_kind_from_name); this
module adds what the rule needs besides the name -- the head counts -- and the
two variants the paper discusses: the whole-tensor treatment of `value`
(its appendix on value partition strategies) and Algorithm 2 ("Partition for
non-Transformers": one block per tensor) for CNNs, diffusion models and GNNs.

Shapes are [out_features, in_features]; a transposed or flattened weight must
be re-ordered by the caller first (the paper's appendix notes the same).
"""
from __future__ import annotations

from typing import Iterable, List, Sequence, Tuple

from . import binding
from .workloads import BF16, HEADS, ROWS, TOKENS, WHOLE, TensorSpec


def descriptors_from_named_shapes(named_shapes: Iterable[Tuple[str, Sequence[int]]], *, n_heads: int = 0,
                                  n_kv_heads: int = 0, grad_dtype: int = BF16, value_whole: bool = False,
                                  non_transformer: bool = False,
                                  no_decay: Sequence[str] = ()) -> List[TensorSpec]:
    """Tensor descriptors for `Partition`, in the order given.

    named_shapes     (name, shape) pairs, e.g. from model.named_parameters()
    n_heads          attention heads (blocks of a "query" tensor)
    n_kv_heads       heads of a "key" tensor under grouped-query attention (default: n_heads)
    value_whole      treat "value" tensors as one block each instead of per output neuron
    non_transformer  Algorithm 2: every tensor is one block
    no_decay         substrings of names exempt from weight decay (e.g. "norm", "bias")

    1-D tensors (norm weights, biases) are always one block.
    """
    out: List[TensorSpec] = []
    for name, shape in named_shapes:
        shape = [int(s) for s in shape]
        if not shape or any(s <= 0 for s in shape):
            raise ValueError(f"{name}: empty shape")
        rows = shape[0] if len(shape) > 1 else 1
        cols = 1
        for s in (shape[1:] if len(shape) > 1 else shape):
            cols *= s
        kind = WHOLE
        heads = 0
        if len(shape) > 1 and not non_transformer:
            kind = binding.kind_from_name(name)
            if kind == ROWS and value_whole and "value" in name:
                kind = WHOLE
            if kind == HEADS:
                heads = (n_kv_heads or n_heads) if "key" in name and "query" not in name else n_heads
                if heads <= 0 or rows % heads:
                    raise ValueError(f"{name}: {rows} rows do not split into {heads} heads")
        if kind == WHOLE:
            rows, cols = 1, rows * cols
        wd = 0 if any(s in name for s in no_decay) else 1
        out.append(TensorSpec(name, rows, cols, kind, n_heads=heads, grad_dtype=grad_dtype, apply_weight_decay=wd))
    return out
