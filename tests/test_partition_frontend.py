"""The (name, shape) front end against the workloads' hand-written descriptors
and the Python transcription of Algorithm 3 (no GPU)."""
import pytest

import paper_2406_16793_b200 as am
from oracle import partition_ref as pr
from paper_2406_16793_b200 import partition as P, workloads as W


def named_shapes(w):
    return [(t.name, (t.rows, t.cols) if t.rows > 1 else (t.cols,)) for t in w.tensors]


@pytest.mark.parametrize("w,heads,kv", [(W.llama3_8b(n_layers=2), 32, 8), (W.llama2_7b(n_layers=1), 32, 32),
                                        (W.gpt2_small(n_layers=2), 12, 12), (W.tiny_gpt2(), 4, 4)],
                         ids=lambda x: getattr(x, "name", str(x)))
def test_front_end_reproduces_the_workload_descriptors(w, heads, kv):
    got = P.descriptors_from_named_shapes(named_shapes(w), n_heads=heads, n_kv_heads=kv,
                                          grad_dtype=w.tensors[0].grad_dtype)
    assert [(t.rows, t.cols, t.kind, t.n_heads) for t in got] == [(t.rows, t.cols, t.kind, t.n_heads) for t in w.tensors]
    rows, total = am.Partition(got).export()
    assert total == w.n_blocks
    for t, r in zip(got, rows):                      # kinds follow Algorithm 3's name tests for 2-D tensors
        assert r.kind == (pr.kind_from_name(t.name) if t.rows > 1 else pr.WHOLE)


def test_value_as_a_whole_and_non_transformer_variants():
    w = W.llama2_7b(n_layers=1)
    whole_v = P.descriptors_from_named_shapes(named_shapes(w), n_heads=32, value_whole=True)
    for t, ref in zip(whole_v, w.tensors):
        if "value" in t.name:
            assert t.kind == W.WHOLE and t.n_blocks == 1 and t.numel == ref.numel
        else:
            assert t.kind == ref.kind
    alg2 = P.descriptors_from_named_shapes(named_shapes(w), non_transformer=True)
    assert all(t.kind == W.WHOLE and t.n_blocks == 1 for t in alg2)     # Algorithm 2: one block per tensor
    assert sum(t.numel for t in alg2) == w.numel


def test_decay_exemptions_and_errors():
    got = P.descriptors_from_named_shapes([("layers.0.ffn_norm.weight", (64,)), ("layers.0.mlp.up.weight", (8, 64))],
                                          no_decay=("norm", "bias"))
    assert [t.apply_weight_decay for t in got] == [0, 1]
    with pytest.raises(ValueError):
        P.descriptors_from_named_shapes([("attention.query.weight", (10, 4))], n_heads=3)
    with pytest.raises(ValueError):
        P.descriptors_from_named_shapes([("attention.query.weight", (12, 4))])          # head count missing
