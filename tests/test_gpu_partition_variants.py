"""GPU parity of tables built by the (name, shape) front end under the paper's
three partitions of a Transformer layer: Algorithm 3 as printed (value by output
neuron), the value-as-a-whole strategy of the appendix on value partition
strategies, and Algorithm 2 (one block per tensor, the partition for
non-Transformers).  Each table is stepped through the C ABI and compared with the
float64 oracle element by element; the kernel family every tensor lands on is
asserted, so that the whole-tensor blocks are seen to take the paths built for them."""
import pytest

import harness as H
from paper_2406_16793_b200 import binding as B, partition as P, workloads as W

pytestmark = pytest.mark.gpu

D, HEAD_DIM, ROWS_CUT = 4096, 128, 256


def layer_named_shapes():
    """One Llama-2-7B layer plus embedding, output and final norm.  `value` keeps its
    full 4096 x 4096; the other matrices are cut to 256 rows (two heads for query and
    key), which keeps every block length of the full model."""
    return [
        ("embed_tokens.weight", (ROWS_CUT, D)),
        ("layers.0.attention_norm.weight", (D,)),
        ("layers.0.attention.query.weight", (ROWS_CUT, D)),
        ("layers.0.attention.key.weight", (ROWS_CUT, D)),
        ("layers.0.attention.value.weight", (D, D)),
        ("layers.0.attn.proj.weight", (ROWS_CUT, D)),
        ("layers.0.ffn_norm.weight", (D,)),
        ("layers.0.mlp.gate.weight", (ROWS_CUT, D)),
        ("layers.0.mlp.up.weight", (ROWS_CUT, D)),
        ("layers.0.mlp.down.weight", (ROWS_CUT, 11008)),
        ("norm.weight", (D,)),
        ("output.weight", (ROWS_CUT, D)),
    ]


def family_elements(opt):
    return {k: opt.query(q) for k, q in (("small", B.Q_ELEMENTS_SMALL), ("stream", B.Q_ELEMENTS_STREAM),
                                         ("cluster", B.Q_ELEMENTS_CLUSTER), ("twopass", B.Q_ELEMENTS_TWOPASS))}


def run(specs, config_id):
    w = W.Workload("front-end", config_id, specs, W.GradRecipe(-5.0, -1.0, outlier_prob=0.01, outlier_scale=100.0), steps=3)
    opt = H.make_optimizer(w)
    fam = family_elements(opt)
    opt.close()
    H.assert_parity(H.run_parity(w))
    return w, fam


def test_algorithm3_default_partition():
    """Token rows, heads, output neurons, whole norms: Algorithm 3 as printed."""
    specs = P.descriptors_from_named_shapes(layer_named_shapes(), n_heads=ROWS_CUT // HEAD_DIM)
    kinds = {t.name.split(".")[-2]: (t.kind, t.block_len) for t in specs}
    assert kinds["query"] == (W.HEADS, HEAD_DIM * D) and kinds["key"] == (W.HEADS, HEAD_DIM * D)
    assert kinds["value"] == (W.ROWS, D) and kinds["down"] == (W.ROWS, 11008) and kinds["embed_tokens"] == (W.TOKENS, D)
    w, fam = run(specs, 41)
    heads = 2 * ROWS_CUT * D
    assert fam == {"small": 0, "stream": w.numel - heads, "cluster": heads, "twopass": 0}
    assert w.n_blocks == 5 * ROWS_CUT + D + 2 * (ROWS_CUT // HEAD_DIM) + 3 + ROWS_CUT


def test_value_as_a_whole():
    """Strategy (II) of the appendix: the value matrix is one block of 16.8 M elements
    (32 MB of bf16 gradients: beyond what a cluster keeps in L2, so g is read twice)."""
    specs = P.descriptors_from_named_shapes(layer_named_shapes(), n_heads=ROWS_CUT // HEAD_DIM, value_whole=True)
    value = [t for t in specs if "value" in t.name]
    assert len(value) == 1 and value[0].kind == W.WHOLE and value[0].block_len == D * D
    w, fam = run(specs, 42)
    heads = 2 * ROWS_CUT * D
    assert fam == {"small": 0, "stream": w.numel - heads - D * D, "cluster": heads, "twopass": D * D}


def test_algorithm2_one_block_per_tensor():
    """Partition for non-Transformers: every tensor is one block.  The cut matrices
    (1 M elements) run on the cluster kernel, value and mlp.down (2.8 M elements,
    5.6 MB of gradients) on the two-pass kernels, the norms on the streaming kernel."""
    specs = P.descriptors_from_named_shapes(layer_named_shapes(), non_transformer=True)
    assert all(t.kind == W.WHOLE and t.n_blocks == 1 for t in specs)
    w, fam = run(specs, 43)
    assert w.n_blocks == len(specs)
    assert fam == {"small": 0, "stream": 3 * D, "cluster": 7 * ROWS_CUT * D, "twopass": D * D + ROWS_CUT * 11008}
