"""The Python partition rules against the paper's counts (no GPU)."""
import os

import pytest

from oracle import partition_ref as pr
from paper_2406_16793_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def descs_of(w):
    return [pr.TensorDesc(t.rows, t.cols, t.kind, t.n_heads, t.fixed_block_len,
                          t.grad_dtype, t.apply_weight_decay) for t in w.tensors]


def table1():
    out = {}
    for line in open(os.path.join(GOLDEN, "table1_optimizer_memory.txt")):
        if line.strip() and not line.startswith("#"):
            name, adamw, mini = line.split()
            out[name] = (float(adamw), float(mini))
    return out


@pytest.mark.parametrize("model,workload", [("Llama-2-7B", W.llama2_7b), ("Llama-3-8B", W.llama3_8b)])
def test_parameter_counts_match_table1(model, workload):
    """Table 1: AdamW's m+v take 8 bytes per parameter in float32; Adam-mini
    keeps m (4 bytes per parameter) and one float per block."""
    adamw_gb, mini_gb = table1()[model]
    rows, n_blocks = pr.build_table(descs_of(workload()))
    n = sum(r.numel for r in rows)
    assert abs(8 * n / 1e9 - adamw_gb) < 0.015
    assert abs((4 * n + 4 * n_blocks) / 1e9 - mini_gb) < 0.015
    # "cuts down >= 99.9% of Adam's v" for mainstream LLMs
    assert n_blocks / n <= 1e-3


def test_block_counts_follow_algorithm3():
    w = W.llama3_8b(n_layers=1)
    rows, total = pr.build_table(descs_of(w))
    by_name = {t.name: r for t, r in zip(w.tensors, rows)}
    assert by_name["embed_tokens.weight"].n_blocks == 128256          # tokens
    assert by_name["output.weight"].block_len == 4096
    assert by_name["layers.0.attention.query.weight"].n_blocks == 32  # heads
    assert by_name["layers.0.attention.key.weight"].n_blocks == 8     # KV heads
    assert by_name["layers.0.attention.key.weight"].block_len == 128 * 4096
    assert by_name["layers.0.attention.value.weight"].n_blocks == 1024  # output neurons
    assert by_name["layers.0.mlp.down.weight"].block_len == 14336
    assert by_name["layers.0.mlp.gate.weight"].n_blocks == 14336
    assert by_name["layers.0.ffn_norm.weight"].n_blocks == 1           # whole tensor
    assert total == sum(r.n_blocks for r in rows)
    offs = 0
    for r in rows:
        assert r.v_offset == offs
        offs += r.n_blocks


def test_workload_kinds_agree_with_name_rule():
    """The kinds written into the workloads are what Algorithm 3's name tests
    give for 2-D tensors; 1-D tensors are whole-tensor blocks."""
    for w in (W.tiny_gpt2(), W.gpt2_small(n_layers=2), W.llama2_7b(n_layers=1), W.llama3_8b(n_layers=1)):
        for t in w.tensors:
            want = pr.kind_from_name(t.name) if t.rows > 1 else pr.WHOLE
            assert t.kind == want, t.name


def test_totals_of_the_five_workloads():
    assert (W.tiny_gpt2().numel, W.tiny_gpt2().n_blocks, len(W.tiny_gpt2().tensors)) == (656640, 3866, 24)
    assert (W.gpt2_small().numel, W.gpt2_small().n_blocks, len(W.gpt2_small().tensors)) == (124475904, 116250, 196)
    assert (W.llama2_7b().numel, W.llama2_7b().n_blocks) == (6738415616, 1163841)
    assert (W.llama3_8b().numel, W.llama3_8b().n_blocks) == (8030261248, 1470273)
    for L, nb in ((1, 1 << 30), (128, 1 << 23), (4096, 1 << 18), (524288, 2048), (1 << 30, 1)):
        rows, total = pr.build_table(descs_of(W.flat_sweep(L)))
        assert total == nb and rows[0].block_len == L


def test_rejects_indivisible_shapes():
    with pytest.raises(ValueError):
        pr.build_table([pr.TensorDesc(10, 4, pr.HEADS, n_heads=3)])
    with pytest.raises(ValueError):
        pr.build_table([pr.TensorDesc(1, 10, pr.FIXED, fixed_block_len=4)])


def test_name_rule_precedence():
    """Algorithm 3 tests the names in a fixed order: embed/output first, then
    query/key, then value/attn.proj/mlp; anything else is one block."""
    assert pr.kind_from_name("output_embed_query") == pr.TOKENS
    assert pr.kind_from_name("embed.key") == pr.TOKENS
    assert pr.kind_from_name("mlp.query") == pr.HEADS
    assert pr.kind_from_name("attn.value.key") == pr.HEADS
    assert pr.kind_from_name("h.0.attn.value") == pr.ROWS
    assert pr.kind_from_name("h.0.attn.proj") == pr.ROWS
    assert pr.kind_from_name("h.0.mlp.fc") == pr.ROWS
    assert pr.kind_from_name("lm_output") == pr.TOKENS
    assert pr.kind_from_name("ln_f") == pr.WHOLE and pr.kind_from_name("attn.c_proj") == pr.WHOLE
