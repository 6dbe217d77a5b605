"""Host-side checks of the CUDA library that need no GPU: the shared object
loads, exports every entry point the header declares, and its partitioner
produces bit-exactly the table the Python partition rules give."""
import ctypes
import os
import re

import pytest

import paper_2406_16793_b200 as am
from oracle import partition_ref as pr
from paper_2406_16793_b200 import binding, build, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "adammini.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adammini_\w+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    names = declared_functions()
    assert len(names) >= 16
    lib = ctypes.CDLL(binding.LIBRARY)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.exported_names()) == set(names)


def parts_workload():
    T = W.TensorSpec
    return W.Workload("parts", 80, [T("tail", 1, 1000, W.PART, fixed_block_len=4096, grad_dtype=W.BF16),
                                    T("rows", 6, 4096, W.ROWS, grad_dtype=W.BF16),
                                    T("head", 1, 3001, W.PART, fixed_block_len=11008, grad_dtype=W.BF16)],
                      W.GradRecipe(-4.0, -1.0), steps=2)


def workloads():
    return [W.tiny_gpt2(), W.gpt2_small(), W.llama2_7b(), W.llama3_8b(), parts_workload()] + \
           [W.flat_sweep(L) for L in (1, 128, 4096, 524288, 1 << 30)]


@pytest.mark.parametrize("w", workloads(), ids=lambda w: w.name)
def test_partition_table_is_bit_exact(w):
    part = am.Partition(w.tensors)
    rows, total = part.export()
    want, want_total = pr.build_table([
        pr.TensorDesc(t.rows, t.cols, t.kind, t.n_heads, t.fixed_block_len, t.grad_dtype, t.apply_weight_decay)
        for t in w.tensors])
    assert total == want_total and len(rows) == len(want)
    for got, ref in zip(rows, want):
        assert (got.numel, got.block_len, got.n_blocks, got.v_offset, got.kind, got.grad_dtype, got.wd, got.mean_len) == \
               (ref.numel, ref.block_len, ref.n_blocks, ref.v_offset, ref.kind, ref.grad_dtype, ref.wd, ref.mean_len)
    part.close()


def test_name_rule_matches_algorithm3():
    names = ["embed_tokens.weight", "output.weight", "layers.0.attention.query.weight", "h.1.attn.key.weight",
             "h.1.attn.value.weight", "h.3.attn.proj.weight", "h.3.mlp.fc.weight", "ln_f.weight",
             "output_embed_query", "mlp.query", "norm"]
    for n in names:
        assert binding.kind_from_name(n) == pr.kind_from_name(n), n


def test_partition_rejects_bad_descriptors():
    bad = [
        W.TensorSpec("heads", 10, 4, W.HEADS, n_heads=3),
        W.TensorSpec("fixed", 1, 10, W.FIXED, fixed_block_len=4),
        W.TensorSpec("empty", 0, 4, W.ROWS),
    ]
    for t in bad:
        with pytest.raises(am.AdamMiniError) as e:
            am.Partition([t])
        assert e.value.status == -2
    with pytest.raises(am.AdamMiniError) as e:
        am.Partition([W.TensorSpec("dtype", 2, 2, W.ROWS, grad_dtype=7)])
    assert e.value.status == -1
    # sizes that overflow int64: one tensor (rows * cols), and the sum over tensors
    with pytest.raises(am.AdamMiniError) as e:
        am.Partition([W.TensorSpec("huge", 1 << 40, 1 << 40, W.ROWS)])
    assert e.value.status == -2
    with pytest.raises(am.AdamMiniError) as e:
        am.Partition([W.TensorSpec(f"t{i}", 1 << 62, 1, W.ROWS) for i in range(3)])
    assert e.value.status == -7


def test_status_strings():
    lib = binding.load()
    seen = {lib.adammini_status_string(s).decode() for s in range(-7, 1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert lib.adammini_status_string(-99).decode() == "unknown status"


def test_missing_library_fails_loudly(tmp_path):
    """Without the shared object the binding raises at once: there is no other path."""
    import subprocess
    import sys
    code = ("import paper_2406_16793_b200 as am\n"
            "from paper_2406_16793_b200 import workloads as W\n"
            "try:\n"
            "    am.Partition(W.tiny_gpt2().tensors)\n"
            "except RuntimeError as e:\n"
            "    assert 'missing' in str(e) and 'no CPU fallback' in str(e), e\n"
            "    print('raised')\n")
    env = dict(os.environ, ADAMMINI_LIBRARY=str(tmp_path / "libadammini.so"), PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == "raised", out.stderr


@pytest.mark.skipif(__import__("torch").cuda.is_available(), reason="checks the behaviour without a device")
def test_creating_a_handle_without_a_device_reports_a_cuda_error():
    part = am.Partition(W.tiny_gpt2().tensors)
    with pytest.raises(am.AdamMiniError) as e:
        am.AdamMini(part, lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
    assert e.value.status == -4
    assert binding.load().adammini_last_cuda_error(None) != 0          # which CUDA error it was
    assert "cudaError" in str(e.value)


def test_random_descriptors_agree_with_the_reference_partitioner():
    """2000 seeded random descriptors, valid and invalid: the library accepts
    exactly what the Python rules accept and exports the same row."""
    import numpy as np
    rng = np.random.default_rng(424242)
    accepted = rejected = 0
    batch = []
    for _ in range(2000):
        kind = int(rng.choice([W.WHOLE, W.ROWS, W.HEADS, W.TOKENS, W.FIXED, W.PART]))
        rows = int(rng.choice([0, 1, 1, 2, 3, 7, 12, 64, 300]))
        cols = int(rng.choice([0, 1, 5, 8, 24, 768, 4096, 100003]))
        n_heads = int(rng.choice([0, 1, 2, 3, 4, 12]))
        fixed = int(rng.choice([0, 1, 2, 4, 5, 8, 24, 4096, 1 << 20, 1 << 33]))
        d = pr.TensorDesc(rows, cols, kind, n_heads, fixed, int(rng.integers(0, 2)), int(rng.integers(0, 2)))
        try:
            want, _ = pr.build_table([d])
        except ValueError:
            want = None
        spec = W.TensorSpec("t", rows, cols, kind, n_heads=n_heads, fixed_block_len=fixed,
                            grad_dtype=d.grad_dtype, apply_weight_decay=d.apply_weight_decay)
        if want is None:
            with pytest.raises(am.AdamMiniError) as e:
                am.Partition([spec])
            assert e.value.status == -2, d
            rejected += 1
            continue
        batch.append((spec, d))
        accepted += 1
    assert accepted > 300 and rejected > 300
    # all accepted descriptors as one table: offsets accumulate the same way
    part = am.Partition([s for s, _ in batch])
    rows_got, total = part.export()
    want, want_total = pr.build_table([d for _, d in batch])
    assert total == want_total
    for got, ref in zip(rows_got, want):
        assert (got.numel, got.block_len, got.n_blocks, got.v_offset, got.kind, got.grad_dtype, got.wd, got.mean_len) == \
               (ref.numel, ref.block_len, ref.n_blocks, ref.v_offset, ref.kind, ref.grad_dtype, ref.wd, ref.mean_len)
    part.close()


def test_random_names_agree_with_the_reference_name_rule():
    import numpy as np
    rng = np.random.default_rng(7)
    words = ["embed", "output", "query", "key", "value", "attn.proj", "mlp", "attn", "proj", "norm", "weight", "bias",
             "layers", "wq", "lm_head", "tok", "fc", "0", "11", "."]
    for _ in range(500):
        name = "".join(rng.choice(words, size=int(rng.integers(1, 6))))
        assert binding.kind_from_name(name) == pr.kind_from_name(name), name


def test_cluster_size_follows_l2_size_and_resident_clusters():
    """The chooser on synthetic devices (no GPU): smallest cluster size whose resident
    clusters keep their blocks' gradients within a share of L2."""
    MB = 1 << 20
    b200 = [0, 148, 74, 45, 33, 26, 22, 15, 15]        # resident clusters of 1..8 CTAs, 126 MB of L2
    choose = lambda caps, l2, block: binding.choose_cluster_size(caps, l2, block)
    assert choose(b200, 126 * MB, 1 * MB) == 6          # bf16 heads of 128 x 4096: 22 x 1 MB is within the share, 26 x 1 MB not
    assert choose(b200, 126 * MB, 2 * MB) == 8          # the same heads with float32 gradients
    assert choose(b200, 126 * MB, 4 * MB) == 8          # nothing fits the share: the largest size
    assert choose(b200, 126 * MB, 3 * MB) == 8          # 7 keeps no more clusters than 8: passed over
    assert choose(b200, 126 * MB, 320 * 1024) == 3      # 74 x 0.31 MB is just over the share, 45 x 0.31 MB within
    assert choose(b200, 126 * MB, 512 * 1024) == 3      # 45 x 0.5 MB
    # monotone in the block size and in the L2 size
    sizes = [choose(b200, 126 * MB, k * 64 * 1024) for k in range(4, 65)]
    assert sizes == sorted(sizes)
    by_l2 = [choose(b200, l2 * MB, 1 * MB) for l2 in (32, 64, 126, 256, 512, 2048)]
    assert by_l2 == sorted(by_l2, reverse=True) and by_l2 == [8, 8, 6, 3, 2, 1]
    # a device half the size with twice the cache per SM keeps smaller clusters
    small = [0, 74, 37, 24, 18, 14, 12, 10, 9]
    assert choose(small, 126 * MB, 1 * MB) == 4
    # clusters of some sizes cannot run; none at all -> 0 (the two-pass kernels take such blocks)
    assert choose([0, 148, 74, 0, 33, 0, 0, 0, 0], 126 * MB, 2 * MB) == 4
    assert choose([0] * 9, 126 * MB, 1 * MB) == 0
    assert choose(b200, 0, 1 * MB) == 8                 # unknown L2 size: the most conservative choice
