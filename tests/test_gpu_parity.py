"""GPU parity: the CUDA library against the float64 oracle, element by element,
on the same seeded inputs, through the C ABI."""
import os

import numpy as np
import pytest
import torch

import harness as H
import paper_2406_16793_b200 as am
from paper_2406_16793_b200 import binding as B, workloads as W

pytestmark = pytest.mark.gpu

TWOPASS = {B.OPT_PATH: 1}


def test_tiny_gpt2_ten_steps():
    """2-layer GPT-2-style model, fp32 gradients, 10 steps."""
    H.assert_parity(H.run_parity(W.tiny_gpt2()))


def test_tiny_gpt2_two_pass_anchor():
    H.assert_parity(H.run_parity(W.tiny_gpt2(), options=TWOPASS))


def test_gpt2_small_hundred_steps():
    """GPT-2-small shapes (two layers, vocabulary rows cut to 4096), bf16 gradients, 100 steps."""
    w = W.scaled_rows(W.gpt2_small(n_layers=2), 4096)
    H.assert_parity(H.run_parity(w, steps=100))


def test_llama2_block_lengths():
    """Every block length of Llama-2-7B (4096, 11008, 524288-element heads), rows cut to 256."""
    w = W.scaled_rows(W.llama2_7b(n_layers=1), 256)
    H.assert_parity(H.run_parity(w))


def test_llama3_gqa_block_lengths():
    """Llama-3-8B shapes with grouped KV heads and Zipf row magnitudes, rows cut to 384."""
    w = W.scaled_rows(W.llama3_8b(n_layers=1), 384)
    H.assert_parity(H.run_parity(w))


@pytest.mark.parametrize("L", [1, 128, 4096, 524288, 1 << 22])
def test_flat_partition_sweep(L):
    """One flat fp32 tensor of 2^22 elements cut into blocks of every degenerate length."""
    H.assert_parity(H.run_parity(W.flat_sweep(L, numel=1 << 22)))


@pytest.mark.parametrize("L", [1, 128, 4096])
def test_flat_sweep_two_pass_anchor(L):
    H.assert_parity(H.run_parity(W.flat_sweep(L, numel=1 << 20), options=TWOPASS))


def ragged_workload(grad_dtype):
    """Block lengths that exercise every path and tail: tiny, unaligned, packed
    with a ragged last stage, long single-CTA rows with a ragged last chunk."""
    T = W.TensorSpec
    gd = dict(grad_dtype=grad_dtype)
    tensors = [
        T("l1", 1, 1027, W.FIXED, fixed_block_len=1, **gd),
        T("l3", 7, 3, W.ROWS, **gd),
        T("l16", 129, 16, W.ROWS, **gd),
        T("l17", 33, 17, W.ROWS, **gd),
        T("l24", 1025, 24, W.ROWS, **gd),
        T("l36", 77, 36, W.ROWS, **gd),
        T("l40", 1031, 40, W.ROWS, **gd),
        T("l1000", 13, 1000, W.ROWS, **gd),
        T("l1001", 5, 1001, W.ROWS, **gd),
        T("l1032", 9, 1032, W.ROWS, **gd),
        T("l2056", 7, 2056, W.ROWS, **gd),
        T("l4104", 5, 4104, W.ROWS, **gd),
        T("l20488", 3, 20488, W.ROWS, **gd),
        T("whole50000", 1, 50000, W.WHOLE, **gd),
        T("whole70001", 1, 70001, W.WHOLE, **gd),
        T("heads", 12, 1000, W.HEADS, n_heads=4, **gd),
        T("nowd", 64, 256, W.ROWS, apply_weight_decay=0, **gd),
        T("one", 1, 1, W.WHOLE, **gd),
    ]
    return W.Workload("ragged", 90 + grad_dtype, tensors, W.GradRecipe(-4.0, -1.0), steps=6)


@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
@pytest.mark.parametrize("options", [None, TWOPASS], ids=["auto", "twopass"])
def test_ragged_shapes(grad_dtype, options):
    H.assert_parity(H.run_parity(ragged_workload(grad_dtype), options=options))


@pytest.mark.parametrize("threads,groups", [(128, 1), (512, 1), (128, 2), (256, 1)])
def test_other_consumer_shapes(threads, groups):
    w = W.scaled_rows(W.llama2_7b(n_layers=1), 128)
    H.assert_parity(H.run_parity(w, steps=3, options={B.OPT_STREAM_THREADS: threads, B.OPT_STREAM_GROUPS: groups}))


def test_consumer_groups_give_identical_bits():
    w = W.scaled_rows(W.llama2_7b(n_layers=2, vocab=1024), 512)
    a = _run_steps(w, 1, 3)
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w, {B.OPT_STREAM_GROUPS: 1})
    for t in (1, 2, 3):
        dev.draw_grads(t)
        opt.step(dev.p, dev.g, dev.m, dev.v, t)
    opt.sync_status()
    opt.close()
    assert _same(a, dev)


@pytest.mark.parametrize("cluster", [1, 2, 3, 4, 5, 6, 7])
def test_other_cluster_sizes(cluster):
    w = W.Workload("heads", 77, [W.TensorSpec("q", 1024, 4096, W.HEADS, n_heads=8, grad_dtype=W.BF16)],
                   W.GradRecipe(-5.0, -1.0), steps=3)
    H.assert_parity(H.run_parity(w, options={B.OPT_CLUSTER_SIZE: cluster}))


def test_zero_gradient_rows_and_an_infinity():
    """Rows with all-zero gradients keep v = 0 and take no Adam step; an
    infinite and a NaN gradient propagate exactly as in the oracle (no skip, no clip)."""
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=512), 64)

    def mutate(step, grads):
        grads[0].view(-1, 4096)[3:9].zero_()          # embedding rows of unseen tokens
        grads[4].view(-1, 4096)[5].zero_()
        if step == 2:
            grads[5].view(-1)[12345] = float("inf")
        if step == 3:
            grads[7].view(-1)[4096 * 3 + 17] = float("nan")      # poisons exactly one block (row 3)

    H.assert_parity(H.run_parity(w, steps=4, mutate_grads=mutate))


def test_learning_rate_schedule():
    sched = lambda t: 1e-3 * min(1.0, t / 3.0) * (0.9 ** t)
    H.assert_parity(H.run_parity(W.tiny_gpt2(), steps=8, lr_schedule=sched))


def test_other_hyperparameters():
    H.assert_parity(H.run_parity(W.tiny_gpt2(), steps=5,
                                 hp_override=dict(lr=3e-4, beta1=0.8, beta2=0.999, eps=1e-6, weight_decay=0.0)))


def _run_steps(w, first, last, state=None, stream=None):
    dev = state or H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w)
    for t in range(first, last + 1):
        dev.draw_grads(t)
        if stream is None:
            opt.step(dev.p, dev.g, dev.m, dev.v, t)
        else:
            stream.wait_stream(torch.cuda.current_stream())
            opt.step(dev.p, dev.g, dev.m, dev.v, t, stream=stream.cuda_stream)
            torch.cuda.current_stream().wait_stream(stream)
    opt.sync_status(stream.cuda_stream if stream is not None else 0)
    opt.close()
    return dev


def _same(a, b):
    return all(torch.equal(x, y) for x, y in zip(a.p + a.m + [a.v], b.p + b.m + [b.v]))


def test_deterministic_and_resumable():
    """Two runs give identical bits; 10 steps equal 5 steps, a new handle, 5 more
    (the state is only p, m, v and the step number)."""
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=256), 128)
    a = _run_steps(w, 1, 10)
    b = _run_steps(w, 1, 10)
    assert _same(a, b)
    c = _run_steps(w, 1, 5)
    c = _run_steps(w, 6, 10, state=c)
    assert _same(a, c)


def test_runs_on_a_side_stream():
    w = W.tiny_gpt2()
    a = _run_steps(w, 1, 3)
    b = _run_steps(w, 1, 3, stream=torch.cuda.Stream())
    assert _same(a, b)


def test_argument_errors():
    w = W.tiny_gpt2()
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w)
    with pytest.raises(am.AdamMiniError) as e:
        opt.step(dev.p, dev.g, dev.m, dev.v, 0)
    assert e.value.status == -1
    bad = list(dev.p)
    bad[3] = dev.p[3][1:]                                  # 4-byte offset: not 16-byte aligned
    with pytest.raises(am.AdamMiniError) as e:
        opt.step(bad, dev.g, dev.m, dev.v, 1)
    assert e.value.status == -3
    nul = [t.data_ptr() for t in dev.m]
    nul[0] = 0
    with pytest.raises(am.AdamMiniError) as e:
        opt.step(dev.p, dev.g, nul, dev.v, 1)
    assert e.value.status == -1
    for kw in (dict(eps=0.0), dict(beta1=1.0), dict(beta2=-0.1), dict(lr=-1.0), dict(weight_decay=float("nan"))):
        with pytest.raises(am.AdamMiniError):
            am.AdamMini(am.Partition(w.tensors), **kw)
    opt.close()


def test_launch_options_are_validated():
    """Consumer groups are whole warps: thread counts that are not a multiple of 32
    from 64 to 512 (and absurd CTA counts) are refused before anything is planned or
    launched, and the handle keeps working with the plan it had."""
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=256), 128)
    ref = _run_steps(w, 1, 2)
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w)
    before = [opt.query(q) for q in (B.Q_LAUNCHES_PER_STEP, B.Q_STREAM_CTAS, B.Q_CLUSTER_SIZE, B.Q_SCRATCH_BYTES)]
    for key, bad in ((B.OPT_STREAM_THREADS, 48), (B.OPT_STREAM_THREADS, 100), (B.OPT_STREAM_THREADS, 1000),
                     (B.OPT_STREAM_THREADS, 32), (B.OPT_STREAM_CTAS, 1 << 20), (B.OPT_STREAM_GROUPS, 3),
                     (B.OPT_CLUSTER_SIZE, 9), (B.OPT_STATISTIC, 5), (B.OPT_PATH, 2)):
        with pytest.raises(am.AdamMiniError) as e:
            opt.set_option(key, bad)
        assert e.value.status == -1, (key, bad)
    assert before == [opt.query(q) for q in (B.Q_LAUNCHES_PER_STEP, B.Q_STREAM_CTAS, B.Q_CLUSTER_SIZE, B.Q_SCRATCH_BYTES)]
    for t in (1, 2):
        dev.draw_grads(t)
        opt.step(dev.p, dev.g, dev.m, dev.v, t)
    opt.sync_status()
    opt.close()
    assert _same(ref, dev)


def test_cluster_shape_follows_the_device():
    """The cluster size of a table is what the chooser gives for the properties the handle
    read from this device; on a B200 (148 SMs, 126 MB of L2) that is 22 clusters of 6 for
    bf16 heads of 128 x 4096 and 15 clusters of 8 for the same heads with float32 gradients."""
    for gd, block_bytes, on_b200 in ((W.BF16, 1 << 20, (22, 6)), (W.F32, 2 << 20, (15, 8))):
        w = W.Workload("heads", 78, [W.TensorSpec("q", 8192, 4096, W.HEADS, n_heads=64, grad_dtype=gd)],
                       W.GradRecipe(-5.0, -1.0), steps=1)
        opt = H.make_optimizer(w)
        resident = [0] + [opt.query(B.Q_RESIDENT_CLUSTERS + c - 1) for c in range(1, 9)]
        l2, smem = opt.query(B.Q_L2_BYTES), opt.query(B.Q_SMEM_BYTES)
        want = B.choose_cluster_size(resident, l2, block_bytes)
        assert want >= 1 and opt.query(B.Q_CLUSTER_SIZE) == want
        assert opt.query(B.Q_CLUSTER_COUNT) == min(resident[want], w.n_blocks)
        props = torch.cuda.get_device_properties(0)
        assert l2 == props.L2_cache_size and smem >= 48 * 1024
        if "B200" in props.name and props.multi_processor_count == 148:
            assert (opt.query(B.Q_CLUSTER_COUNT), opt.query(B.Q_CLUSTER_SIZE)) == on_b200, (resident, l2)
        opt.set_option(B.OPT_CLUSTER_SIZE, 7)               # a caller's size is kept when it can run
        assert opt.query(B.Q_CLUSTER_SIZE) == max(c for c in range(1, 8) if resident[c] > 0)
        opt.close()


def test_empty_partition_and_queries():
    opt = am.AdamMini(am.Partition([]))
    opt.step([], [], [], 0, 1)
    opt.close()
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=256), 128)
    opt = H.make_optimizer(w)
    n = opt.query(B.Q_TOTAL_ELEMENTS)
    assert n == w.numel and opt.query(B.Q_TOTAL_BLOCKS) == w.n_blocks
    assert opt.query(B.Q_ELEMENTS_STREAM) + opt.query(B.Q_ELEMENTS_CLUSTER) == n
    assert opt.query(B.Q_ELEMENTS_CLUSTER) == 2 * 128 * 4096
    assert opt.query(B.Q_LAUNCHES_PER_STEP) == 2
    assert opt.query(B.Q_ALGORITHMIC_BYTES) == 18 * n + 8 * w.n_blocks
    opt.close()


def _host_step_equals_device_step(w, staging):
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w)
    hp = [x.cpu().pin_memory() for x in dev.p]
    hm = [x.cpu().pin_memory() for x in dev.m]
    hv = dev.v.cpu().pin_memory()
    for t in (1, 2, 3):
        dev.draw_grads(t)
        hg = [x.cpu() for x in dev.g]                       # pageable on purpose
        opt.step(dev.p, dev.g, dev.m, dev.v, t)
        opt.step_host(hp, hg, hm, hv, t, staging_bytes=staging)
        if t == 2:                                          # the staged handles follow an option change
            opt.set_option(B.OPT_STREAM_CHUNK, 3)
    opt.sync_status()
    for a, b in zip(dev.p + dev.m + [dev.v], hp + hm + [hv]):
        assert torch.equal(a.cpu(), b)
    opt.close()


@pytest.mark.parametrize("staging", [0, 3 * (24 << 20)], ids=["default-staging", "many-groups"])
def test_host_buffer_step_matches_device_step(staging):
    """adammini_step_host (state in host memory, streamed through staging slots)
    gives the same bits as adammini_step on device-resident state."""
    _host_step_equals_device_step(W.scaled_rows(W.llama2_7b(n_layers=1, vocab=512), 128), staging)


def test_host_buffer_step_keeps_the_cluster_size_of_the_whole_table():
    """Heads of 0.35 MB and of 1.3 MB land in different staging groups; on its own
    the first would run on smaller clusters than the table as a whole does, and its
    sums would round differently."""
    T = W.TensorSpec
    bf = dict(grad_dtype=W.BF16)
    tensors = [T("rows", 300, 768, W.ROWS, **bf), T("head_a", 4, 179456, W.ROWS, **bf),
               T("whole", 1, 2319092, W.WHOLE, **bf), T("head_b", 4, 640128, W.ROWS, **bf),
               T("tail", 150, 1424, W.ROWS, **bf)]
    w = W.Workload("two-head-sizes", 77, tensors, W.GradRecipe(-4.0, -1.0), steps=3)
    _host_step_equals_device_step(w, 3 * (40 << 20))


def test_full_size_llama2_7b_sampled_blocks():
    """All 6.74 G parameters of the Llama-2-7B shape set, stepped exactly as the
    benchmark steps them; the oracle recomputes sampled blocks of every kind
    (token rows, heads, output-neuron rows of 4096 and 11008, norms) from the
    first, a middle and the last layer."""
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 75 * (1 << 30):
        pytest.skip("needs about 70 GB of free device memory")
    w = W.llama2_7b()
    picks = [0, len(w.tensors) - 1, len(w.tensors) - 2]
    for layer in (0, 17, 31):
        picks += list(range(1 + 9 * layer, 1 + 9 * (layer + 1)))
    worst = H.run_sampled_parity(w, steps=w.steps, tensor_indices=picks, blocks_per_tensor=3)     # 20 steps
    assert worst["blocks"] >= 60
    H.assert_parity(worst)


@pytest.mark.parametrize("chunk", [1, 7, 1000000])
def test_dynamic_work_distribution_gives_identical_bits(chunk):
    w = W.scaled_rows(W.llama2_7b(n_layers=2, vocab=1024), 512)
    a = _run_steps(w, 1, 3)
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w, {B.OPT_STREAM_CHUNK: chunk})
    for t in (1, 2, 3):
        dev.draw_grads(t)
        opt.step(dev.p, dev.g, dev.m, dev.v, t)
    opt.sync_status()
    opt.close()
    assert _same(a, dev)


def test_gpt2_small_full_model_hundred_steps():
    """All 124 M parameters of the GPT-2-small shape set (196 tensors, bf16
    gradients), 100 steps, every element compared with the oracle."""
    H.assert_parity(H.run_parity(W.gpt2_small(), steps=100))


def _need_free_memory(gib):
    torch.cuda.empty_cache()                # memory cached by earlier tests counts as free
    free, _ = torch.cuda.mem_get_info()
    if free < gib * (1 << 30):
        pytest.skip(f"needs about {gib} GiB of free device memory")


def test_full_size_llama3_8b_sampled_blocks():
    """All 8.03 G parameters of the Llama-3-8B shape set (grouped KV heads,
    14336-element rows, Zipf-scaled vocabulary rows), stepped as the benchmark
    steps them; the oracle recomputes sampled blocks of every kind."""
    _need_free_memory(90)
    w = W.llama3_8b()
    picks = [0, len(w.tensors) - 1, len(w.tensors) - 2]
    for layer in (0, 31):
        picks += list(range(1 + 9 * layer, 1 + 9 * (layer + 1)))
    worst = H.run_sampled_parity(w, steps=w.steps, tensor_indices=picks, blocks_per_tensor=3)     # 20 steps
    assert worst["blocks"] >= 40
    H.assert_parity(worst)


@pytest.mark.parametrize("L", [1, 128, 4096, 524288])
def test_full_size_flat_sweep_sampled_blocks(L):
    """One flat fp32 tensor of 2^30 elements at every block length of the
    partition-degeneracy sweep; the oracle recomputes sampled runs of blocks."""
    _need_free_memory(20)
    w = W.flat_sweep(L)
    if L < 4096:
        # sample runs of 4096/L consecutive blocks by viewing them as one tensor of short blocks
        worst = H.run_sampled_runs(w, steps=w.steps, run_elems=4096, n_runs=24)                   # 10 steps
    else:
        worst = H.run_sampled_parity(w, steps=w.steps, tensor_indices=[0], blocks_per_tensor=6)
    H.assert_parity(worst)


def test_full_size_whole_tensor_block():
    """2^30 elements as ONE block (the two-pass path at full size): the oracle
    runs the whole tensor for the ten steps of the partition-degeneracy sweep."""
    _need_free_memory(20)
    w = W.flat_sweep(1 << 30)
    assert w.steps == 10
    H.assert_parity(H.run_parity(w))


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_ranks_tile_the_unsharded_step(world):
    """Whole-block sharding: every rank's share is stepped on its own (here one
    after the other on the one GPU; the shares do not interact), and together
    they must reproduce the unsharded step bit for bit."""
    from paper_2406_16793_b200 import sharding
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=300), 200)
    ref = _run_steps(w, 1, 3)
    dev = H.DeviceState(w, guarded=False)
    ranks = [sharding.ShardedStep(w.tensors, world, r, **w.hparams) for r in range(world)]
    v_local = [torch.zeros(max(r.local_blocks, 1), device="cuda") for r in ranks]
    for t in (1, 2, 3):
        dev.draw_grads(t)
        for r, v in zip(ranks, v_local):
            r.step(dev.p, dev.g, dev.m, v, t)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(ref.p + ref.m, dev.p + dev.m))
    v_all = torch.cat([v[:r.local_blocks] for r, v in zip(ranks, v_local)])
    assert torch.equal(v_all, ref.v)
    for r in ranks:
        r.close()


def test_profile_ring_reports_per_family_times():
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=256), 128)
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w)
    with pytest.raises(am.AdamMiniError):
        opt.get_profile()                                   # profiling is off
    opt.set_option(B.OPT_PROFILE, 4)
    for t in range(1, 7):
        dev.draw_grads(t)
        opt.step(dev.p, dev.g, dev.m, dev.v, t)
    ms, n = opt.get_profile()
    assert n == 4                                           # the ring keeps the latest 4 of 6 steps
    assert ms[0] < 0.05 and ms[3] < 0.05                    # no tiny blocks, nothing on the two-pass path
    assert 0.0 < ms[1] < 50.0 and 0.0 < ms[2] < 50.0        # streaming kernel and cluster kernel ran
    opt.set_option(B.OPT_PROFILE, 0)
    opt.close()


def test_new_buffers_every_step():
    """Callers may hand in different gradient (and state) buffers at every step:
    the library re-reads the addresses each call."""
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=256), 128)
    ref = _run_steps(w, 1, 4)
    dev = H.DeviceState(w, guarded=False)
    opt = H.make_optimizer(w)
    for t in range(1, 5):
        dev.draw_grads(t)
        grads = [g.clone() for g in dev.g]                 # fresh allocations
        if t == 3:                                         # and the state moves once
            dev.p = [x.clone() for x in dev.p]
            dev.m = [x.clone() for x in dev.m]
        opt.step(dev.p, grads, dev.m, dev.v, t)
        del grads
    opt.sync_status()
    opt.close()
    assert _same(ref, dev)


@pytest.mark.parametrize("L", [1, 4096, 0], ids=["L1", "L4096", "whole"])
def test_more_than_2_to_31_elements_in_one_tensor(L):
    """Element offsets beyond 32 bits: one tensor of 2^31 + 2^20 elements; the
    oracle recomputes runs at the very end (and start) of the tensor."""
    _need_free_memory(40)
    numel = (1 << 31) + (1 << 20)
    if L == 0:
        # one block: check v against a float64 sum of squares and a sampled update at the far end
        w = W.Workload("huge-whole", 71, [W.TensorSpec("t", 1, numel, W.WHOLE, grad_dtype=W.BF16)],
                       W.GradRecipe(-3.0, -1.0), steps=1)
        dev = H.DeviceState(w, guarded=False)
        opt = H.make_optimizer(w)
        dev.draw_grads(1)
        tail = slice(numel - 4096, numel)
        p0 = dev.p[0][tail].double().cpu().numpy()
        opt.step(dev.p, dev.g, dev.m, dev.v, 1)
        opt.sync_status()
        sum_sq = 0.0
        for lo in range(0, numel, 1 << 28):
            sum_sq += float(dev.g[0][lo:lo + (1 << 28)].double().square().sum())
        hp = w.hparams
        v_want = (1 - hp["beta2"]) * sum_sq / numel
        assert abs(float(dev.v[0]) - v_want) <= 1e-5 * v_want
        g = dev.g[0][tail].double().cpu().numpy()
        m_want = (1 - hp["beta1"]) * g
        denom = np.sqrt(v_want / (1 - hp["beta2"])) + hp["eps"]
        p_want = p0 * (1 - hp["lr"] * hp["weight_decay"]) - hp["lr"] * (m_want / (1 - hp["beta1"])) / denom
        assert H.block_relative_error(dev.m[0][tail].cpu().numpy(), m_want, 4096) <= H.TOL
        assert H.block_relative_error(dev.p[0][tail].cpu().numpy(), p_want, 4096) <= H.TOL
        opt.close()
        return
    w = W.Workload(f"huge-L{L}", 70, [W.TensorSpec("t", 1, numel, W.FIXED, fixed_block_len=L, grad_dtype=W.BF16)],
                   W.GradRecipe(-3.0, -1.0), steps=2)
    H.assert_parity(H.run_sampled_runs(w, steps=2, run_elems=4096, n_runs=12))


def _flat_model():
    T = W.TensorSpec
    bf = dict(grad_dtype=W.BF16)
    tensors = [
        T("embed", 300, 4096, W.TOKENS, **bf),
        T("query", 256, 4096, W.HEADS, n_heads=2, **bf),
        T("down", 40, 11008, W.ROWS, **bf),
        T("odd", 9, 1001, W.ROWS, **bf),
        T("short", 500, 36, W.ROWS, grad_dtype=W.F32),
        T("norm", 1, 4096, W.WHOLE, **bf),
        T("whole", 1, 3 << 20, W.WHOLE, **bf),
    ]
    return W.Workload("flat-shards", 62, tensors, W.GradRecipe(-4.0, -1.0), steps=3)


@pytest.mark.parametrize("world", [2, 3, 5])
def test_flat_shards_that_cut_blocks(world):
    """FSDP-style flat shards: every rank owns an equal contiguous range of the
    flat parameter space, blocks cut by a range boundary get their sum of g*g
    through one exchange of partial sums.  The ranks' shares are stepped one
    after the other on the one GPU (phase 1 of all, the exchange, phase 2 of
    all) and must match the oracle's unsharded run; blocks that no boundary
    cuts must equal the unsharded GPU run bit for bit."""
    from paper_2406_16793_b200 import sharding
    w = _flat_model()
    ref = _run_steps(w, 1, w.steps)
    dev = H.DeviceState(w, guarded=True)
    ora = ostep_state(w, dev)
    ranks = [sharding.ShardedFlatStep(w.tensors, world, r, **w.hparams) for r in range(world)]
    assert sum(r.n_parts for r in ranks) >= 2                      # some block is cut
    v_local = [torch.zeros(max(r.local_blocks, 1), device="cuda") for r in ranks]
    for t in range(1, w.steps + 1):
        dev.draw_grads(t)
        # The ranks run one after the other here, so what the all-gather would return is put
        # together first (gradients do not change during a step); every rank then runs its
        # whole step() -- local sums, exchange, combine, apply -- with a stand-in exchange that
        # checks what the rank contributes and hands back the gathered rows.
        gathered = torch.stack([r.local_sums(dev.g).clone() for r in ranks])
        for k, (r, v) in enumerate(zip(ranks, v_local)):
            def exchange(local, k=k):
                assert torch.equal(local, gathered[k])
                return gathered
            r.step(dev.p, dev.g, dev.m, v, t, exchange)
        H.oracle_step_all(ora, [g.cpu() for g in dev.g], t, w.hparams)
    torch.cuda.synchronize()
    assert dev.guards_intact()
    cut = set()
    for r in ranks:
        cut |= set(r.plan.part_keys)
    for i, spec in enumerate(w.tensors):
        L = spec.block_len
        assert H.block_relative_error(dev.p[i].cpu().numpy(), ora.p[i], L) <= H.TOL
        assert H.block_relative_error(dev.m[i].cpu().numpy(), ora.m[i], L) <= H.TOL
        same = (dev.p[i] == ref.p[i]).view(-1, L).all(dim=1).cpu()
        for b in range(spec.n_blocks):
            if (i, b) not in cut:
                assert bool(same[b]), (i, b)
    # every holder of a cut block keeps the same second moment, and it matches the oracle
    v_off = np.cumsum([0] + [t.n_blocks for t in w.tensors])
    for r, v in zip(ranks, v_local):
        k = 0
        for p in r.pieces:
            got = v[k:k + p.n_blocks].cpu().numpy()
            want = ora.v[p.tensor][p.block:p.block + p.n_blocks]
            assert H.v_relative_error(got, want) <= H.TOL
            k += p.n_blocks
    for r in ranks:
        r.close()


def ostep_state(w, dev):
    from oracle import step as ostep
    return ostep.OracleState([p.cpu() for p in dev.p], [t.block_len for t in w.tensors],
                             [bool(t.apply_weight_decay) for t in w.tensors])


def test_many_small_tensors_of_mixed_kinds():
    """Hundreds of small tensors of seeded random shapes, kinds and gradient
    dtypes in one table: segment walking, ragged last stages, the end of v."""
    rng = np.random.default_rng(20240616)
    cols_choices = [1, 3, 8, 24, 40, 128, 768, 1000, 1001, 3072, 4096, 5000, 11008]
    tensors = []
    for i in range(400):
        cols = int(rng.choice(cols_choices))
        rows = int(rng.integers(1, 40))
        gd = int(rng.integers(0, 2))
        kind = int(rng.choice([W.WHOLE, W.ROWS, W.TOKENS, W.HEADS, W.FIXED]))
        kw = {}
        if kind == W.HEADS:
            divs = [d for d in range(1, rows + 1) if rows % d == 0]
            kw["n_heads"] = int(rng.choice(divs))
        if kind == W.FIXED:
            n = rows * cols
            divs = [d for d in (1, 2, 4, 8, 16, cols, n) if n % d == 0]
            kw["fixed_block_len"] = int(rng.choice(divs))
        if kind == W.WHOLE:
            rows, cols = 1, rows * cols
        tensors.append(W.TensorSpec(f"t{i}", rows, cols, kind, grad_dtype=gd,
                                    apply_weight_decay=int(rng.integers(0, 2)), **kw))
    w = W.Workload("many-small", 63, tensors, W.GradRecipe(-4.0, -1.0), steps=3)
    H.assert_parity(H.run_parity(w))
    H.assert_parity(H.run_parity(w, steps=2, options={B.OPT_STREAM_CHUNK: 3}))


def _random_table(rng):
    """A seeded random table that mixes every path: thread-per-block, packed rows,
    block lengths that are not a multiple of 16 bytes, long single-CTA rows,
    cluster-sized blocks, whole tensors beyond the cluster limit, heads."""
    T = W.TensorSpec
    tensors, budget = [], 12_000_000
    for i in range(int(rng.integers(2, 14))):
        gd = int(rng.integers(0, 2))
        gsz = 2 if gd == W.BF16 else 4
        kw = dict(grad_dtype=gd, apply_weight_decay=int(rng.integers(0, 2)))
        cls = rng.choice(["small", "packed", "odd", "long", "cluster", "whole", "heads"])
        if cls == "small":
            t = T(f"t{i}", int(rng.integers(1, 3000)), int(rng.integers(1, 17)), W.ROWS, **kw)
        elif cls == "packed":
            L = int(rng.integers(3, 513)) * 8
            t = T(f"t{i}", int(rng.integers(1, max(2, 400000 // L))), L, W.ROWS, **kw)
        elif cls == "odd":
            L = int(rng.integers(17, 9000))
            t = T(f"t{i}", int(rng.integers(1, max(2, 200000 // L))), L, W.ROWS, **kw)
        elif cls == "long":
            L = int(rng.integers(513, (256 * 1024 // gsz) // 8 + 1)) * 8
            t = T(f"t{i}", int(rng.integers(1, 9)), L, W.ROWS, **kw)
        elif cls == "cluster":
            lo = (256 * 1024 // gsz) // 64 + 1
            L = int(rng.integers(lo, lo + 8001)) * 64
            t = T(f"t{i}", int(rng.integers(1, 5)), L, W.ROWS, **kw)
        elif cls == "heads":
            nh, rph, cols = int(rng.integers(1, 9)), int(rng.integers(1, 65)), int(rng.integers(1, 65)) * 8
            t = T(f"t{i}", nh * rph, cols, W.HEADS, n_heads=nh, **kw)
        else:
            t = T(f"t{i}", 1, int(rng.integers(1, 3_000_000)), W.WHOLE, **kw)
        if t.numel <= budget:
            budget -= t.numel
            tensors.append(t)
    return tensors or [T("t", 4, 64, W.ROWS)]


def _random_options(rng):
    o = {}
    for key, values in ((B.OPT_STREAM_THREADS, [128, 256, 512]), (B.OPT_STREAM_GROUPS, [1, 2]),
                        (B.OPT_CLUSTER_SIZE, [1, 2, 4, 8]), (B.OPT_STREAM_CHUNK, [1, 2, 5, 64, 1000000]),
                        (B.OPT_CLUSTER_CHUNK, [1, 2, 3, 1000000]), (B.OPT_STREAM_CTAS, [1, 3, 7, 37, 148])):
        if rng.random() < 0.5:
            o[key] = int(rng.choice(values))
    return o


def test_random_tables_and_launch_options():
    """Seeded random tables, each under random launch options, two steps.
    ADAMMINI_RANDOM_TABLES sets how many (default 40, a few seconds)."""
    for seed in range(int(os.environ.get("ADAMMINI_RANDOM_TABLES", "40"))):
        rng = np.random.default_rng(7000 + seed)
        w = W.Workload(f"random{seed}", 800 + seed, _random_table(rng), W.GradRecipe(-4.0, -1.0), steps=2)
        options = _random_options(rng)
        worst = H.run_parity(w, options=options)
        assert max(worst[k] for k in "pmv") <= H.TOL, (seed, options, worst)


@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_every_short_block_length(grad_dtype):
    """Block lengths 1..64, each over a few tiles of the short-block kernel plus a
    ragged last tile (whole blocks that end off any 16-byte boundary), with and
    without weight decay, against the oracle; then the same with a gradient scale,
    a bf16 copy and an ablation statistic, which take the same kernel."""
    tensors = [W.TensorSpec(f"l{L}", 3 * (4096 // L) + 5, L, W.ROWS, grad_dtype=grad_dtype, apply_weight_decay=L % 2)
               for L in range(1, 65)]
    w = W.Workload("short-blocks", 91 + grad_dtype, tensors, W.GradRecipe(-4.0, -1.0), steps=3)
    H.assert_parity(H.run_parity(w))
    H.assert_parity(H.run_parity(w, steps=2, statistic=B.STAT_TWO_NORM))
    # a bf16 copy does not change the float32 result and is its rounding
    a, b = H.DeviceState(w, guarded=False), H.DeviceState(w, guarded=True)
    copies = [H.Guarded(t.numel, torch.bfloat16, "cuda") for t in w.tensors]
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    a.draw_grads(1)
    for x, y in zip(a.g, b.g):
        y.copy_(x)
    oa.step(a.p, a.g, a.m, a.v, 1)
    ob.step_ex(b.p, b.g, b.m, b.v, 1, params_bf16=[c.view for c in copies])
    oa.sync_status(); ob.sync_status()
    assert _same(a, b) and b.guards_intact()
    for c, p in zip(copies, b.p):
        assert torch.equal(c.view, p.to(torch.bfloat16)) and c.intact()
    oa.close(); ob.close()


@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_blocks_of_two_and_three_elements(grad_dtype):
    """Blocks of two and three elements whose tensors are 16-byte aligned throughout run
    straight from registers (a thread takes 4 or 12 elements), several CTAs and a ragged
    last one; the same lengths at offsets of v or element counts that break the alignment
    stay on the tile kernel.  All against the oracle, also with an ablation statistic, a
    gradient scale and a bf16 copy."""
    gd = dict(grad_dtype=grad_dtype)
    T = W.TensorSpec
    tensors = [
        T("a2", 2 * 4096 * 3 + 2 * 18, 2, W.ROWS, **gd),                 # L = 2: twelve full CTAs of 4096 elements and 72 elements
        T("a3", 4 * 1024 * 2 + 4 * 7, 3, W.ROWS, apply_weight_decay=0, **gd),     # L = 3: eight full CTAs of 3072 elements and 84 elements
        T("a1", 1, 4096 + 8, W.FIXED, fixed_block_len=1, **gd),
        T("odd", 3, 5, W.ROWS, **gd),                                    # three blocks: what follows has an odd offset in v
        T("b2", 1000, 2, W.ROWS, **gd),                                  # v offset odd: tile kernel
        T("b3", 1001, 3, W.ROWS, **gd),                                  # 3003 elements: not a multiple of 12: tile kernel
        T("c2", 1001, 2, W.ROWS, **gd),                                  # 2002 elements: not a multiple of 4: tile kernel
    ]
    w = W.Workload("tiny-blocks", 97 + grad_dtype, tensors, W.GradRecipe(-4.0, -1.0), steps=4)
    opt = H.make_optimizer(w)
    assert opt.query(B.Q_LAUNCHES_PER_STEP) == 4                         # lengths 1, 2, 3 from registers + one launch of tiles
    assert opt.query(B.Q_ELEMENTS_SMALL) == w.numel
    opt.close()
    H.assert_parity(H.run_parity(w))
    for statistic in (B.STAT_MAX, B.STAT_MIN, B.STAT_ONE_NORM, B.STAT_TWO_NORM):
        H.assert_parity(H.run_parity(w, steps=2, statistic=statistic))
    a, b = H.DeviceState(w, guarded=False), H.DeviceState(w, guarded=True)
    copies = [H.Guarded(t.numel, torch.bfloat16, "cuda") for t in w.tensors]
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    a.draw_grads(1)
    for x, y in zip(a.g, b.g):
        y.copy_(x * 0.5)
    oa.step_ex(a.p, a.g, a.m, a.v, 1, grad_scale=0.5)
    ob.step_ex(b.p, b.g, b.m, b.v, 1, params_bf16=[c.view for c in copies])
    oa.sync_status(); ob.sync_status()
    assert _same(a, b) and b.guards_intact()
    for c, p in zip(copies, b.p):
        assert torch.equal(c.view, p.to(torch.bfloat16)) and c.intact()
    oa.close(); ob.close()


@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_unaligned_block_lengths_up_to_a_tile(grad_dtype):
    """Block lengths whose blocks start off the 16-byte grid, from just above the
    short-block limit to the tile size and one past it: several tiles each, so that
    tiles start at every offset within 32 bytes; with a bf16 copy and guards."""
    lengths = [65, 66, 67, 69, 100, 127, 255, 257, 1001, 1365, 2047, 4095, 4097]
    tensors = [W.TensorSpec(f"l{L}", max(3 * (4096 // L) + 3, 5), L, W.ROWS, grad_dtype=grad_dtype,
                            apply_weight_decay=i % 2) for i, L in enumerate(lengths)]
    w = W.Workload("unaligned-blocks", 93 + grad_dtype, tensors, W.GradRecipe(-4.0, -1.0), steps=3)
    H.assert_parity(H.run_parity(w))
    H.assert_parity(H.run_parity(w, steps=2, statistic=B.STAT_MAX))
    opt = H.make_optimizer(w)
    assert opt.query(B.Q_ELEMENTS_TWOPASS) == 0
    vec = 8 if grad_dtype == W.BF16 else 4                   # elements per 16 bytes of gradients
    on_tiles = sum(t.numel for t in tensors if t.cols <= 4096 and t.cols % vec)
    assert opt.query(B.Q_ELEMENTS_SMALL) == on_tiles and opt.query(B.Q_ELEMENTS_STREAM) == w.numel - on_tiles
    opt.close()
    a, b = H.DeviceState(w, guarded=False), H.DeviceState(w, guarded=True)
    copies = [H.Guarded(t.numel, torch.bfloat16, "cuda") for t in w.tensors]
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    a.draw_grads(1)
    for x, y in zip(a.g, b.g):
        y.copy_(x)
    oa.step(a.p, a.g, a.m, a.v, 1)
    ob.step_ex(b.p, b.g, b.m, b.v, 1, params_bf16=[c.view for c in copies], grad_scale=1.0)
    oa.sync_status(); ob.sync_status()
    assert _same(a, b) and b.guards_intact()
    for c, p in zip(copies, b.p):
        assert torch.equal(c.view, p.to(torch.bfloat16)) and c.intact()
    oa.close(); ob.close()


@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_long_blocks_with_unaligned_starts_are_read_once(grad_dtype):
    """Rows of more than 4096 elements whose byte length is not a multiple of 16 (so that
    rows start at every offset within 32 bytes) stay on the single-read streaming kernel:
    the aligned middle of every chunk is staged in shared memory, the up to seven elements
    either side come from global memory.  Lengths around the stage sizes, a few rows each;
    against the oracle, with guards, then with ablation statistics, a gradient scale and
    bf16 copies.  Rows beyond 256 KB of gradients take the two-pass kernels as before."""
    gsz = 2 if grad_dtype == W.BF16 else 4
    lengths = [4097, 4099, 4101, 4103, 8191, 8199, 8209, 10007, 20481, 20489, 24577, 50257, 65543, 131063]
    tensors = [W.TensorSpec(f"l{L}", 5 + i % 5, L, W.ROWS, grad_dtype=grad_dtype, apply_weight_decay=i % 2)
               for i, L in enumerate(lengths)]
    tensors.insert(3, W.TensorSpec("aligned", 7, 4104, W.ROWS, grad_dtype=grad_dtype))     # the ordinary launch beside it
    w = W.Workload("long-unaligned", 99 + grad_dtype, tensors, W.GradRecipe(-4.0, -1.0), steps=3)
    opt = H.make_optimizer(w)
    beyond = sum(t.numel for t in tensors if t.cols * gsz > 256 * 1024)
    assert opt.query(B.Q_ELEMENTS_TWOPASS) == beyond and opt.query(B.Q_ELEMENTS_STREAM) == w.numel - beyond
    assert opt.query(B.Q_LAUNCHES_PER_STEP) == 2 + (3 if beyond else 0)
    opt.close()
    H.assert_parity(H.run_parity(w))
    H.assert_parity(H.run_parity(w, steps=2, options={B.OPT_STREAM_CHUNK: 1, B.OPT_STREAM_THREADS: 128}))
    for statistic in (B.STAT_MAX, B.STAT_TWO_NORM):
        H.assert_parity(H.run_parity(w, steps=2, statistic=statistic))
    a, b = H.DeviceState(w, guarded=False), H.DeviceState(w, guarded=True)
    copies = [H.Guarded(t.numel, torch.bfloat16, "cuda") for t in w.tensors]
    oa, ob = H.make_optimizer(w), H.make_optimizer(w, {B.OPT_STREAM_CTAS: 5, B.OPT_STREAM_GROUPS: 1})
    for step in (1, 2):
        a.draw_grads(step)
        for x, y in zip(a.g, b.g):
            y.copy_(x * 0.5)
        oa.step_ex(a.p, a.g, a.m, a.v, step, grad_scale=0.5)
        ob.step_ex(b.p, b.g, b.m, b.v, step, params_bf16=[c.view for c in copies])
    oa.sync_status(); ob.sync_status()
    assert _same(a, b) and b.guards_intact()                   # whatever the CTAs and groups, the same bits
    for c, p in zip(copies, b.p):
        assert torch.equal(c.view, p.to(torch.bfloat16)) and c.intact()
    oa.close(); ob.close()


@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_long_unaligned_blocks_alone_and_beside_short_ones(grad_dtype):
    """Tiles of blocks of up to 64 elements and tiles of longer blocks are launched
    separately, each with its own shared-memory layout.  Rows of more than 64 elements
    must come out bit for bit the same from a table of their own and from one that
    also holds short blocks, with a gradient scale as well (long blocks apply it while
    reading the staged gradients), and both must match the oracle."""
    long_rows = [W.TensorSpec(f"l{L}", 3 * (4096 // L) + 2, L, W.ROWS, grad_dtype=grad_dtype) for L in (67, 255, 1001, 4095)]
    short_rows = [W.TensorSpec("s7", 2051, 7, W.ROWS, grad_dtype=grad_dtype)]
    alone = W.Workload("long-alone", 95 + grad_dtype, long_rows, W.GradRecipe(-4.0, -1.0), steps=3)
    mixed = W.Workload("long-alone", 95 + grad_dtype, long_rows + short_rows, W.GradRecipe(-4.0, -1.0), steps=3)
    H.assert_parity(H.run_parity(alone))
    H.assert_parity(H.run_parity(mixed))
    for scale in (None, 0.25):
        a, b = H.DeviceState(alone), H.DeviceState(mixed)
        oa, ob = H.make_optimizer(alone), H.make_optimizer(mixed)
        assert (oa.query(B.Q_LAUNCHES_PER_STEP), ob.query(B.Q_LAUNCHES_PER_STEP)) == (1, 2)
        for step in (1, 2):
            a.draw_grads(step); b.draw_grads(step)
            for i in range(len(long_rows)):
                assert torch.equal(a.g[i], b.g[i]) and (step > 1 or torch.equal(a.p[i], b.p[i]))
            if scale is None:
                oa.step(a.p, a.g, a.m, a.v, step); ob.step(b.p, b.g, b.m, b.v, step)
            else:
                oa.step_ex(a.p, a.g, a.m, a.v, step, grad_scale=scale); ob.step_ex(b.p, b.g, b.m, b.v, step, grad_scale=scale)
        oa.sync_status(); ob.sync_status()
        n_long = sum(t.n_blocks for t in long_rows)
        for i in range(len(long_rows)):
            assert torch.equal(a.p[i], b.p[i]) and torch.equal(a.m[i], b.m[i])
        assert torch.equal(a.v[:n_long], b.v[:n_long])
        assert a.guards_intact() and b.guards_intact()
        oa.close(); ob.close()
