"""The optional extras of adammini_step_ex: bf16 working copies of the updated
parameters, gradient scaling on load, and the device flag that skips a step."""
import numpy as np
import pytest
import torch

import harness as H
from oracle import step as ostep
from paper_2406_16793_b200 import binding as B, workloads as W
from test_gpu_parity import ragged_workload, _same

pytestmark = pytest.mark.gpu


mixed_workload = H.mixed_workload


def test_bf16_copy_is_the_rounded_parameter():
    """The bf16 copy must be the float32 result rounded to nearest even, for
    every kernel family; the float32 result itself must not change."""
    w = mixed_workload()
    a = H.DeviceState(w, guarded=False)
    b = H.DeviceState(w, guarded=True)
    copies = [H.Guarded(t.numel, torch.bfloat16, "cuda") for t in w.tensors]
    copies[2] = None                                            # entries may be absent
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    for t in (1, 2, 3):
        a.draw_grads(t)
        for x, y in zip(a.g, b.g):
            y.copy_(x)
        oa.step(a.p, a.g, a.m, a.v, t)
        ob.step_ex(b.p, b.g, b.m, b.v, t, params_bf16=[None if c is None else c.view for c in copies])
    oa.sync_status(); ob.sync_status()
    assert _same(a, b)
    for c, p in zip(copies, b.p):
        if c is not None:
            assert torch.equal(c.view, p.to(torch.bfloat16))
            assert c.intact()
    assert b.guards_intact()
    oa.close(); ob.close()


def test_power_of_two_gradient_scale_is_exact():
    """Scaling by 2^-10 on load equals stepping on gradients already scaled."""
    w = mixed_workload()
    a = H.DeviceState(w, guarded=False)
    b = H.DeviceState(w, guarded=False)
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    dev_two = torch.tensor([2.0], device="cuda")
    for t in (1, 2):
        a.draw_grads(t)
        for x, y in zip(a.g, b.g):
            y.copy_(x * (2.0 ** -10))
        oa.step_ex(a.p, a.g, a.m, a.v, t, grad_scale=2.0 ** -11, grad_scale_device=dev_two)
        ob.step(b.p, b.g, b.m, b.v, t)
    oa.sync_status(); ob.sync_status()
    assert _same(a, b)
    oa.close(); ob.close()


def test_gradient_scale_against_the_oracle():
    """An unscale factor that is not a power of two: the oracle steps on
    float64 gradients g * s, the GPU multiplies in float32 on load."""
    w = ragged_workload(W.BF16)
    dev = H.DeviceState(w)
    opt = H.make_optimizer(w)
    scale_host, scale_dev = 0.37, 1.0 / 3.0
    dscale = torch.tensor([scale_dev], device="cuda", dtype=torch.float32)
    s = float(np.float32(scale_host)) * float(np.float32(scale_dev))
    ora = ostep.OracleState([p.cpu() for p in dev.p], [t.block_len for t in w.tensors],
                            [bool(t.apply_weight_decay) for t in w.tensors])
    unit = {i: H.ShortBlockScale(ora.p[i]) for i, t in enumerate(w.tensors) if t.block_len < H.OWN_SCALE_MIN_L}
    for t in range(1, 5):
        dev.draw_grads(t)
        opt.step_ex(dev.p, dev.g, dev.m, dev.v, t, grad_scale=scale_host, grad_scale_device=dscale)
        for i, g in enumerate(dev.g):
            g64 = ostep.widen(g.cpu()) * s
            ostep.adammini_step(ora.p[i], ora.m[i], ora.v[i], g64, ora.block_lens[i], step=t,
                                apply_wd=ora.wd_flags[i], **w.hparams)
            if i in unit:
                unit[i].update(g64, ora.p[i], ora.m[i], w.hparams["beta1"])
    opt.sync_status()
    assert dev.guards_intact()
    worst = {"p": 0.0, "m": 0.0, "v": 0.0}
    v_gpu, off = dev.v.cpu().numpy(), 0
    for i, t in enumerate(w.tensors):
        u = unit.get(i)
        worst["p"] = max(worst["p"], H.block_relative_error(dev.p[i].cpu().numpy(), ora.p[i], t.block_len, u.p if u else None))
        worst["m"] = max(worst["m"], H.block_relative_error(dev.m[i].cpu().numpy(), ora.m[i], t.block_len, u.m if u else None))
        worst["v"] = max(worst["v"], H.v_relative_error(v_gpu[off:off + t.n_blocks], ora.v[i]))
        off += t.n_blocks
    H.assert_parity(worst)
    opt.close()


def test_skip_flag_leaves_the_state_untouched():
    w = mixed_workload()
    a = H.DeviceState(w, guarded=False)
    b = H.DeviceState(w, guarded=False)
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    flag = torch.zeros(1, device="cuda")
    a.draw_grads(1)
    for x, y in zip(a.g, b.g):
        y.copy_(x)
    oa.step(a.p, a.g, a.m, a.v, 1)
    ob.step_ex(b.p, b.g, b.m, b.v, 1, skip_flag=flag)           # flag clear: a normal step
    assert _same(a, b)
    before = [x.clone() for x in b.p + b.m + [b.v]]
    flag.fill_(1.0)                                             # e.g. an overflow was found in the gradients
    b.g[1].fill_(float("inf"))
    ob.step_ex(b.p, b.g, b.m, b.v, 2, skip_flag=flag)
    ob.sync_status()
    assert all(torch.equal(x, y) for x, y in zip(before, b.p + b.m + [b.v]))
    oa.close(); ob.close()


@pytest.mark.filterwarnings("ignore:The CUDA Graph is empty")
def test_a_capturing_stream_is_refused():
    """A step carries t and the learning rate as kernel arguments and alternates
    between two work counters, so a graph replay would repeat a stale step: the
    call refuses a stream that is being captured, enqueues nothing, and the
    handle steps normally afterwards."""
    w = mixed_workload()
    a = H.DeviceState(w, guarded=False)
    b = H.DeviceState(w, guarded=False)
    oa, ob = H.make_optimizer(w), H.make_optimizer(w)
    a.draw_grads(1)
    for x, y in zip(a.g, b.g):
        y.copy_(x)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    torch.cuda.synchronize()
    before = [x.clone() for x in b.p + b.m + [b.v]]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            with pytest.raises(B.AdamMiniError) as info:
                ob.step(b.p, b.g, b.m, b.v, 1, stream=side.cuda_stream)
        finally:
            graph.capture_end()
    assert info.value.status == -1                                # AM_ERR_INVALID_ARGUMENT
    torch.cuda.synchronize()
    assert all(torch.equal(x, y) for x, y in zip(before, b.p + b.m + [b.v]))
    oa.step(a.p, a.g, a.m, a.v, 1)
    ob.step(b.p, b.g, b.m, b.v, 1)
    ob.sync_status()
    assert _same(a, b)
    oa.close(); ob.close()


@pytest.mark.parametrize("statistic", [B.STAT_MAX, B.STAT_MIN, B.STAT_ONE_NORM, B.STAT_TWO_NORM],
                         ids=["max", "min", "one-norm", "two-norm"])
@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_ablation_statistics(statistic, grad_dtype):
    """The block statistics of the paper's ablation (max, min, 1-norm, 2-norm of
    g*g in place of the mean) against the oracle's variant routine."""
    H.assert_parity(H.run_parity(ragged_workload(grad_dtype), steps=4, statistic=statistic))


@pytest.mark.parametrize("statistic", [B.STAT_MAX, B.STAT_MIN, B.STAT_ONE_NORM, B.STAT_TWO_NORM],
                         ids=["max", "min", "one-norm", "two-norm"])
def test_ablation_statistics_on_model_shapes(statistic):
    """Llama-2-7B block lengths: the statistic is a parameter of the single-read
    reductions (packed rows, long rows re-read from L2, heads on clusters with the
    exchange through distributed shared memory), so nothing falls back to the
    two-pass kernels."""
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=128), 128)
    opt = H.make_optimizer(w, {B.OPT_STATISTIC: statistic})
    assert opt.query(B.Q_ELEMENTS_TWOPASS) == 0 and opt.query(B.Q_ELEMENTS_CLUSTER) == 2 * 128 * 4096
    assert opt.query(B.Q_LAUNCHES_PER_STEP) == 2
    opt.close()
    H.assert_parity(H.run_parity(w, steps=3, statistic=statistic))


def test_ablation_statistics_with_float32_heads_and_a_gradient_scale():
    """float32 gradients on clusters of six, consumer groups of other sizes, and a
    gradient scale that must come out as scale^2 on every statistic of g*g."""
    T = W.TensorSpec
    w = W.Workload("stat-f32", 66, [T("q", 256, 4096, W.HEADS, n_heads=2), T("rows", 40, 11008, W.ROWS),
                                    T("packed", 100, 2048, W.ROWS)], W.GradRecipe(-4.0, -1.0), steps=2)
    for statistic in (B.STAT_MAX, B.STAT_TWO_NORM):
        H.assert_parity(H.run_parity(w, statistic=statistic, options={B.OPT_STREAM_THREADS: 128}))
    a, b = H.DeviceState(w, guarded=False), H.DeviceState(w, guarded=False)
    oa = H.make_optimizer(w, {B.OPT_STATISTIC: B.STAT_MIN})
    ob = H.make_optimizer(w, {B.OPT_STATISTIC: B.STAT_MIN})
    for t in (1, 2):
        a.draw_grads(t)
        for x, y in zip(a.g, b.g):
            y.copy_(x * 0.25)
        oa.step_ex(a.p, a.g, a.m, a.v, t, grad_scale=0.25)
        ob.step(b.p, b.g, b.m, b.v, t)
    oa.sync_status(); ob.sync_status()
    assert _same(a, b)
    oa.close(); ob.close()
