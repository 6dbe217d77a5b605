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


def mixed_workload():
    """Every kernel family at once: tiny blocks, packed rows, long rows, a clustered head, a two-pass block."""
    T = W.TensorSpec
    bf = dict(grad_dtype=W.BF16)
    tensors = [
        T("tiny", 1, 4096, W.FIXED, fixed_block_len=1, **bf),
        T("rows", 96, 4096, W.ROWS, **bf),
        T("short", 300, 768, W.ROWS, **bf),
        T("long", 24, 11008, W.ROWS, **bf),
        T("head", 256, 4096, W.HEADS, n_heads=2, **bf),
        T("whole", 1, 3 << 20, W.WHOLE, **bf),
        T("odd", 5, 1001, W.ROWS, **bf),
        T("f32rows", 64, 512, W.ROWS, grad_dtype=W.F32),
    ]
    return W.Workload("mixed", 61, tensors, W.GradRecipe(-4.0, -1.0), steps=3)


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


@pytest.mark.parametrize("statistic", [B.STAT_MAX, B.STAT_MIN, B.STAT_ONE_NORM, B.STAT_TWO_NORM],
                         ids=["max", "min", "one-norm", "two-norm"])
@pytest.mark.parametrize("grad_dtype", [W.F32, W.BF16], ids=["f32", "bf16"])
def test_ablation_statistics(statistic, grad_dtype):
    """The block statistics of the paper's ablation (max, min, 1-norm, 2-norm of
    g*g in place of the mean) against the oracle's variant routine."""
    H.assert_parity(H.run_parity(ragged_workload(grad_dtype), steps=4, statistic=statistic))


def test_ablation_statistics_on_model_shapes():
    w = W.scaled_rows(W.llama2_7b(n_layers=1, vocab=128), 128)
    H.assert_parity(H.run_parity(w, steps=3, statistic=B.STAT_TWO_NORM))
