"""The allocation-free entry point against the handle-based one and the oracle.

adammini_step_tensor_noalloc serves callers that cannot allocate device memory
(allocator callbacks, loops whose pool owns the whole device, sections that
cannot afford an allocation's synchronisation): its scratch is a fixed array
inside the library.  Here it runs two steps in a row on several shapes and must
agree, within the tolerance the parity tests use, with adammini_step (whose
scratch comes from cudaMalloc) and with the float64 oracle.  The file sorts last
on purpose, so that a run that stops at the first failure has already covered
everything else.
"""
import pytest
import torch

import harness as H
import paper_2406_16793_b200 as am
from oracle import step as ostep
from paper_2406_16793_b200 import binding as B, workloads as W

pytestmark = pytest.mark.gpu

CASES = [
    # rows, cols, kind, n_heads, fixed block length, gradient dtype
    (1, 1 << 20, W.WHOLE, 0, 0, W.F32),        # one block, 32 partial sums
    (256, 4096, W.ROWS, 0, 0, W.BF16),         # 256 row blocks
    (512, 1024, W.HEADS, 4, 0, W.BF16),        # 4 head blocks of 131072 elements: 4 partial sums each
    (1, 70001, W.FIXED, 0, 70001, W.F32),      # odd length: single elements after the last group of four
    (9, 10007, W.ROWS, 0, 0, W.BF16),          # odd rows: blocks start off the 16-byte grid
    (3, 100003, W.ROWS, 0, 0, W.BF16),         # odd bf16 rows of several pieces each
    (1, 32768, W.FIXED, 0, 1, W.F32),          # block length 1 at the block limit
    (1, 9 << 20, W.WHOLE, 0, 0, W.BF16),       # 288 partial sums in one block (the other path adds them in another order)
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"{c[0]}x{c[1]}-k{c[2]}-d{c[5]}")
def test_noalloc_matches_handle_based_step_two_calls_in_a_row(case):
    rows, cols, kind, n_heads, fixed, gd = case
    spec = W.TensorSpec("t", rows, cols, kind, n_heads=n_heads, fixed_block_len=fixed, grad_dtype=gd)
    w = W.Workload("noalloc", 55, [spec], W.GradRecipe(-4.0, -1.0), steps=2)
    L = spec.block_len
    ref = H.DeviceState(w, guarded=True)
    new = H.DeviceState(w, guarded=True)
    ora = ostep.OracleState([new.p[0].cpu()], [L], [True])
    unit = H.ShortBlockScale(ora.p[0]) if L < H.OWN_SCALE_MIN_L else None
    opt = H.make_optimizer(w, {B.OPT_PATH: 1})
    for step in (1, 2):
        ref.draw_grads(step)
        new.g[0].copy_(ref.g[0])
        opt.step(ref.p, ref.g, ref.m, ref.v, step)
        B.step_tensor_noalloc(new.p[0], new.g[0], new.m[0], new.v, L, step, **w.hparams)
        g_cpu = new.g[0].cpu()
        ora.step([g_cpu], step, **w.hparams)
        if unit is not None:
            unit.update(ostep.widen(g_cpu), ora.p[0], ora.m[0], w.hparams["beta1"])
        torch.cuda.synchronize()
        fp, fm = (unit.p, unit.m) if unit is not None else (None, None)
        for want_p, want_m, want_v in ((ora.p[0], ora.m[0], ora.v[0]),
                                       (ref.p[0].cpu().numpy(), ref.m[0].cpu().numpy(), ref.v.cpu().numpy())):
            assert H.block_relative_error(new.p[0].cpu().numpy(), want_p, L, fp) <= H.TOL
            assert H.block_relative_error(new.m[0].cpu().numpy(), want_m, L, fm) <= H.TOL
            assert H.v_relative_error(new.v.cpu().numpy(), want_v) <= H.TOL
    assert new.guards_intact() and ref.guards_intact()
    opt.close()


def test_noalloc_rejects_sizes_beyond_its_scratch():
    n = (B.NOALLOC_MAX_BLOCKS + 1) * 4
    p = torch.zeros(n, device="cuda"); g = torch.zeros(n, device="cuda"); m = torch.zeros(n, device="cuda")
    v = torch.zeros(B.NOALLOC_MAX_BLOCKS + 1, device="cuda")
    with pytest.raises(am.AdamMiniError) as e:
        B.step_tensor_noalloc(p, g, m, v, 4, 1)
    assert e.value.status == -7
    with pytest.raises(am.AdamMiniError) as e:
        B.step_tensor_noalloc(p, g, m, v, 7, 1)          # 7 does not divide numel
    assert e.value.status == -2
    assert not p.any() and not m.any() and not v.any()   # a rejected call does nothing


def test_noalloc_rejects_too_many_partial_sums():
    """Fewer blocks than the limit, but two partial sums per block put the count of
    partial sums over it: refused, and nothing is written."""
    L, nb = 32768 + 8, B.NOALLOC_MAX_PIECES // 2 + 1
    assert nb <= B.NOALLOC_MAX_BLOCKS and 2 * nb > B.NOALLOC_MAX_PIECES
    free, _ = torch.cuda.mem_get_info()
    if free < 8 * (1 << 30):
        pytest.skip("needs about 6 GB of free device memory")
    p = torch.zeros(nb * L, device="cuda"); m = torch.zeros(nb * L, device="cuda")
    g = torch.ones(nb * L, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros(nb, device="cuda")
    with pytest.raises(am.AdamMiniError) as e:
        B.step_tensor_noalloc(p, g, m, v, L, 1)
    assert e.value.status == -7
    torch.cuda.synchronize()
    assert not p.any() and not m.any() and not v.any()
