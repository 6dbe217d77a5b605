"""The allocation-free entry point against the handle-based one.

adammini_step_tensor_noalloc serves callers that cannot allocate device memory
(allocator callbacks, loops whose pool owns the whole device, sections that
cannot afford an allocation's synchronisation): its scratch is a fixed array
inside the library.  Here it runs two steps in a row on several shapes and must
agree with adammini_step, whose scratch comes from cudaMalloc, within the
tolerance the parity tests use.  The file sorts last on purpose, so that a run
that stops at the first failure has already covered everything else.
"""
import pytest
import torch

import harness as H
import paper_2406_16793_b200 as am
from paper_2406_16793_b200 import binding as B, workloads as W

pytestmark = pytest.mark.gpu

CASES = [
    # rows, cols, kind, n_heads, fixed block length, gradient dtype
    (1, 1 << 20, W.WHOLE, 0, 0, W.F32),        # one block, 32 partial sums
    (256, 4096, W.ROWS, 0, 0, W.BF16),         # 256 row blocks
    (512, 1024, W.HEADS, 4, 0, W.BF16),        # 4 head blocks of 131072 elements
    (1, 70001, W.FIXED, 0, 70001, W.F32),      # odd length: single elements after the last group of four
    (9, 10007, W.ROWS, 0, 0, W.BF16),          # odd rows: blocks start off the 16-byte grid
    (1, 32768, W.FIXED, 0, 1, W.F32),          # block length 1 at the block limit
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"{c[0]}x{c[1]}-k{c[2]}-d{c[5]}")
def test_noalloc_matches_handle_based_step_two_calls_in_a_row(case):
    rows, cols, kind, n_heads, fixed, gd = case
    spec = W.TensorSpec("t", rows, cols, kind, n_heads=n_heads, fixed_block_len=fixed, grad_dtype=gd)
    w = W.Workload("noalloc", 55, [spec], W.GradRecipe(-4.0, -1.0), steps=2)
    ref = H.DeviceState(w, guarded=True)
    new = H.DeviceState(w, guarded=True)
    opt = H.make_optimizer(w, {B.OPT_PATH: 1})
    for step in (1, 2):
        ref.draw_grads(step)
        new.g[0].copy_(ref.g[0])
        opt.step(ref.p, ref.g, ref.m, ref.v, step)
        B.step_tensor_noalloc(new.p[0], new.g[0], new.m[0], new.v, spec.block_len, step, **w.hparams)
        torch.cuda.synchronize()
        L = spec.block_len
        assert H.block_relative_error(new.p[0].cpu().numpy(), ref.p[0].cpu().numpy(), L) <= H.TOL
        assert H.block_relative_error(new.m[0].cpu().numpy(), ref.m[0].cpu().numpy(), L) <= H.TOL
        assert H.v_relative_error(new.v.cpu().numpy(), ref.v.cpu().numpy()) <= H.TOL
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
