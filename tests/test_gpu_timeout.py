"""The error path of the bounded device-side waits, taken for real.

Every wait inside the kernels (for a staged copy, for a consumer group's
barrier, for a cluster's exchange) polls for a limited time and then gives up:
the kernel ends through its normal exit and the handle reports AM_ERR_TIMEOUT.
Here the limit is set to a few milliseconds and the thread that stages data is
told to withhold its stages (a test option of the library), so the consumers'
waits run out.  Nothing faults, no wait is without a limit, and the same handle
then steps normally again.
"""
import time

import pytest

import harness as H
import paper_2406_16793_b200 as am
from paper_2406_16793_b200 import binding as B, workloads as W

pytestmark = pytest.mark.gpu

T = W.TensorSpec
BF = dict(grad_dtype=W.BF16)


def rows_workload():
    """Single-CTA streaming kernel: packed rows and long rows re-read from L2, aligned and
    not (the latter in a launch of their own)."""
    return W.Workload("stall-rows", 71, [T("rows", 600, 4096, W.ROWS, **BF), T("short", 3000, 768, W.ROWS, **BF),
                                         T("long", 300, 11008, W.ROWS, **BF), T("longodd", 150, 10007, W.ROWS, **BF), T("held", 300, 4099, W.ROWS, **BF)], W.GradRecipe(-4.0, -1.0), steps=2)


def heads_workload():
    """Cluster kernel: heads of 524288 elements split over the CTAs of a cluster."""
    return W.Workload("stall-heads", 72, [T("q", 1024, 4096, W.HEADS, n_heads=8, **BF),
                                          T("k", 512, 4096, W.HEADS, n_heads=4, grad_dtype=W.F32)],
                      W.GradRecipe(-4.0, -1.0), steps=2)


def tiles_workload():
    """Tile kernel: short blocks and unaligned longer ones (two launches)."""
    return W.Workload("stall-tiles", 73, [T("l24", 5000, 24, W.ROWS, **BF), T("l1001", 700, 1001, W.ROWS, **BF),
                                          T("l3", 9000, 3, W.ROWS, grad_dtype=W.F32)], W.GradRecipe(-4.0, -1.0), steps=2)


def everything():
    from test_gpu_extras import mixed_workload
    return mixed_workload()


@pytest.mark.parametrize("make,stall", [(rows_workload, 1), (rows_workload, 4), (heads_workload, 1), (heads_workload, 3),
                                        (tiles_workload, 1), (everything, 2)],
                         ids=["rows-nothing-staged", "rows-three-stages", "heads-nothing-staged", "heads-two-stages",
                              "tiles", "every-family"])
def test_a_wait_that_runs_out_is_reported_and_the_handle_recovers(make, stall):
    w = make()
    dev = H.DeviceState(w, guarded=True)
    opt = H.make_optimizer(w, {B.OPT_WAIT_LIMIT_US: 5000, B.OPT_TEST_STALL: stall})
    dev.draw_grads(1)
    t0 = time.perf_counter()
    opt.step(dev.p, dev.g, dev.m, dev.v, 1)
    with pytest.raises(am.AdamMiniError) as e:
        opt.sync_status()
    assert e.value.status == -5                                   # AM_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 20.0                        # the waits really are bounded
    assert dev.guards_intact()                                    # a partly updated step stays inside its buffers
    opt.sync_status()                                             # reading the status cleared it
    # the same handle, hook off and default limit back: an ordinary run against the oracle
    opt.set_option(B.OPT_TEST_STALL, 0)
    opt.set_option(B.OPT_WAIT_LIMIT_US, 0)
    H.assert_parity(H.run_parity(w, optimizer=opt))
    opt.close()


def test_wait_limit_is_validated():
    w = rows_workload()
    opt = H.make_optimizer(w)
    for bad in (1, 99, 60_000_001):
        with pytest.raises(am.AdamMiniError) as e:
            opt.set_option(B.OPT_WAIT_LIMIT_US, bad)
        assert e.value.status == -1
    opt.set_option(B.OPT_WAIT_LIMIT_US, 100)
    opt.set_option(B.OPT_WAIT_LIMIT_US, 0)
    opt.close()


def test_a_short_limit_alone_changes_nothing():
    """With data flowing, waits last microseconds: a 20 ms limit never fires."""
    w = rows_workload()
    H.assert_parity(H.run_parity(w, options={B.OPT_WAIT_LIMIT_US: 20000}))
