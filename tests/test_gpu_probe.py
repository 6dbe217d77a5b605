"""The copy through the streaming kernel's ring (adammini_probe_ring_copy), the
measurement aid behind the benchmark's read/write-mix ceiling: it must move exactly
the bytes it claims to, or the bandwidth computed from it means nothing."""
import pytest
import torch

import harness as H
from paper_2406_16793_b200 import binding as B, workloads as W

pytestmark = pytest.mark.gpu


def _optimizer():
    return H.make_optimizer(W.tiny_gpt2())


class GuardedBytes:
    """A byte buffer with 256 sentinel bytes either side (16-byte aligned view)."""

    def __init__(self, n: int):
        self.raw = torch.full((n + 512 + (-n) % 16,), 0xA5, dtype=torch.uint8, device="cuda")
        self.view = self.raw[256:256 + n]
        self.n = n

    def intact(self) -> bool:
        return bool((self.raw[:256] == 0xA5).all() and (self.raw[256 + self.n:] == 0xA5).all())


@pytest.mark.parametrize("load_bytes,store_bytes", [(40960, 32768), (40960, 40960), (40960, 27296), (4096, 16), (16, 16)])
def test_ring_copy_moves_every_item(load_bytes, store_bytes):
    n_items = 2011                                              # several per CTA, and a ragged last round
    opt = _optimizer()
    gen = torch.Generator(device="cuda").manual_seed(7)
    src = torch.randint(0, 256, (n_items * load_bytes,), dtype=torch.uint8, device="cuda", generator=gen)
    dst = GuardedBytes(n_items * store_bytes)
    dst.view.fill_(0)
    opt.probe_ring_copy(src, dst.view, n_items, load_bytes, store_bytes)
    opt.sync_status()
    want = src.view(n_items, load_bytes)[:, :store_bytes].reshape(-1)
    assert torch.equal(dst.view, want)
    assert dst.intact()
    opt.close()


def test_ring_copy_read_only_and_write_only():
    """Loads without stores leave dst alone; stores without loads need no src."""
    opt = _optimizer()
    src = torch.ones(64 * 40960, dtype=torch.uint8, device="cuda")
    dst = GuardedBytes(64 * 40960)
    dst.view.fill_(7)
    opt.probe_ring_copy(src, None, 64, 40960, 0)
    opt.sync_status()
    assert bool((dst.view == 7).all())
    opt.probe_ring_copy(None, dst.view, 64, 0, 40960)           # writes whatever the stages hold
    opt.sync_status()
    assert dst.intact()
    opt.close()


def test_ring_copy_rejects_bad_arguments():
    opt = _optimizer()
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    for load_bytes, store_bytes in ((0, 0), (40976, 16), (100, 16), (4096, 8192), (-16, 16), (4096, 24)):
        with pytest.raises(B.AdamMiniError) as e:
            opt.probe_ring_copy(buf, buf, 4, load_bytes, store_bytes)
        assert e.value.status == -1, (load_bytes, store_bytes)
    with pytest.raises(B.AdamMiniError) as e:
        opt.probe_ring_copy(buf[8:], buf, 4, 4096, 4096)        # 8 bytes off the 16-byte grid
    assert e.value.status == -3
    with pytest.raises(B.AdamMiniError) as e:
        opt.probe_ring_copy(None, buf, 4, 4096, 4096)
    assert e.value.status == -1
    opt.probe_ring_copy(buf, buf, 0, 4096, 4096)                # nothing to do
    opt.sync_status()
    opt.close()
