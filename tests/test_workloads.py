"""Layouts of the five benchmark configurations and the seeded gradient generators."""
import numpy as np
import pytest
import torch

from paper_1905_10936_b200 import workloads as wl


def test_layout_sizes():
    c1, c2, c3, c4, c5 = (wl.make_workload(c) for c in range(1, 6))
    assert (c1.d, c1.B, c1.M) == (1 << 20, 16, 2)
    assert (c2.d, c2.B, c2.M, c2.num_words) == (269_722, 59, 8, 8437)
    assert (c3.d, c3.B, c3.M) == (25_557_032, 161, 7)       # ResNet-50's parameter count
    assert (c4.d, c4.B, c4.M, c4.steps) == (1 << 28, 256, 7, 20)
    assert (c5.d, c5.B, c5.M) == (354_821_120, 290, 4)
    assert max(c5.sizes) == 50257 * 1024
    for c in (c1, c2, c3, c4, c5):
        assert c.offsets[0] == 0 and np.all(np.diff(c.offsets) > 0)
        assert np.all(c.offsets[:-1] % 4 == 0)               # every block starts 16-byte aligned
    assert min(c2.sizes) == 10 and 1000 in c3.sizes


@pytest.mark.parametrize("cid", [1, 2])
def test_gradients_are_seeded_and_scaled(cid):
    w = wl.make_workload(cid)
    g0 = w.draw_grad(0, 0, "cpu")
    g0b = w.draw_grad(0, 0, "cpu")
    g1 = w.draw_grad(0, 1, "cpu")
    assert g0.dtype == torch.float32 and g0.shape == (w.d,)
    assert torch.equal(g0, g0b) and not torch.equal(g0, g1)
    sb = w.block_scales()
    if w.scale_range is not None:
        lo, hi = w.scale_range
        assert sb.min() >= lo and sb.max() <= hi
    b = int(np.argmax(w.sizes))
    blk = g0[w.offsets[b]:w.offsets[b + 1]].double()
    assert abs(blk.std().item() / sb[b] - 1) < 0.05


def test_laplace_generator_is_finite_and_scaled():
    w = wl.custom_workload("lap", [1 << 16], M=1, law="laplace", scale_range=(0.01, 0.010001))
    g = w.draw_grad(3, 0, "cpu").double()
    assert torch.isfinite(g).all()
    assert abs(g.abs().mean().item() / 0.01 - 1) < 0.03      # E|Laplace(b)| = b
    assert abs((g < 0).double().mean().item() - 0.5) < 0.02


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_shard_blocks_tiles_the_layout(world):
    for cid in (2, 3, 5):
        w = wl.make_workload(cid)
        cuts = [wl.shard_blocks(w.sizes, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == w.B
        for a, b in zip(cuts, cuts[1:]):
            assert a[1] == b[0]
        assert all(lo <= hi for lo, hi in cuts)
