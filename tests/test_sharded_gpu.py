"""A layout cut by element count, INSIDE blocks, over several rank contexts on one GPU
(paper_1905_10936_b200/sharded.py): each rank holds all M workers' state for its element range;
the only exchange is one fp64 sum per cut block and call.  The sharded object runs through the
same step-locked protocol against the oracle as the plain engine (packed words bit-exact after
tie-zone adoption, scales and state to 1e-5)."""
import numpy as np
import pytest
import torch

from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.engine import EFEngine
from paper_1905_10936_b200.sharded import ShardedEngine
from parity import run_parity

pytestmark = pytest.mark.gpu

TILE = 4096
BIG = 4 * TILE


@pytest.mark.parametrize("sizes,M,ranks", [
    ([20 * TILE], 2, 2),                                   # one block cut in two
    ([20 * TILE + 100, 777, 9 * TILE], 3, 3),              # the large block spans all three ranks
    ([3 * BIG, 100, 64, 5 * BIG + 36, 2 * TILE], 7, 4),
    ([1000] * 40, 4, 3),                                   # small blocks only: no cut, no exchange
    ([33 * TILE + 5], 9, 8),                               # one block over eight ranks
])
@pytest.mark.parametrize("batched", [False, True])
def test_cut_layout_against_the_oracle(sizes, M, ranks, batched):
    w = wl.custom_workload("cut", sizes, M, steps=5, scale_range=(1e-3, 1.0), config_id=600)
    factory = lambda *a, **kw: ShardedEngine(*a, ranks=ranks, **kw)
    eng, orc, stats = run_parity(w, engine_factory=factory, batched=batched,
                                 etas=[0.1, 0.1, 0.05, 0.2, 0.2])
    assert stats["adopted"] <= 2
    if sum(1 for s in sizes if s > sum(sizes) // ranks):
        assert eng.cut


def test_gpt2_shaped_layout_cut_over_eight_ranks_sampled_steps():
    """The embedding (14.5 % of d) is larger than an eighth of the vector: it is cut, and so
    are seven weight matrices.  Scaled-down widths keep it small; structure as the real layout."""
    wd = 128
    sizes = [50257 * wd // 8, 1024 * wd // 8]
    for _ in range(6):
        sizes += [wd, wd, wd * 3 * wd, 3 * wd, wd * wd, wd, wd, wd, wd * 4 * wd, 4 * wd, 4 * wd * wd, wd]
    w = wl.custom_workload("gpt2-small", sizes, 4, steps=3, scale_range=(1e-5, 1e-2), config_id=601)
    factory = lambda *a, **kw: ShardedEngine(*a, ranks=8, **kw)
    eng, orc, stats = run_parity(w, engine_factory=factory, batched=True, check_every_step=False)
    assert eng.cut and stats["adopted"] <= 2


def test_calls_that_need_open_scales_are_refused():
    sizes = [8 * TILE]
    sh = wl.shard_elements(sizes, 2, 0)
    assert sh.local_sizes == [4 * TILE] and sh.full_sizes == [8 * TILE]
    e = EFEngine([0, 4 * TILE], 1, 0.9, 0.1)
    with pytest.raises(ef.EFError) as ei:
        e.set_block_divisors([TILE])                        # smaller than the piece
    assert ei.value.status == ef.EF_ERR_INVALID_ARG
    e.set_block_divisors([8 * TILE])
    g = torch.randn(4 * TILE, device="cuda")
    e.worker_step(0, g)
    for call in (lambda: e.server_step(), lambda: e.server_step_range(0, 1)):
        with pytest.raises(ef.EFError) as ei:
            call()
        assert ei.value.status == ef.EF_ERR_BAD_STATE       # the worker's scale is still open
    sums = torch.zeros(1, dtype=torch.float64, device="cuda")
    e.block_sums(0, sums)
    torch.cuda.synchronize()
    assert abs(sums.item() - (1.9 * g.double().abs()).sum().item()) < 1e-6 * sums.item()   # p = (1 + mu) g at t = 0
    e.complete_scales(0, sums * 2)                           # pretend the other piece had the same sum
    with pytest.raises(ef.EFError) as ei:
        e.complete_scales(0, sums)                           # nothing open any more
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    assert abs(e.worker_scales(0).item() - 2 * sums.item() / (8 * TILE)) < 1e-6
    e.server_step_range(0, 1)
    with pytest.raises(ef.EFError) as ei:
        e.apply_update(0, 1)                                 # the server's scale is open
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    e.block_sums(-1, sums)
    e.complete_scales(-1, sums * 2)
    e.apply_update(0, 1)
    assert e.step_count == 1
    torch.cuda.synchronize()
