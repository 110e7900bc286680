"""GPU parity of signum with majority vote (ef_vote_*), through the C ABI, against its oracle.

Both sides evaluate m = fma(mu, m, g) and x -+ eta in binary32, and everything else is integer
work, so the bar is exact: packed words bit for bit after every call, momentum and parameters
equal in value after every step.
"""
import numpy as np
import pytest
import torch

from oracle import SignumOracle
from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.engine import EFEngine
from parity import BlockSample

pytestmark = pytest.mark.gpu

TILE = 4096
BIG = 4 * TILE


def run_vote_parity(w, steps, blocks=None, batched=False, grads=None, x0=None):
    eng = EFEngine(w.offsets, w.M, w.mu, w.eta)
    smp = BlockSample(w.offsets, blocks)
    orc = SignumOracle(smp.sub_offsets, w.M, w.mu, w.eta)
    if x0 is not None:
        eng.params().copy_(x0.cuda())
        orc.x[:] = smp.elems(x0.cuda())
    es = w.element_scales("cuda")
    stride = (w.d + 3) // 4 * 4
    gall = torch.zeros(w.M, stride, device="cuda") if batched else None
    gbuf = torch.empty(w.d, device="cuda")
    for t in range(steps):
        if batched:
            for i in range(w.M):
                if grads is not None:
                    gall[i, :w.d].copy_(grads[t][i])
                else:
                    w.draw_grad(t, i, "cuda", es, out=gall[i, :w.d])
            eng.vote_worker_step_all(gall)
        for i in range(w.M):
            if batched:
                g = gall[i, :w.d]
            else:
                g = grads[t][i].cuda() if grads is not None else w.draw_grad(t, i, "cuda", es, out=gbuf)
                eng.vote_worker_step(i, g)
            orc.worker_step(i, smp.elems(g))
            assert np.array_equal(smp.words(eng.worker_words(i)), orc.words(i)), f"worker {i} step {t}"
        eng.vote_server_step()
        orc.server_step()
        assert np.array_equal(smp.words(eng.server_words()), orc.words(-1)), f"vote of step {t}"
        assert np.array_equal(smp.elems(eng.params()), orc.x), f"x after step {t}"
    for i in range(w.M):
        assert np.array_equal(smp.elems(eng.momentum(i)), orc.momentum(i))
    assert eng.step_count == steps == orc.t
    return eng, orc


def _wl(sizes, M, mu=0.9, eta=0.01, cid=300):
    return wl.custom_workload("vote", sizes, M, mu, eta, 5, "normal", (1e-3, 1.0), config_id=cid)


@pytest.mark.parametrize("sizes,M", [
    ([4], 1), ([1], 2), ([64], 3), ([1] * 50, 4), ([10, 32, 458, 500], 1),
    ([3, 5, 31, 33, 63, 65, 127, 129], 3),            # unaligned block starts: scalar paths
    ([40, 64, 5, 300, 7, 1000, 13], 5),
    ([TILE], 2), ([TILE - 1], 2), ([TILE + 1], 2), ([TILE - 4, 8, TILE + 4], 7),
    ([2 * TILE, TILE // 2, 3 * TILE + 36, 100], 8),   # even M: ties are sent as +1
    ([5 * TILE + 2, 3, 2 * TILE + 1, 4 * TILE], 2),
    ([1000] * 40, 16), ([12345, 54321, 99999], 9), ([TILE + 3, BIG + 40, 777], 15),
    ([BIG + 5, 300, 2 * TILE], 17), ([640, TILE], 33), ([BIG + 36, 100], 100), ([2 * TILE + 8], 255),
])
@pytest.mark.parametrize("batched", [False, True])
def test_small_layouts(sizes, M, batched):
    run_vote_parity(_wl(sizes, M), steps=4, batched=batched, x0=torch.randn(sum(sizes)))


def test_ties_and_zero_momenta():
    """M = 4 with gradients built so that every coordinate ties 2:2 in the first step, two
    workers' momenta cancel to exactly zero in the second, and the third is a 3:1 vote that
    follows the sign of the base vector: ties vote +1, sign(+-0) = +1."""
    w = _wl([64, TILE + 32, 7], 4, mu=0.5)
    gen = torch.Generator().manual_seed(3)
    base = torch.randn(w.d, generator=gen)
    z = torch.zeros(w.d)
    grads = [[base, -base, base, -base],                 # every coordinate ties
             [-0.5 * base, 0.5 * base, z, torch.full((w.d,), -0.0)],   # workers 0, 1: m = 0 exactly
             [base, base, base, -base]]
    eng, orc = run_vote_parity(w, steps=3, grads=grads)
    negatives = int(np.unpackbits(orc.words(-1).view(np.uint8)).sum())
    assert negatives == int((base < 0).sum())            # last vote = sign(base)
    eta = np.float32(w.eta)
    x = (np.zeros(w.d, dtype=np.float32) - eta) - eta     # two all-(+1) votes, then sign(base)
    assert np.array_equal(orc.x, np.where(base.numpy() < 0, x + eta, x - eta))


def test_signsgd_is_the_mu_0_case_and_denormals_are_not_flushed():
    w = _wl([TILE + 64, 96], 3, mu=0.0)
    gen = torch.Generator().manual_seed(8)
    grads = [[torch.randn(w.d, generator=gen) * 1e-41 for _ in range(3)] for _ in range(3)]
    run_vote_parity(w, steps=3, grads=grads)


@pytest.mark.parametrize("cid", [1, 2, 3])
def test_benchmark_layouts_whole_vector(cid):
    w = wl.make_workload(cid)
    w.eta = 0.001
    run_vote_parity(w, steps=4, batched=True)


def test_flat_2_28_layout_sampled_blocks():
    """Full-size launch (d = 2^28, M = 7, batched worker call); the oracle follows 6 of the 256
    blocks (blocks are independent: the method is coordinate-wise)."""
    w = wl.make_workload(4)
    w.eta = 0.001
    run_vote_parity(w, steps=3, blocks=[0, 1, 100, 127, 128, 255], batched=True)


def test_methods_cannot_be_mixed_inside_one_iteration():
    w = _wl([64, 64], 2)
    e = EFEngine(w.offsets, w.M, w.mu, w.eta)
    g = torch.zeros(w.d, device="cuda")
    e.worker_step(0, g)
    with pytest.raises(ef.EFError) as ei:
        e.vote_worker_step(1, g)
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    e.worker_step(1, g)
    with pytest.raises(ef.EFError) as ei:
        e.vote_server_step()
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    e.server_step()
    e.vote_worker_step(0, g)
    with pytest.raises(ef.EFError) as ei:
        e.vote_worker_step(0, g)
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    with pytest.raises(ef.EFError) as ei:
        e.worker_step(1, g)
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    e.vote_worker_step(1, g)
    with pytest.raises(ef.EFError) as ei:
        e.server_step()
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    e.vote_server_step()
    assert e.step_count == 2
    torch.cuda.synchronize()


def test_host_gradients_match_device_gradients():
    """ef_vote_worker_step_host (pinned host gradients through the two staging buffers) and the
    voted signs read back with ef_read_update_host equal the device path bit for bit."""
    w = wl.custom_workload("vote-host", [TILE * 3 + 11, 100, TILE], 3, 0.9, 0.1, 4, "normal", (1e-3, 1.0),
                           config_id=330)
    a = EFEngine(w.offsets, w.M, w.mu, w.eta)
    b = EFEngine(w.offsets, w.M, w.mu, w.eta, host_staging=True)
    words = torch.empty(b.W, dtype=torch.int32).pin_memory()
    scales = torch.empty(b.B, dtype=torch.float32).pin_memory()
    for t in range(4):
        hs = [w.draw_grad(t, i, "cpu").pin_memory() for i in range(w.M)]
        for i in range(w.M):
            a.vote_worker_step(i, hs[i].cuda())
            b.vote_worker_step_host(i, hs[i])
        a.vote_server_step(); b.vote_server_step()
        b.read_update_host(words, scales)
        torch.cuda.synchronize()
        assert torch.equal(words, a.server_words().cpu())
    assert torch.equal(a.params(), b.params())
    for i in range(w.M):
        assert torch.equal(a.momentum(i), b.momentum(i))
    plain = EFEngine(w.offsets, w.M, w.mu, w.eta)
    with pytest.raises(ef.EFError) as ei:
        plain.vote_worker_step_host(0, hs[0])
    assert ei.value.status == ef.EF_ERR_BAD_STATE            # no staging buffers requested
