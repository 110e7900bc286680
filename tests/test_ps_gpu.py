"""The parameter-server protocol in pieces (block-range server, fused messages) on one GPU.

G ranks are emulated one after the other on the same device: each rank is a context with ONE
local worker (EF_FLAG_ONE_LOCAL_WORKER, M = G) that serves one block range; the exchange is the
slice copies of ps.step_emulated.  Everything must equal, bit for bit, the plain engine that
holds all M workers and runs ef_server_step -- and through it the oracle (the plain engine is
what the parity tests lock to the oracle)."""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import ps
from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.engine import EFEngine

pytestmark = pytest.mark.gpu

TILE = 4096
BIG = 4 * TILE


def _wl(sizes, M, steps=4, cid=400):
    return wl.custom_workload("ps", sizes, M, 0.9, 0.1, steps, "normal", (1e-3, 1.0), config_id=cid)


@pytest.mark.parametrize("sizes,G", [
    ([64, 64], 2), ([700, 33, 4096, 10, 2500, 64, 1200], 3), ([5, 3, 31, 33, 63, 65, 127, 129], 2),
    ([2 * TILE, TILE // 2, 3 * TILE + 36, 100, BIG + 8, 777], 4),
    ([BIG - 4, 3 * BIG + TILE + 4, 2 * BIG + 2 * TILE, 40], 7), ([1000] * 40, 8), ([12345, 54321, 99999], 15),
    ([100, 200], 3),                                         # more ranks than blocks: one serves nothing
])
@pytest.mark.parametrize("scale_mode", ["fused", "split"])
def test_emulated_ranks_equal_the_plain_engine(sizes, G, scale_mode):
    w = _wl(sizes, G)
    ref = EFEngine(w.offsets, G, w.mu, w.eta, scale_mode=scale_mode)
    ranks = [ps.Rank(EFEngine(w.offsets, G, w.mu, w.eta, scale_mode=scale_mode, one_local_worker=True),
                     w.sizes, r, G) for r in range(G)]
    es = w.element_scales("cuda")
    etas = [0.1, 0.1, 0.05, 0.2]
    for t in range(w.steps):
        if t > 0:
            ref.set_eta(etas[t])
            for rk in ranks:
                rk.engine.set_eta(etas[t])
        grads = [w.draw_grad(t, i, "cuda", es) for i in range(G)]
        for i in range(G):
            ref.worker_step(i, grads[i])
        ref.server_step()
        ps.step_emulated(ranks, grads)
        for r, rk in enumerate(ranks):
            assert torch.equal(rk.engine.worker_words(0), ref.worker_words(r))
            assert torch.equal(rk.engine.worker_scales(0), ref.worker_scales(r))
            assert torch.equal(rk.engine.params(), ref.params()), f"x on rank {r} after step {t}"
            assert rk.engine.step_count == t + 1
            m = rk.mine
            if m.b1 > m.b0:
                lo, hi = int(w.offsets[m.b0]), int(w.offsets[m.b1])
                assert torch.equal(rk.engine.residual(-1)[lo:hi], ref.residual(-1)[lo:hi])
                assert torch.equal(rk.engine.server_scales()[m.b0:m.b1], ref.server_scales()[m.b0:m.b1])
            # the gathered update decodes to the plain engine's server message
            sc, wd = ps.unpack_message(rk.update.cpu().numpy(), w.sizes, 0, w.B)
            assert np.array_equal(sc, ref.server_scales().cpu().numpy())
            assert np.array_equal(wd, ref.server_words().cpu().numpy().view(np.uint32))
    for r, rk in enumerate(ranks):
        assert torch.equal(rk.engine.momentum(0), ref.momentum(r))
        assert torch.equal(rk.engine.residual(0), ref.residual(r))


def test_ranges_on_a_plain_context_equal_one_server_step():
    """All workers local: covering [0, B) with range calls in any order equals ef_server_step."""
    w = _wl([TILE + 100, 777, 2 * BIG + 36, 3, 64, 5 * TILE], 3)
    a = EFEngine(w.offsets, w.M, w.mu, w.eta)
    b = EFEngine(w.offsets, w.M, w.mu, w.eta)
    es = w.element_scales("cuda")
    for t in range(3):
        for i in range(w.M):
            g = w.draw_grad(t, i, "cuda", es)
            a.worker_step(i, g); b.worker_step(i, g)
        a.server_step()
        for b0, b1 in [(4, 6), (0, 1), (1, 4)]:
            b.server_step_range(b0, b1)
        assert b.step_count == t                     # not complete before the update is applied
        for b0, b1 in [(0, 3), (3, 6)]:
            b.apply_update(b0, b1)
        assert b.step_count == t + 1
        assert torch.equal(a.params(), b.params())
        assert torch.equal(a.server_words(), b.server_words())
        assert torch.equal(a.server_scales(), b.server_scales())
        assert torch.equal(a.residual(-1), b.residual(-1))


def test_sharded_server_against_the_oracle_with_weight_decay():
    """The emulated protocol checked directly against the oracle (words after hint adoption,
    state within 1e-5), with the weight-decay side path in the update."""
    sizes, G = [3 * TILE + 5, 640, 10, BIG + 64, 333], 3
    w = _wl(sizes, G, steps=4, cid=401)
    ranks = [ps.Rank(EFEngine(w.offsets, G, w.mu, w.eta, weight_decay=True, one_local_worker=True),
                     w.sizes, r, G) for r in range(G)]
    orc = Oracle(w.offsets, G, w.mu, w.eta)
    orc.set_weight_decay(0.01)
    x0 = torch.randn(w.d, generator=torch.Generator().manual_seed(1))
    orc.x[:] = x0.numpy()
    for rk in ranks:
        rk.engine.set_weight_decay(0.01)
        rk.engine.params().copy_(x0.cuda())
    es = w.element_scales("cuda")
    for t in range(w.steps):
        grads = [w.draw_grad(t, i, "cuda", es) for i in range(G)]
        ps.step_emulated(ranks, grads)
        for i in range(G):
            gw = ranks[i].engine.worker_words(0).cpu().numpy().view(np.uint32)
            orc.worker_step(i, grads[i].cpu().numpy(), hint=gw)
            assert np.array_equal(orc.words(i), gw)
        sc, wd = ps.unpack_message(ranks[0].update.cpu().numpy(), w.sizes, 0, w.B)
        orc.server_step(hint=wd)
        assert np.array_equal(orc.words(-1), wd)
        assert np.all(np.abs(sc - orc.scales(-1)) <= 1e-5 * np.abs(orc.scales(-1)))
        for rk in ranks:
            got = rk.engine.params().cpu().numpy()
            assert np.abs(got - orc.x).max() <= 1e-5 * np.abs(orc.x).max()


def test_call_order_of_the_range_calls():
    w = _wl([64, 64, 64], 2)
    e = EFEngine(w.offsets, w.M, w.mu, w.eta)
    g = torch.zeros(w.d, device="cuda")
    with pytest.raises(ef.EFError) as ei:
        e.server_step_range(0, 1)
    assert ei.value.status == ef.EF_ERR_BAD_STATE            # workers not stepped
    e.worker_step(0, g); e.worker_step(1, g)
    for bad in ((-1, 1), (1, 1), (2, 4)):
        with pytest.raises(ef.EFError) as ei:
            e.server_step_range(*bad)
        assert ei.value.status == ef.EF_ERR_INVALID_ARG
    e.server_step_range(0, 2)
    with pytest.raises(ef.EFError) as ei:
        e.server_step_range(1, 3)                            # block 1 served twice
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    with pytest.raises(ef.EFError) as ei:
        e.apply_update(0, 3)                                 # block 2 not served here, no message given
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    with pytest.raises(ef.EFError) as ei:
        e.server_step()                                      # range calls under way
    assert ei.value.status == ef.EF_ERR_BAD_STATE
    e.server_step_range(2, 3)
    e.apply_update(0, 3)
    assert e.step_count == 1
    one = EFEngine(w.offsets, w.M, w.mu, w.eta, one_local_worker=True)
    one.worker_step(0, g)
    with pytest.raises(ef.EFError) as ei:
        one.worker_step(1, g)                                # only one worker lives here
    assert ei.value.status == ef.EF_ERR_INVALID_ARG
    for call in (one.server_step, lambda: one.server_step_range(0, 3)):
        with pytest.raises(ef.EFError) as ei:
            call()                                           # the other worker's message is needed
        assert ei.value.status == ef.EF_ERR_BAD_STATE
    assert ef.ef_message_units(one.ctx, 0, 3) == 3 * (1 + 2) and ef.ef_message_units(one.ctx, 2, 2) == -1
    torch.cuda.synchronize()
