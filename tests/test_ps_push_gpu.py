"""The push variant of the parameter-server protocol on one GPU: the worker kernel stores block
b's fused message directly into the receive buffer of the rank that serves b, and every server
stores its update slice into every rank's update buffer (no pack kernel on the worker side, no
collective).  With all ranks emulated on one device the "peer" buffers are local tensors; the
kernels and the address tables are exactly those a multi-device run uses.  Everything must equal
the plain engine bit for bit, and the receive buffers must equal what the collective variant
delivers."""
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


def _wl(sizes, M, steps=4, cid=410):
    return wl.custom_workload("ps-push", sizes, M, 0.9, 0.1, steps, "normal", (1e-3, 1.0), config_id=cid)


def _ranks(w, G, **kw):
    ranks = [ps.Rank(EFEngine(w.offsets, G, w.mu, w.eta, one_local_worker=True, **kw), w.sizes, r, G)
             for r in range(G)]
    ps.connect_emulated(ranks)
    return ranks


@pytest.mark.parametrize("sizes,G", [
    ([64, 64], 2), ([700, 33, 4096, 10, 2500, 64, 1200], 3), ([5, 3, 31, 33, 63, 65, 127, 129], 2),
    ([2 * TILE, TILE // 2, 3 * TILE + 36, 100, BIG + 8, 777], 4),
    ([BIG - 4, 3 * BIG + TILE + 4, 2 * BIG + 2 * TILE, 40], 7), ([1000] * 40, 8), ([12345, 54321, 99999], 15),
    ([100, 200], 3),                                         # more ranks than blocks: one serves nothing
    ([300 * TILE + 17, 5], 2),                               # > 1024 chunks: scales by the follow-up kernel
])
@pytest.mark.parametrize("scale_mode", ["fused", "split"])
def test_pushed_messages_equal_the_collective_variant_and_the_plain_engine(sizes, G, scale_mode):
    w = _wl(sizes, G)
    ref = EFEngine(w.offsets, G, w.mu, w.eta, scale_mode=scale_mode)
    ranks = _ranks(w, G, scale_mode=scale_mode)
    coll = [ps.Rank(EFEngine(w.offsets, G, w.mu, w.eta, scale_mode=scale_mode, one_local_worker=True),
                    w.sizes, r, G) for r in range(G)]
    es = w.element_scales("cuda")
    etas = [0.1, 0.1, 0.05, 0.2]
    for t in range(w.steps):
        if t > 0:
            ref.set_eta(etas[t])
            for rk in ranks + coll:
                rk.engine.set_eta(etas[t])
        grads = [w.draw_grad(t, i, "cuda", es) for i in range(G)]
        for i in range(G):
            ref.worker_step(i, grads[i])
        ref.server_step()
        ps.step_emulated(coll, grads)
        ps.step_emulated_push(ranks, grads)
        for r, rk in enumerate(ranks):
            m = rk.mine
            if m.units:
                assert torch.equal(rk.recv[:, :m.units], coll[r].recv[:, :m.units]), f"recv of rank {r}, step {t}"
            assert torch.equal(rk.update, coll[r].update)
            assert torch.equal(rk.engine.worker_scales(0), ref.worker_scales(r))
            assert torch.equal(rk.engine.params(), ref.params()), f"x on rank {r} after step {t}"
            assert rk.engine.step_count == t + 1
            if m.b1 > m.b0:
                lo, hi = int(w.offsets[m.b0]), int(w.offsets[m.b1])
                assert torch.equal(rk.engine.residual(-1)[lo:hi], ref.residual(-1)[lo:hi])
            sc, wd = ps.unpack_message(rk.update.cpu().numpy(), w.sizes, 0, w.B)
            assert np.array_equal(sc, ref.server_scales().cpu().numpy())
            assert np.array_equal(wd, ref.server_words().cpu().numpy().view(np.uint32))
    for r, rk in enumerate(ranks):
        assert torch.equal(rk.engine.momentum(0), ref.momentum(r))
        assert torch.equal(rk.engine.residual(0), ref.residual(r))


def test_push_stores_nothing_outside_the_messages():
    """Guard units around every destination stay untouched, and a block's message is exactly
    1 + ceil(d_b/32) units."""
    sizes = [TILE + 37, 31, 2 * BIG + 5, 64]
    w = _wl(sizes, 1, steps=2, cid=411)
    e = EFEngine(w.offsets, 1, w.mu, w.eta)
    ref = EFEngine(w.offsets, 1, w.mu, w.eta)
    units = [1 + (n + 31) // 32 for n in sizes]
    GUARD = 8
    SENT = 0x5A5A5A5A
    bufs = [torch.full((u + 2 * GUARD,), SENT, dtype=torch.int32, device="cuda") for u in units]
    table = torch.tensor([b.data_ptr() + 4 * GUARD for b in bufs], dtype=torch.int64, device="cuda")
    es = w.element_scales("cuda")
    for t in range(w.steps):
        g = w.draw_grad(t, 0, "cuda", es)
        e.worker_step_push(0, g, table)
        ref.worker_step(0, g)
        torch.cuda.synchronize()
        rw = ref.worker_words(0).cpu().numpy().view(np.uint32)
        rs = ref.worker_scales(0).cpu().numpy()
        wo = 0
        for b, u in enumerate(units):
            got = bufs[b].cpu().numpy().view(np.uint32)
            assert np.all(got[:GUARD] == SENT) and np.all(got[GUARD + u:] == SENT), f"block {b}"
            assert got[GUARD:GUARD + 1].view(np.float32)[0] == rs[b]
            assert np.array_equal(got[GUARD + 1:GUARD + u], rw[wo:wo + u - 1])
            wo += u - 1
        # the rest of the iteration needs the words in the context: refused after a push
        with pytest.raises(ef.EFError):
            e.pack_message(0, 0, len(sizes), torch.zeros(sum(units), dtype=torch.int32, device="cuda"))
        with pytest.raises(ef.EFError):
            e.server_step()
        # ... served from the pushed messages instead (M = 1: one row)
        msg = torch.cat([bufs[b][GUARD:GUARD + u] for b, u in enumerate(units)]).view(1, -1).contiguous()
        e.server_step_range(0, len(sizes), msg)
        e.apply_update(0, len(sizes))
        ref.server_step()
        assert torch.equal(e.params(), ref.params())


def test_push_with_diagnostics_and_argument_checks():
    sizes = [3 * TILE + 5, 640, 10]
    w = _wl(sizes, 1, steps=2, cid=412)
    e = EFEngine(w.offsets, 1, w.mu, w.eta, diagnostics=True)
    ref = EFEngine(w.offsets, 1, w.mu, w.eta, diagnostics=True)
    units = [1 + (n + 31) // 32 for n in sizes]
    buf = torch.zeros(sum(units), dtype=torch.int32, device="cuda")
    starts = np.concatenate([[0], np.cumsum(units)[:-1]])
    table = torch.tensor([buf.data_ptr() + 4 * int(s) for s in starts], dtype=torch.int64, device="cuda")
    es = w.element_scales("cuda")
    g = w.draw_grad(0, 0, "cuda", es)
    e.worker_step_push(0, g, table)
    ref.worker_step(0, g)
    packed = torch.zeros_like(buf)
    ref.pack_message(0, 0, len(sizes), packed)
    assert torch.equal(buf, packed)
    assert torch.equal(e.worker_diagnostics(0), ref.worker_diagnostics(0))
    # argument checks: null table, worker stepped twice
    with pytest.raises(ef.EFError):
        ef.ef_worker_step_push(e.ctx, 0, g.data_ptr(), None)
    with pytest.raises(ef.EFError):
        e.worker_step_push(0, g, table)
    with pytest.raises(ef.EFError):
        ef.ef_push_message(ref.ctx, 0, 0, 1, [])
    with pytest.raises(ef.EFError):
        ef.ef_push_message(ref.ctx, 0, 0, 1, [buf.data_ptr()] * 65)


def test_pushed_protocol_against_the_oracle():
    sizes, G = [3 * TILE + 5, 640, 10, BIG + 64, 333], 3
    w = _wl(sizes, G, steps=4, cid=413)
    ranks = _ranks(w, G)
    orc = Oracle(w.offsets, G, w.mu, w.eta)
    es = w.element_scales("cuda")
    unit = ps.message_unit_offsets(w.sizes)
    for t in range(w.steps):
        grads = [w.draw_grad(t, i, "cuda", es) for i in range(G)]
        ps.step_emulated_push(ranks, grads)
        for i in range(G):
            # worker i's words as the servers received them (row i of every rank's receive buffer)
            parts = [ps.unpack_message(rk.recv[i, :rk.mine.units].cpu().numpy(), w.sizes, rk.mine.b0, rk.mine.b1)
                     for rk in ranks if rk.mine.units]
            gw = np.concatenate([p[1] for p in parts])
            orc.worker_step(i, grads[i].cpu().numpy(), hint=gw)
            assert np.array_equal(orc.words(i), gw)
            gs = np.concatenate([p[0] for p in parts])
            assert np.all(np.abs(gs - orc.scales(i)) <= 1e-5 * np.abs(orc.scales(i)))
        sc, wd = ps.unpack_message(ranks[0].update.cpu().numpy(), w.sizes, 0, w.B)
        orc.server_step(hint=wd)
        assert np.array_equal(orc.words(-1), wd)
        for rk in ranks:
            got = rk.engine.params().cpu().numpy()
            assert np.abs(got - orc.x).max() <= 1e-5 * np.abs(orc.x).max()
