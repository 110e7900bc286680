"""Out-of-bounds protection without a device memory checker.

(1) Guard bands: the workspace and every buffer handed to the library sit inside larger
    allocations whose margins hold a known pattern; after whole iterations of every call family
    on ragged layouts and on the ResNet-20 / ResNet-50 layouts the margins must be untouched.
(2) The checked build (libef_debug.so, -DEF_DEBUG): every kernel validates its work item against
    the problem's sizes before touching memory.  It must give the results of the regular build,
    report nothing on valid problems, and refuse (EF_ERR_BOUNDS, no trap) a tile descriptor that
    a test hook moved past the end of its arrays.  The moved descriptor still points inside the
    workspace allocation, so nothing here can fault the device.
"""
import os

import numpy as np
import pytest
import torch

from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import build as efbuild
from paper_1905_10936_b200 import ps
from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.engine import EFEngine

pytestmark = pytest.mark.gpu

TILE = 4096
BIG = 4 * TILE
MARGIN = 1 << 16           # bytes on each side
PATTERN = 0xA5


class Guarded:
    """A device buffer of `nbytes` inside a larger allocation with patterned margins."""

    def __init__(self, nbytes, dtype=torch.uint8):
        nbytes = (nbytes + 255) // 256 * 256
        self.raw = torch.full((nbytes + 2 * MARGIN,), PATTERN, dtype=torch.uint8, device="cuda")
        self.inner = self.raw[MARGIN:MARGIN + nbytes]
        self.inner.zero_()
        self.view = self.inner.view(dtype)

    def intact(self):
        return bool((self.raw[:MARGIN] == PATTERN).all()) and bool((self.raw[-MARGIN:] == PATTERN).all())


def _layouts():
    yield "ragged", [3, 5, 31, 33, 63, 65, 127, 129, TILE + 1, 2 * BIG + 36, 777], 3
    yield "tiles", [BIG - 4, 3 * BIG + TILE + 4, 2 * BIG + 2 * TILE, 40], 7
    yield "many-workers", [12345, 54321, 99999], 15
    yield "resnet20", wl.make_workload(2).sizes, 8
    yield "resnet50", wl.make_workload(3).sizes, 7


@pytest.mark.parametrize("name,sizes,M", list(_layouts()), ids=[l[0] for l in _layouts()])
def test_guard_bands_stay_intact(name, sizes, M):
    w = wl.custom_workload(name, sizes, M, steps=2, scale_range=(1e-3, 1.0), config_id=500)
    flags = ef.EF_FLAG_WEIGHT_DECAY | ef.EF_FLAG_DIAGNOSTICS
    ws = Guarded(ef.ef_workspace_bytes(w.d, w.B, w.offsets, w.M, flags))
    eng = EFEngine(w.offsets, w.M, w.mu, w.eta, weight_decay=True, diagnostics=True, workspace=ws.inner)
    eng.set_weight_decay(1e-3)
    stride = (w.d + 3) // 4 * 4
    grads = Guarded(4 * w.M * stride, torch.float32)
    gall = grads.view[:w.M * stride].view(w.M, stride)
    out = Guarded(4 * w.d, torch.float32)
    msg = Guarded(4 * eng.message_units(0, w.B), torch.int32)
    es = w.element_scales("cuda")
    guards = [ws, grads, out, msg]
    for t in range(2):
        for i in range(w.M):
            w.draw_grad(t, i, "cuda", es, out=gall[i, :w.d])
        if t == 0:
            eng.worker_step_all(gall)
            eng.server_step()
        else:
            for i in range(w.M):
                eng.worker_step(i, gall[i, :w.d])
            eng.pack_message(0, 0, w.B, msg.view)
            half = max(1, w.B // 2)
            eng.server_step_range(half, w.B) if half < w.B else None
            eng.server_step_range(0, half)
            eng.pack_message(-1, 0, w.B, msg.view)
            eng.apply_update(0, w.B, msg.view[:eng.message_units(0, w.B)])
        ef.ef_get_residual(eng.ctx, -1, out.view.data_ptr())
        ef.ef_get_momentum(eng.ctx, w.M - 1, out.view.data_ptr())
    eng.vote_worker_step_all(gall)
    eng.vote_server_step()
    tk_ws = Guarded(ef.ef_topk_workspace_bytes(w.d))
    k = max(1, w.d // 50)
    idx = Guarded(8 * k, torch.int64)
    val = Guarded(4 * k, torch.float32)
    ef.ef_topk_compress(gall.data_ptr(), w.d, k, idx.view.data_ptr(), val.view.data_ptr(),
                        out.view.data_ptr(), tk_ws.inner.data_ptr(), tk_ws.inner.numel(), 0)
    torch.cuda.synchronize()
    ef.ef_check_status(eng.ctx)
    for g in guards + [tk_ws, idx, val]:
        assert g.intact(), "a guard band was overwritten"


@pytest.fixture
def checked_library():
    path = efbuild.build_library(debug=True)
    ef.use_library(path)
    try:
        assert ef.ef_debug_build()
        yield
    finally:
        torch.cuda.synchronize()
        ef.use_library(None)


def _run(w, steps, seed_cfg=510):
    eng = EFEngine(w.offsets, w.M, w.mu, w.eta)
    es = w.element_scales("cuda")
    for t in range(steps):
        for i in range(w.M):
            eng.worker_step(i, w.draw_grad(t, i, "cuda", es))
        eng.server_step()
    ef.ef_check_status(eng.ctx)
    return (eng.params().clone(), eng.server_words().clone(), eng.server_scales().clone(),
            eng.residual(-1), eng.residual(0), eng.momentum(w.M - 1))


@pytest.mark.parametrize("name,sizes,M", list(_layouts())[:4], ids=[l[0] for l in list(_layouts())[:4]])
def test_checked_build_equals_the_regular_build(name, sizes, M, checked_library):
    w = wl.custom_workload(name, sizes, M, steps=3, scale_range=(1e-3, 1.0), config_id=510)
    checked = _run(w, 3)
    ef.use_library(None)
    assert not ef.ef_debug_build()
    regular = _run(w, 3)
    ef.use_library(efbuild.DEBUG_LIB)
    for a, b in zip(checked, regular):
        assert torch.equal(a, b)


def test_checked_build_refuses_a_descriptor_past_the_end(checked_library):
    sizes = [TILE + 100, 777, 2 * BIG]
    w = wl.custom_workload("shift", sizes, 2, steps=1, config_id=511)
    ws = Guarded(ef.ef_workspace_bytes(w.d, w.B, w.offsets, w.M, 0))
    eng = EFEngine(w.offsets, w.M, w.mu, w.eta, workspace=ws.inner)
    g = torch.randn(w.d, device="cuda")
    eng.worker_step(0, g); eng.worker_step(1, g); eng.server_step()
    ef.ef_check_status(eng.ctx)                              # a valid problem reports nothing
    x_before = eng.params().clone()
    # the last tile (the last TILE elements of this small layout), moved TILE elements to the
    # right: it now ends past d, but still inside the workspace (the next array follows x directly)
    ef.ef_debug_shift_tile(eng.ctx, -1, TILE)
    eng.worker_step(0, g); eng.worker_step(1, g); eng.server_step()
    with pytest.raises(ef.EFError) as ei:
        ef.ef_check_status(eng.ctx)
    assert ei.value.status == ef.EF_ERR_BOUNDS
    # the refused tile was not processed: its parameters are unchanged
    lo = int(w.offsets[-1]) - TILE                           # start of the last tile
    assert torch.equal(eng.params()[lo:], x_before[lo:])
    assert ws.intact()
    ef.ef_check_status(eng.ctx)                              # the word was cleared


def test_regular_build_has_no_shift_hook():
    w = wl.custom_workload("hook", [64], 1, config_id=512)
    eng = EFEngine(w.offsets, w.M, w.mu, w.eta)
    with pytest.raises(ef.EFError) as ei:
        ef.ef_debug_shift_tile(eng.ctx, 0, 4)
    assert ei.value.status == ef.EF_ERR_BAD_STATE


def test_stream_probe_kernels_do_what_the_header_says():
    """The no-compute stream kernels behind bench.py --ceiling, inside guard bands."""
    n = 3 * TILE
    a, b, c = (Guarded(4 * n, torch.float32) for _ in range(3))
    gen = torch.Generator(device="cuda").manual_seed(4)
    a.view.copy_(torch.randn(n, device="cuda", generator=gen))
    b.view.copy_(torch.randn(n, device="cuda", generator=gen))
    c.view.copy_(torch.randn(n, device="cuda", generator=gen))
    a0, b0, c0 = a.view.clone(), b.view.clone(), c.view.clone()
    st = torch.cuda.current_stream().cuda_stream
    ef.ef_stream_probe(ef.EF_PROBE_3R2W, a.view.data_ptr(), b.view.data_ptr(), c.view.data_ptr(), n, st)
    assert torch.equal(a.view, a0) and torch.equal(b.view, b0 + a0) and torch.equal(c.view, c0 + (b0 + a0))
    b1 = b.view.clone()
    ef.ef_stream_probe(ef.EF_PROBE_1R1W, a.view.data_ptr(), b.view.data_ptr(), c.view.data_ptr(), n, st)
    pattern = torch.tensor([1.0, -1.0, 1.0, -1.0], device="cuda").repeat(n // 4)
    assert torch.equal(b.view, b1 + pattern)
    ef.ef_stream_probe(ef.EF_PROBE_COPY, a.view.data_ptr(), b.view.data_ptr(), c.view.data_ptr(), n, st)
    assert torch.equal(c.view, a0)
    torch.cuda.synchronize()
    assert a.intact() and b.intact() and c.intact()
