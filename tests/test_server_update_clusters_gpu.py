"""ef_server_step on layouts of few chunks whose blocks span at most 16 chunks: ONE kernel,
launched in thread-block clusters, does the server lines and the parameter update (a cluster per
block; the block's scale is agreed at the cluster barrier; every CTA updates its own chunk of x).
It must equal the two-kernel path (EF_FLAG_SEPARATE_UPDATE) bit for bit in everything the step
leaves behind, launch one kernel less, and replay from a CUDA graph."""
import numpy as np
import pytest
import torch

from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import workloads as wl
from paper_1905_10936_b200.engine import EFEngine

pytestmark = pytest.mark.gpu

CH = 4096


def _wl(sizes, M, steps=4, cid=420):
    return wl.custom_workload("server-update", sizes, M, 0.9, 0.1, steps, "normal", (1e-3, 1.0), config_id=cid)


@pytest.mark.parametrize("sizes,M", [
    ([65536] * 16, 2),                                       # every block a full cluster of 16 chunks
    ([5, 3, 31, 33, 63, 65, 127, 129], 3),                   # single-chunk blocks only, unaligned starts
    ([700, 33, 4096, 10, 2500, 64, 1200] * 5, 8),            # 35 single-chunk blocks: three shared clusters
    ([3 * CH + 5, 640, 10, 16 * CH, 333, 9 * CH + 1], 7),    # ragged multi-chunk blocks, scalar tiles behind them
    ([2 * CH, CH // 2, 3 * CH + 36, 100, 4 * CH + 8, 777], 17),   # M beyond the table path
    ([2 * CH, CH // 2, 3 * CH + 36, 100, 4 * CH + 8, 777], 12),   # the wide table
    ([12345, 54321, 9999], 1),
])
def test_one_launch_equals_the_two_kernel_path(sizes, M):
    w = _wl(sizes, M)
    one = EFEngine(w.offsets, M, w.mu, w.eta)
    two = EFEngine(w.offsets, M, w.mu, w.eta, extra_flags=ef.EF_FLAG_SEPARATE_UPDATE)
    x0 = torch.randn(w.d, device="cuda", generator=torch.Generator("cuda").manual_seed(3))
    one.params().copy_(x0); two.params().copy_(x0)
    es = w.element_scales("cuda")
    etas = [0.1, 0.1, 0.05, 0.2]
    for t in range(w.steps):
        if t > 0:
            one.set_eta(etas[t]); two.set_eta(etas[t])
        for i in range(M):
            g = w.draw_grad(t, i, "cuda", es)
            one.worker_step(i, g); two.worker_step(i, g)
        n1, n2 = one.launch_count, two.launch_count
        one.server_step(); two.server_step()
        assert one.launch_count - n1 == 1 and two.launch_count - n2 == 2
        assert torch.equal(one.params(), two.params()), f"x after step {t}"
        assert torch.equal(one.server_words(), two.server_words())
        assert torch.equal(one.server_scales(), two.server_scales())
        assert torch.equal(one.residual(-1), two.residual(-1))
    assert one.step_count == two.step_count == w.steps


@pytest.mark.parametrize("sizes", [[17 * CH, 100], [CH] * 1025])
def test_layouts_outside_the_rule_keep_two_kernels(sizes):
    """A block of more than 16 chunks, or more than 1024 chunks in all: the ordinary path."""
    w = _wl(sizes, 2)
    e = EFEngine(w.offsets, 2, w.mu, w.eta)
    es = w.element_scales("cuda")
    for i in range(2):
        e.worker_step(i, w.draw_grad(0, i, "cuda", es))
    n = e.launch_count
    e.server_step()
    assert e.launch_count - n >= 2


def test_weight_decay_keeps_the_update_kernel():
    """The decay side path lives in the update kernel: with lambda > 0 the call uses two launches."""
    w = _wl([3 * CH + 5, 640, 10], 2)
    e = EFEngine(w.offsets, 2, w.mu, w.eta, weight_decay=True)
    e.set_weight_decay(0.01)
    es = w.element_scales("cuda")
    for i in range(2):
        e.worker_step(i, w.draw_grad(0, i, "cuda", es))
    n = e.launch_count
    e.server_step()
    assert e.launch_count - n == 2


def test_one_launch_replays_from_a_cuda_graph():
    w = _wl([65536] * 4 + [100, 5000], 2)
    b = EFEngine(w.offsets, 2, w.mu, w.eta, extra_flags=ef.EF_FLAG_SEPARATE_UPDATE)
    es = w.element_scales("cuda")
    grads = torch.stack([w.draw_grad(0, i, "cuda", es) for i in range(2)])
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ga = EFEngine(w.offsets, 2, w.mu, w.eta, stream=stream)
        ga.worker_step_all(grads); ga.server_step()             # warm-up outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            ga.worker_step_all(grads); ga.server_step()
        for _ in range(3):
            graph.replay()
        stream.synchronize()
    for _ in range(4):
        b.worker_step_all(grads); b.server_step()
    # one eager step and three replays (the capture itself runs nothing) leave what four eager steps leave
    assert torch.equal(ga.params(), b.params())
    assert torch.equal(ga.residual(-1), b.residual(-1))


@pytest.mark.parametrize("sizes,M", [([65536] * 16, 2), ([3 * CH + 5, 640, 10, 16 * CH, 333, 9 * CH + 1], 7)])
def test_programmatic_launches_change_nothing(sizes, M):
    """With EF_FLAG_PROGRAMMATIC_LAUNCH the worker kernel loads the worker's state, and the
    one-launch server kernel its x values, before they wait for the kernel ahead of them.  State
    imports (ef_set_state) directly before a step, steps back to back and a parameter overwrite by
    a torch kernel in between must give what ordinary launches give."""
    w = _wl(sizes, M, steps=6, cid=421)
    pdl = EFEngine(w.offsets, M, w.mu, w.eta, extra_flags=ef.EF_FLAG_PROGRAMMATIC_LAUNCH)
    ref = EFEngine(w.offsets, M, w.mu, w.eta, extra_flags=ef.EF_FLAG_SEPARATE_UPDATE)
    es = w.element_scales("cuda")
    gen = torch.Generator("cuda").manual_seed(5)
    for t in range(w.steps):
        stride = (w.d + 3) // 4 * 4                        # rows start on 16-byte boundaries
        grads = torch.zeros(M, stride, device="cuda")
        for i in range(M):
            w.draw_grad(t, i, "cuda", es, out=grads[i, :w.d])
        if t == 2:                                         # imported state, used by the very next kernel
            m = torch.randn(w.d, device="cuda", generator=gen)
            e = torch.randn(w.d, device="cuda", generator=gen) * 1e-2
            for eng in (pdl, ref):
                for i in range(M):
                    eng.set_state(i, m, e)
        if t == 4:
            for eng in (pdl, ref):
                eng.params().mul_(0.5)
        for eng in (pdl, ref):
            if t % 2:
                eng.worker_step_all(grads)
            else:
                for i in range(M):
                    eng.worker_step(i, grads[i, :w.d])
            eng.server_step()
        assert torch.equal(pdl.params(), ref.params()), f"x after step {t}"
        assert torch.equal(pdl.server_words(), ref.server_words())
        for i in range(M):
            assert torch.equal(pdl.momentum(i), ref.momentum(i))
            assert torch.equal(pdl.residual(i), ref.residual(i))
