"""The no-allocation worker step (ef_worker_step_noalloc) against the regular entry point and
against the CPU oracle.

Who needs it: hosts that may not call cudaMalloc where they step the optimizer (code running
under another framework's allocator or stream, plugins with a fixed arena, latency-critical
loops).  The variant keeps its scratch in a fixed array inside the library, so the caller passes
only inputs and outputs.  Here it is called several times in a row through the C ABI, carrying
its state in caller-owned tensors.  Every output must equal, bit for bit, what ef_worker_step
produces for a layout with one block of the same size (the header promises exactly that), and
must agree with the oracle's worker step under the tolerances of the other parity tests.

This file sorts last on purpose, so that a run that stops at the first failure has already run
every other test; it does not depend on anything the other tests leave behind.
"""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200.engine import EFEngine

pytestmark = pytest.mark.gpu

RTOL = 1e-5


def _materialise(p: torch.Tensor, s: torch.Tensor) -> torch.Tensor:
    """Residual e = p - s*sign(p) (sign(+-0) = +1) from the deferred form the caller keeps."""
    return torch.where(p < 0, p + s, p - s)


class _NoAllocState:
    """The caller-owned state of one block for ef_worker_step_noalloc."""

    def __init__(self, n, dev):
        self.n = n
        self.m = torch.zeros(n, device=dev)
        self.p = torch.zeros(n, device=dev)
        self.s_prev = torch.zeros(1, device=dev)
        self.words = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
        self.scale = torch.empty(1, device=dev)

    def step(self, g, mu):
        ef.ef_worker_step_noalloc(g.data_ptr(), self.m.data_ptr(), self.p.data_ptr(),
                                  self.s_prev.data_ptr(), self.n, mu, self.words.data_ptr(),
                                  self.scale.data_ptr(), torch.cuda.current_stream().cuda_stream)


def _check_call(st, eng, orc, g, mu, what):
    eng.worker_step(0, g)
    st.step(g, mu)
    torch.cuda.synchronize()
    # against the regular entry point: identical in every bit
    assert torch.equal(st.words, eng.worker_words(0)), f"{what}: packed words differ"
    assert st.scale.item() == eng.worker_scales(0).item(), f"{what}: scale differs"
    assert st.s_prev.item() == st.scale.item()
    assert torch.equal(st.m, eng.momentum(0)), f"{what}: momentum differs"
    e = _materialise(st.p, st.s_prev)
    assert torch.equal(e, eng.residual(0)), f"{what}: residual differs"
    # against the oracle (one block, one worker): words bit-exact after tie-zone adoption,
    # scale / momentum / residual within 1e-5 (of the largest magnitude for the vectors)
    gw = st.words.cpu().numpy().view(np.uint32)
    adopted = orc.worker_step(0, g.cpu().numpy(), hint=gw)
    assert np.array_equal(orc.words(0), gw), f"{what}: words differ from the oracle's"
    ref_s = float(orc.scales(0)[0])
    assert abs(st.scale.item() - ref_s) <= RTOL * abs(ref_s)
    for got, ref in ((st.m, orc.momentum(0)), (e, orc.residual(0))):
        got = got.cpu().numpy()
        assert np.abs(got - ref).max() <= RTOL * np.abs(ref).max()
        if len(adopted) == 0 and st.scale.item() == ref_s:
            assert np.array_equal(got, ref)
    eng.server_step()              # closes the iteration on both reference sides (M = 1)
    orc.server_step()


@pytest.mark.parametrize("n", [5 * 4096 + 37, 1000, 16384 * 3, 4096])
def test_two_calls_in_a_row_match_the_regular_worker_step_and_the_oracle(n):
    mu = 0.9
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev); gen.manual_seed(1234 + n)
    eng = EFEngine([0, n], 1, mu, 0.1)
    orc = Oracle([0, n], 1, mu, 0.1)
    st = _NoAllocState(n, dev)
    for call in range(2):
        g = torch.randn(n, device=dev, generator=gen) * 0.3
        _check_call(st, eng, orc, g, mu, f"n={n} call {call}")


def test_a_smaller_problem_after_a_larger_one_ignores_stale_scratch():
    """All calls share one scratch array, which keeps the previous call's partial sums: a
    40-chunk problem leaves 40 slots behind, the 3-chunk problem after it must read only its
    own three; then the large one again."""
    mu = 0.5
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev); gen.manual_seed(99)
    sizes = [40 * 4096 + 5, 3 * 4096 - 8]
    engs = [EFEngine([0, n], 1, mu, 0.1) for n in sizes]
    orcs = [Oracle([0, n], 1, mu, 0.1) for n in sizes]
    sts = [_NoAllocState(n, dev) for n in sizes]
    for call, k in enumerate([0, 1, 0, 1]):
        g = torch.randn(sizes[k], device=dev, generator=gen) * (10.0 if k == 0 else 0.01)
        _check_call(sts[k], engs[k], orcs[k], g, mu, f"problem {k} call {call}")


def test_limits_are_enforced_without_launching():
    dev = torch.device("cuda")
    buf = torch.zeros(64, device=dev)
    w = torch.zeros(4, dtype=torch.int32, device=dev)
    one = torch.zeros(1, device=dev)
    args = lambda n, g=buf: (g.data_ptr(), buf.data_ptr(), buf.data_ptr(), one.data_ptr(), n, 0.9,
                             w.data_ptr(), one.data_ptr(), 0)
    with pytest.raises(ef.EFError) as ei:
        ef.ef_worker_step_noalloc(*args(ef.EF_NOALLOC_MAX_ELEMS + 1))
    assert ei.value.status == ef.EF_ERR_TOO_LARGE
    assert "scratch" in str(ei.value)
    with pytest.raises(ef.EFError) as ei:
        ef.ef_worker_step_noalloc(*args(0))
    assert ei.value.status == ef.EF_ERR_INVALID_ARG
    with pytest.raises(ef.EFError) as ei:
        ef.ef_worker_step_noalloc(buf.data_ptr() + 4, buf.data_ptr(), buf.data_ptr(), one.data_ptr(),
                                  8, 0.9, w.data_ptr(), one.data_ptr(), 0)
    assert ei.value.status == ef.EF_ERR_ALIGNMENT
    torch.cuda.synchronize()
