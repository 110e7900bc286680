"""The no-allocation worker step (ef_worker_step_noalloc) against the regular entry point.

Who needs it: hosts that may not call cudaMalloc where they step the optimizer (code running
under another framework's allocator or stream, plugins with a fixed arena, latency-critical
loops).  The variant keeps its scratch in a fixed array inside the library, so the caller passes
only inputs and outputs.  Here it is called twice in a row through the C ABI, carrying its state
in caller-owned tensors, and every output is compared with what ef_worker_step produces for a
layout with one block of the same size: packed words and scale bit for bit, momentum and the
residual within the tolerance of the other parity tests.

This file sorts last on purpose, so that a run that stops at the first failure has already run
every other test; it does not depend on anything the other tests leave behind.
"""
import numpy as np
import pytest
import torch

from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200.engine import EFEngine

pytestmark = pytest.mark.gpu

RTOL = 1e-5


def _materialise(p: torch.Tensor, s: torch.Tensor) -> torch.Tensor:
    """Residual e = p - s*sign(p) (sign(+-0) = +1) from the deferred form the caller keeps."""
    return torch.where(p < 0, p + s, p - s)


@pytest.mark.parametrize("n", [5 * 4096 + 37, 1000, 16384 * 3, 4096])
def test_two_calls_in_a_row_match_the_regular_worker_step(n):
    mu = 0.9
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev); gen.manual_seed(1234 + n)
    grads = [torch.randn(n, device=dev, generator=gen) * 0.3 for _ in range(2)]

    eng = EFEngine([0, n], 1, mu, 0.1)
    m = torch.zeros(n, device=dev)
    p = torch.zeros(n, device=dev)
    s_prev = torch.zeros(1, device=dev)
    words = torch.empty((n + 31) // 32, dtype=torch.int32, device=dev)
    scale = torch.empty(1, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    for call, g in enumerate(grads):
        eng.worker_step(0, g)
        ef.ef_worker_step_noalloc(g.data_ptr(), m.data_ptr(), p.data_ptr(), s_prev.data_ptr(), n, mu,
                                  words.data_ptr(), scale.data_ptr(), stream)
        torch.cuda.synchronize()
        assert torch.equal(words, eng.worker_words(0)), f"call {call}: packed words differ"
        ref_scale = eng.worker_scales(0)
        assert abs(scale.item() - ref_scale.item()) <= RTOL * abs(ref_scale.item())
        assert s_prev.item() == scale.item()
        ref_m, ref_e = eng.momentum(0), eng.residual(0)
        assert (m - ref_m).abs().max().item() <= RTOL * ref_m.abs().max().item()
        e = _materialise(p, s_prev)
        assert (e - ref_e).abs().max().item() <= RTOL * ref_e.abs().max().item()
        eng.server_step()          # closes the iteration of the regular engine


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
