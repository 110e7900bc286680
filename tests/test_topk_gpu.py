"""GPU parity of the top-k compressor (ef_topk_compress), through the C ABI, against its oracle.
All outputs are integer or copied values, so the bar is exact equality."""
import numpy as np
import pytest
import torch

from oracle import topk_compress
from paper_1905_10936_b200 import binding as ef

pytestmark = pytest.mark.gpu


def gpu_topk(v: torch.Tensor, k: int, in_place: bool = False):
    n = v.numel()
    nbytes = ef.ef_topk_workspace_bytes(n)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    idx = torch.full((k,), -1, dtype=torch.int64, device="cuda")
    val = torch.full((k,), float("nan"), device="cuda")
    src = v.clone()
    resid = src if in_place else torch.full((n,), float("nan"), device="cuda")
    ef.ef_topk_compress(src.data_ptr(), n, k, idx.data_ptr(), val.data_ptr(), resid.data_ptr(),
                        ws.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), val.cpu().numpy(), resid.cpu().numpy()


def check(v: torch.Tensor, k: int, in_place: bool = False):
    idx, val, resid = gpu_topk(v.cuda(), k, in_place)
    ridx, rval, rresid = topk_compress(v.cpu().numpy(), k)
    assert np.array_equal(idx, ridx), f"n={v.numel()} k={k}: kept coordinates differ"
    assert np.array_equal(val, rval)
    assert np.array_equal(resid, rresid)


@pytest.mark.parametrize("n", [1, 2, 5, 31, 127, 4095, 4096, 4097, 3 * 4096 + 1, 10 * 4096 - 3, 70001])
def test_sizes_around_the_chunk_boundaries(n):
    gen = torch.Generator().manual_seed(n)
    v = torch.randn(n, generator=gen)
    for k in sorted({1, max(1, n // 100), max(1, n // 3), n - 1 if n > 1 else 1, n}):
        check(v, k)


@pytest.mark.parametrize("n", [10_000, 50_000])          # one-CTA path for short vectors, general path
@pytest.mark.parametrize("law", ["normal", "laplace", "cauchy", "quantised", "constant", "zeros", "denormal"])
def test_value_distributions_and_ties(law, n):
    gen = torch.Generator().manual_seed(7)
    if law == "normal":
        v = torch.randn(n, generator=gen)
    elif law == "laplace":
        u = torch.rand(n, generator=gen) - 0.5
        v = -torch.sign(u) * torch.log1p(-2 * u.abs().clamp(max=0.499999))
    elif law == "cauchy":
        v = torch.randn(n, generator=gen) / torch.randn(n, generator=gen).abs().clamp(min=1e-3)
    elif law == "quantised":
        v = torch.randint(-8, 9, (n,), generator=gen).float() * 0.25      # many equal magnitudes
    elif law == "constant":
        v = torch.where(torch.rand(n, generator=gen) < 0.5, -1.5, 1.5)    # every magnitude ties
    elif law == "zeros":
        v = torch.zeros(n); v[::3] = -0.0; v[7] = 1.0
    else:
        v = torch.randn(n, generator=gen) * 1e-41                          # binary32 denormals
    for k in (1, 13, n // 64, n // 2, n - 5):
        check(v, k)


def test_residual_may_overwrite_the_input():
    gen = torch.Generator().manual_seed(1)
    check(torch.randn(3 * 4096 + 77, generator=gen), 500, in_place=True)


@pytest.mark.parametrize("n,k", [(1 << 24, 1 << 14), ((1 << 26) + 12345, 1 << 20)])
def test_large_vectors(n, k):
    """Sizes that span thousands of chunks (the oracle sorts 2^26 values in a few seconds)."""
    gen = torch.Generator(device="cuda").manual_seed(n % 1000)
    v = torch.randn(n, device="cuda", generator=gen) * torch.rand(n, device="cuda", generator=gen)
    check(v.cpu(), k)


@pytest.mark.parametrize("law", ["one-bin", "constant", "two-levels", "narrow-then-wide"])
def test_vectors_whose_candidates_do_not_fit_the_list(law):
    """The keys that share the threshold's leading digit are normally a few per cent of the
    vector and are copied to a list; here they are (nearly) all of it, more than the list holds,
    and the later digits and the counts must come from the vector itself."""
    n = 300_000 + 77
    gen = torch.Generator().manual_seed(11)
    if law == "one-bin":
        v = (1.0 + torch.rand(n, generator=gen) * 0.05) * torch.where(torch.rand(n, generator=gen) < 0.5, -1.0, 1.0)
    elif law == "constant":
        v = torch.where(torch.rand(n, generator=gen) < 0.5, -2.5, 2.5)
    elif law == "two-levels":
        v = torch.where(torch.rand(n, generator=gen) < 0.3, 4.0, 1.0)          # k decides which level ties
    else:
        v = torch.randn(n, generator=gen)
        v[: n // 2] = 3.0 + torch.rand(n // 2, generator=gen) * 1e-3
    for k in (1, n // 1000, n // 10, n // 2 + 5, n - 1):
        check(v, k)


@pytest.mark.parametrize("n", [16383, 16384, 16385, 65536, 65537, 8 * 65536, 8 * 65536 + 8, 1_000_003])
def test_sizes_around_the_list_capacity(n):
    """Vectors of up to 16384 elements are handled by one CTA; beyond that the candidate list holds
    max(n/8, min(n, 65536)) keys.  Vectors on both sides of the break points,
    ordinary values (the list is used) and all-equal magnitudes (it is not, beyond 65536)."""
    gen = torch.Generator().manual_seed(n % 97)
    v = torch.randn(n, generator=gen)
    for k in (n // 100, n // 7):
        check(v, k)
    check(torch.full((n,), -0.75), n // 3)


def test_arguments_are_checked():
    v = torch.zeros(64, device="cuda")
    idx = torch.zeros(64, dtype=torch.int64, device="cuda")
    nbytes = ef.ef_topk_workspace_bytes(64)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    args = lambda n, k, w=ws.data_ptr(), wb=nbytes, src=v.data_ptr(): (
        src, n, k, idx.data_ptr(), v.data_ptr(), None, w, wb, 0)
    for n, k in ((64, 0), (64, 65), (0, 1)):
        with pytest.raises(ef.EFError) as ei:
            ef.ef_topk_compress(*args(n, k))
        assert ei.value.status == ef.EF_ERR_INVALID_ARG
    with pytest.raises(ef.EFError) as ei:
        ef.ef_topk_compress(*args(64, 4, wb=16))
    assert ei.value.status == ef.EF_ERR_WORKSPACE
    with pytest.raises(ef.EFError) as ei:
        ef.ef_topk_compress(*args(60, 4, src=v.data_ptr() + 4))
    assert ei.value.status == ef.EF_ERR_ALIGNMENT
    torch.cuda.synchronize()
