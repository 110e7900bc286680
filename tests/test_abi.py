"""Host-only checks of the C ABI: the library loads, exports every symbol the header declares,
and validates its arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import build as efbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    efbuild.build_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ef.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ef_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(ef.LIB_PATH)
    names = declared_symbols()
    assert "ef_init" in names and "ef_worker_step" in names and "ef_server_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in ef.h but not exported"
    assert sorted(ef.SIGNATURES) == names, "python binding and header disagree"


def test_workspace_bytes_accounts_for_all_state():
    d, B, M = 1 << 20, 16, 2
    off = np.arange(B + 1) * (d // B)
    n = ef.ef_workspace_bytes(d, B, off, M)
    state = 4 * d * (2 * M + 2)                  # x, etilde, and (m, e) per worker
    words = 4 * (d // 32) * (M + 1)
    assert state + words <= n <= state + words + (1 << 20)
    n2 = ef.ef_workspace_bytes(d, B, off, M, ef.EF_FLAG_HOST_STAGING)
    assert n2 - n == 2 * 4 * d
    n3 = ef.ef_workspace_bytes(d, B, off, M, ef.EF_FLAG_WEIGHT_DECAY)
    assert n3 - n == 4 * d


@pytest.mark.parametrize("d,offsets,M", [
    (0, [0], 1), (4, [0, 2, 2, 4], 1), (4, [1, 4], 1), (4, [0, 3], 1), (4, [0, 4], 0),
    (4, [0, 4], ef.EF_MAX_WORKERS + 1), (4, [0, 3, 2, 4], 1),
])
def test_invalid_problems_are_rejected(d, offsets, M):
    with pytest.raises(ef.EFError) as ei:
        ef.ef_workspace_bytes(d, len(offsets) - 1, offsets, M)
    assert ei.value.status == ef.EF_ERR_INVALID_ARG


def test_init_validates_before_using_the_device():
    off = [0, 64, 128]
    for mu, eta in [(1.0, 0.1), (-0.1, 0.1), (0.9, 0.0), (0.9, float("inf")), (float("nan"), 0.1)]:
        with pytest.raises(ef.EFError) as ei:
            ef.ef_init(128, 2, off, 2, mu, eta, 0, 256, 1 << 30, 0)
        assert ei.value.status == ef.EF_ERR_INVALID_ARG
    with pytest.raises(ef.EFError) as ei:
        ef.ef_init(128, 2, off, 2, 0.9, 0.1, 0, 0, 1 << 30, 0)
    assert ei.value.status == ef.EF_ERR_WORKSPACE
    with pytest.raises(ef.EFError) as ei:
        ef.ef_init(128, 2, off, 2, 0.9, 0.1, 0, 256, 16, 0)
    assert ei.value.status == ef.EF_ERR_WORKSPACE
    with pytest.raises(ef.EFError) as ei:
        ef.ef_init(128, 2, off, 2, 0.9, 0.1, 0, 264, 1 << 30, 0)
    assert ei.value.status == ef.EF_ERR_ALIGNMENT
    with pytest.raises(ef.EFError) as ei:
        ef.ef_init(128, 2, off, 2, 0.9, 0.1, 1 << 20, 256, 1 << 30, 0)    # unknown flag
    assert ei.value.status == ef.EF_ERR_INVALID_ARG
    for bad in (ef.EF_FLAG_FUSED_SCALE | ef.EF_FLAG_SPLIT_SCALE,          # contradictory flags
                ef.EF_FLAG_FUSED_SCALE | ef.EF_FLAG_DIAGNOSTICS):
        with pytest.raises(ef.EFError) as ei:
            ef.ef_init(128, 2, off, 2, 0.9, 0.1, bad, 256, 1 << 30, 0)
        assert ei.value.status == ef.EF_ERR_INVALID_ARG


def test_null_context_is_rejected():
    lib = ef.load_library()
    assert lib.ef_worker_step(None, 0, 16) == ef.EF_ERR_INVALID_ARG
    assert lib.ef_server_step(None) == ef.EF_ERR_INVALID_ARG
    assert lib.ef_destroy(None) == ef.EF_OK
    assert lib.ef_params(None) is None
    assert ef.ef_strerror(ef.EF_ERR_BAD_STATE) == "call order violated"


def test_later_entry_points_check_their_arguments_without_a_device():
    """Argument checks of the entry points that do not belong to the core path come before any
    device use, so they can be exercised without a GPU."""
    lib = ef.load_library()
    null = ctypes.c_void_p(None)
    for name, args in [
        ("ef_vote_worker_step", (null, 0, null)), ("ef_vote_worker_step_all", (null, null, 0)),
        ("ef_vote_server_step", (null,)), ("ef_server_step_range", (null, 0, 1, null, 0)),
        ("ef_apply_update", (null, 0, 1, null)), ("ef_pack_message", (null, 0, 0, 1, null)),
        ("ef_set_block_divisors", (null, null)), ("ef_block_sums", (null, 0, null)),
        ("ef_complete_scales", (null, 0, null)), ("ef_check_status", (null,)),
        ("ef_debug_shift_tile", (null, 0, 0)),
    ]:
        rc = getattr(lib, name)(*args)
        assert rc in (ef.EF_ERR_INVALID_ARG, ef.EF_ERR_BAD_STATE), (name, rc)
    assert lib.ef_message_units(null, 0, 1) == -1 and lib.ef_status_word(null) is None
    assert lib.ef_debug_build() in (0, 1)
    # top-k: sizes and null pointers
    out = ctypes.c_size_t(0)
    assert lib.ef_topk_workspace_bytes(0, ctypes.byref(out)) == ef.EF_ERR_INVALID_ARG
    assert lib.ef_topk_workspace_bytes(1 << 20, ctypes.byref(out)) == ef.EF_OK and out.value >= 3 * 2048 * 8
    assert lib.ef_topk_compress(null, 16, 4, null, null, null, null, 0, null) == ef.EF_ERR_INVALID_ARG
    buf = 4096                                                   # any non-null, 256-byte aligned value
    assert lib.ef_topk_compress(buf, 16, 17, buf, buf, None, buf, 1 << 20, None) == ef.EF_ERR_INVALID_ARG
    assert lib.ef_topk_compress(buf, 16, 4, buf, buf, None, buf, 8, None) == ef.EF_ERR_WORKSPACE
    # stream probe: n must be a positive multiple of 4096, pointers 16-byte aligned
    assert lib.ef_stream_probe(0, buf, buf, buf, 1000, None) == ef.EF_ERR_INVALID_ARG
    assert lib.ef_stream_probe(7, buf, buf, buf, 4096, None) == ef.EF_ERR_INVALID_ARG
    assert lib.ef_stream_probe(0, buf + 4, buf, buf, 4096, None) == ef.EF_ERR_ALIGNMENT
    assert lib.ef_worker_step_noalloc(buf, buf, buf, buf, (1 << 24) + 1, 0.9, buf, buf, None) == ef.EF_ERR_TOO_LARGE
