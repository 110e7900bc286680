"""Thin ctypes binding of libef (see include/ef.h): argument marshalling only.

Every function has the name and the argument order of its C counterpart.  Device pointers
are passed as integers (``tensor.data_ptr()``); torch is used only to own device memory and
to name the CUDA stream.  There is no fallback: if the shared library is missing the import
of a symbol raises, and on a device that is not compute capability 10.x ``ef_init`` fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libef.so")

EF_OK = 0
EF_ERR_INVALID_ARG = 1
EF_ERR_BAD_STATE = 2
EF_ERR_WORKSPACE = 3
EF_ERR_ALIGNMENT = 4
EF_ERR_CUDA = 5
EF_ERR_UNSUPPORTED_DEVICE = 6
EF_ERR_TIMEOUT = 7
EF_ERR_TOO_LARGE = 8
EF_ERR_NO_MEMORY = 9
EF_ERR_BOUNDS = 10
EF_NOALLOC_MAX_ELEMS = 1 << 24
EF_FLAG_HOST_STAGING = 1
EF_FLAG_FUSED_SCALE = 2
EF_FLAG_SPLIT_SCALE = 4
EF_FLAG_WEIGHT_DECAY = 8
EF_FLAG_DIAGNOSTICS = 16
EF_FLAG_ONE_LOCAL_WORKER = 32
EF_FLAG_SERVER_NO_BULK = 512
EF_FLAG_PROGRAMMATIC_LAUNCH = 1024
EF_FLAG_SEPARATE_UPDATE = 2048
EF_MAX_WORKERS = 4096
EF_PROBE_3R2W, EF_PROBE_1R1W, EF_PROBE_COPY = 0, 1, 2

_vp, _i64, _i32, _u32, _f32 = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32,
                               ctypes.c_float)

# name -> (restype, argtypes); mirrors include/ef.h
SIGNATURES = {
    "ef_workspace_bytes": (ctypes.c_int, [_i64, _i32, _vp, _i32, _u32, ctypes.POINTER(ctypes.c_size_t)]),
    "ef_init": (ctypes.c_int, [ctypes.POINTER(_vp), _i64, _i32, _vp, _i32, _f32, _f32, _u32, _vp,
                               ctypes.c_size_t, _vp]),
    "ef_worker_step": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_worker_step_all": (ctypes.c_int, [_vp, _vp, _i64]),
    "ef_worker_step_host": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_server_step": (ctypes.c_int, [_vp]),
    "ef_worker_diagnostics": (_vp, [_vp, _i32]),
    "ef_set_eta": (ctypes.c_int, [_vp, _f32]),
    "ef_set_weight_decay": (ctypes.c_int, [_vp, _f32]),
    "ef_decay_momentum": (_vp, [_vp]),
    "ef_read_update_host": (ctypes.c_int, [_vp, _vp, _vp]),
    "ef_worker_words": (_vp, [_vp, _i32]),
    "ef_worker_scales": (_vp, [_vp, _i32]),
    "ef_server_words": (_vp, [_vp]),
    "ef_server_scales": (_vp, [_vp]),
    "ef_params": (_vp, [_vp]),
    "ef_num_words": (_i64, [_vp]),
    "ef_get_momentum": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_get_residual": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_set_state": (ctypes.c_int, [_vp, _i32, _vp, _vp]),
    "ef_step_count": (ctypes.c_int, [_vp, ctypes.POINTER(_i64)]),
    "ef_check_status": (ctypes.c_int, [_vp]),
    "ef_status_word": (_vp, [_vp]),
    "ef_debug_build": (ctypes.c_int, []),
    "ef_debug_shift_tile": (ctypes.c_int, [_vp, _i64, _i64]),
    "ef_launch_count": (_i64, [_vp]),
    "ef_worker_step_noalloc": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _f32, _vp, _vp, _vp]),
    "ef_message_units": (_i64, [_vp, _i32, _i32]),
    "ef_pack_message": (ctypes.c_int, [_vp, _i32, _i32, _i32, _vp]),
    "ef_server_step_range": (ctypes.c_int, [_vp, _i32, _i32, _vp, _i64]),
    "ef_worker_step_push": (ctypes.c_int, [_vp, _i32, _vp, _vp]),
    "ef_push_message": (ctypes.c_int, [_vp, _i32, _i32, _i32, _i32, _vp]),
    "ef_apply_update": (ctypes.c_int, [_vp, _i32, _i32, _vp]),
    "ef_set_block_divisors": (ctypes.c_int, [_vp, _vp]),
    "ef_block_sums": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_complete_scales": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_vote_worker_step": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_vote_worker_step_all": (ctypes.c_int, [_vp, _vp, _i64]),
    "ef_vote_worker_step_host": (ctypes.c_int, [_vp, _i32, _vp]),
    "ef_vote_server_step": (ctypes.c_int, [_vp]),
    "ef_topk_workspace_bytes": (ctypes.c_int, [_i64, ctypes.POINTER(ctypes.c_size_t)]),
    "ef_topk_compress": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]),
    "ef_stream_probe": (ctypes.c_int, [_i32, _vp, _vp, _vp, _i64, _vp]),
    "ef_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "ef_last_cuda_error": (ctypes.c_int, [_vp]),
    "ef_destroy": (ctypes.c_int, [_vp]),
}

_lib = None


def use_library(path: Optional[str] = None) -> None:
    """Selects the shared library the binding calls from now on (None: the regular libef.so);
    used to run the checked build (libef_debug.so).  Contexts of one library must not be
    passed to another."""
    global _lib, LIB_PATH
    LIB_PATH = path if path is not None else os.path.join(_PKG, "libef.so")
    _lib = None


def load_library() -> ctypes.CDLL:
    """Loads the selected library (libef.so in the package directory unless use_library chose
    another); raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_1905_10936_b200.build` (there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class EFError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = load_library().ef_strerror(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


def _check(status: int, where: str) -> None:
    if status != EF_OK:
        raise EFError(status, where)


def _offsets_array(offsets: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(offsets, dtype=np.int64)


# ---- functions with the C names ------------------------------------------------------------
def ef_workspace_bytes(d: int, B: int, offsets, M: int, flags: int = 0) -> int:
    off = _offsets_array(offsets)
    out = ctypes.c_size_t(0)
    _check(load_library().ef_workspace_bytes(d, B, off.ctypes.data, M, flags, ctypes.byref(out)),
           "ef_workspace_bytes")
    return out.value


def ef_init(d: int, B: int, offsets, M: int, mu: float, eta: float, flags: int,
            workspace_ptr: int, workspace_bytes: int, cuda_stream: int) -> int:
    off = _offsets_array(offsets)
    ctx = _vp(None)
    _check(load_library().ef_init(ctypes.byref(ctx), d, B, off.ctypes.data, M, mu, eta, flags,
                                  workspace_ptr, workspace_bytes, cuda_stream), "ef_init")
    return ctx.value


def ef_worker_step(ctx: int, i: int, grad_ptr: int) -> None:
    _check(load_library().ef_worker_step(ctx, i, grad_ptr), "ef_worker_step")


def ef_worker_step_all(ctx: int, grads_ptr: int, stride: int) -> None:
    _check(load_library().ef_worker_step_all(ctx, grads_ptr, stride), "ef_worker_step_all")


def ef_worker_step_host(ctx: int, i: int, grad_host_ptr: int) -> None:
    _check(load_library().ef_worker_step_host(ctx, i, grad_host_ptr), "ef_worker_step_host")


def ef_server_step(ctx: int) -> None:
    _check(load_library().ef_server_step(ctx), "ef_server_step")


def ef_worker_diagnostics(ctx: int, i: int) -> Optional[int]:
    return load_library().ef_worker_diagnostics(ctx, i)


def ef_set_eta(ctx: int, eta: float) -> None:
    _check(load_library().ef_set_eta(ctx, eta), "ef_set_eta")


def ef_set_weight_decay(ctx: int, lam: float) -> None:
    _check(load_library().ef_set_weight_decay(ctx, lam), "ef_set_weight_decay")


def ef_decay_momentum(ctx: int) -> Optional[int]:
    return load_library().ef_decay_momentum(ctx)


def ef_read_update_host(ctx: int, words_host_ptr: int, scales_host_ptr: int) -> None:
    _check(load_library().ef_read_update_host(ctx, words_host_ptr, scales_host_ptr),
           "ef_read_update_host")


def ef_worker_words(ctx: int, i: int) -> Optional[int]:
    return load_library().ef_worker_words(ctx, i)


def ef_worker_scales(ctx: int, i: int) -> Optional[int]:
    return load_library().ef_worker_scales(ctx, i)


def ef_server_words(ctx: int) -> Optional[int]:
    return load_library().ef_server_words(ctx)


def ef_server_scales(ctx: int) -> Optional[int]:
    return load_library().ef_server_scales(ctx)


def ef_params(ctx: int) -> Optional[int]:
    return load_library().ef_params(ctx)


def ef_num_words(ctx: int) -> int:
    return load_library().ef_num_words(ctx)


def ef_get_momentum(ctx: int, i: int, dst_ptr: int) -> None:
    _check(load_library().ef_get_momentum(ctx, i, dst_ptr), "ef_get_momentum")


def ef_get_residual(ctx: int, i: int, dst_ptr: int) -> None:
    _check(load_library().ef_get_residual(ctx, i, dst_ptr), "ef_get_residual")


def ef_set_state(ctx: int, i: int, momentum_ptr: Optional[int], residual_ptr: int) -> None:
    _check(load_library().ef_set_state(ctx, i, momentum_ptr, residual_ptr), "ef_set_state")


def ef_step_count(ctx: int) -> int:
    t = _i64(0)
    _check(load_library().ef_step_count(ctx, ctypes.byref(t)), "ef_step_count")
    return t.value


def ef_check_status(ctx: int) -> None:
    _check(load_library().ef_check_status(ctx), "ef_check_status")


def ef_debug_build() -> bool:
    return bool(load_library().ef_debug_build())


def ef_debug_shift_tile(ctx: int, tile: int, delta: int) -> None:
    _check(load_library().ef_debug_shift_tile(ctx, tile, delta), "ef_debug_shift_tile")


def ef_status_word(ctx: int) -> Optional[int]:
    return load_library().ef_status_word(ctx)


def ef_launch_count(ctx: int) -> int:
    return load_library().ef_launch_count(ctx)


def ef_worker_step_noalloc(grad_ptr: int, momentum_ptr: int, residual_ptr: int,
                           residual_scale_ptr: int, n: int, mu: float, words_ptr: int,
                           scale_ptr: int, cuda_stream: int) -> None:
    """Worker step of one block without any workspace (scratch is a fixed array in the library);
    for callers that must not allocate device memory.  See include/ef.h for the contract."""
    _check(load_library().ef_worker_step_noalloc(grad_ptr, momentum_ptr, residual_ptr,
                                                 residual_scale_ptr, n, mu, words_ptr, scale_ptr,
                                                 cuda_stream), "ef_worker_step_noalloc")


def ef_message_units(ctx: int, b0: int, b1: int) -> int:
    return load_library().ef_message_units(ctx, b0, b1)


def ef_pack_message(ctx: int, who: int, b0: int, b1: int, dst_ptr: int) -> None:
    _check(load_library().ef_pack_message(ctx, who, b0, b1, dst_ptr), "ef_pack_message")


def ef_worker_step_push(ctx: int, i: int, grad_ptr: int, block_dst_ptr: int) -> None:
    """block_dst_ptr: device array of B device pointers (one destination per block)."""
    _check(load_library().ef_worker_step_push(ctx, i, grad_ptr, block_dst_ptr), "ef_worker_step_push")


def ef_push_message(ctx: int, who: int, b0: int, b1: int, dst_ptrs) -> None:
    """dst_ptrs: sequence of device addresses; the message is written to each of them."""
    arr = (ctypes.c_void_p * len(dst_ptrs))(*[int(p) for p in dst_ptrs])
    _check(load_library().ef_push_message(ctx, who, b0, b1, len(dst_ptrs), arr), "ef_push_message")


def ef_server_step_range(ctx: int, b0: int, b1: int, msgs_ptr: Optional[int], msg_stride: int) -> None:
    _check(load_library().ef_server_step_range(ctx, b0, b1, msgs_ptr, msg_stride), "ef_server_step_range")


def ef_apply_update(ctx: int, b0: int, b1: int, update_ptr: Optional[int]) -> None:
    _check(load_library().ef_apply_update(ctx, b0, b1, update_ptr), "ef_apply_update")


def ef_set_block_divisors(ctx: int, full_len) -> None:
    arr = np.ascontiguousarray(full_len, dtype=np.int64)
    _check(load_library().ef_set_block_divisors(ctx, arr.ctypes.data), "ef_set_block_divisors")


def ef_block_sums(ctx: int, who: int, dst_ptr: int) -> None:
    _check(load_library().ef_block_sums(ctx, who, dst_ptr), "ef_block_sums")


def ef_complete_scales(ctx: int, who: int, totals_ptr: int) -> None:
    _check(load_library().ef_complete_scales(ctx, who, totals_ptr), "ef_complete_scales")


def ef_vote_worker_step(ctx: int, i: int, grad_ptr: int) -> None:
    _check(load_library().ef_vote_worker_step(ctx, i, grad_ptr), "ef_vote_worker_step")


def ef_vote_worker_step_all(ctx: int, grads_ptr: int, stride: int) -> None:
    _check(load_library().ef_vote_worker_step_all(ctx, grads_ptr, stride), "ef_vote_worker_step_all")


def ef_vote_worker_step_host(ctx: int, i: int, grad_host_ptr: int) -> None:
    _check(load_library().ef_vote_worker_step_host(ctx, i, grad_host_ptr), "ef_vote_worker_step_host")


def ef_vote_server_step(ctx: int) -> None:
    _check(load_library().ef_vote_server_step(ctx), "ef_vote_server_step")


def ef_topk_workspace_bytes(n: int) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().ef_topk_workspace_bytes(n, ctypes.byref(out)), "ef_topk_workspace_bytes")
    return out.value


def ef_topk_compress(v_ptr: int, n: int, k: int, idx_ptr: int, val_ptr: int, resid_ptr: Optional[int],
                     workspace_ptr: int, workspace_bytes: int, cuda_stream: int) -> None:
    _check(load_library().ef_topk_compress(v_ptr, n, k, idx_ptr, val_ptr, resid_ptr, workspace_ptr,
                                           workspace_bytes, cuda_stream), "ef_topk_compress")


def ef_stream_probe(mode: int, a_ptr: int, b_ptr: int, c_ptr: int, n: int, cuda_stream: int) -> None:
    """No-compute stream kernel (measurement aid); see include/ef.h."""
    _check(load_library().ef_stream_probe(mode, a_ptr, b_ptr, c_ptr, n, cuda_stream), "ef_stream_probe")


def ef_last_cuda_error(ctx: int) -> int:
    return load_library().ef_last_cuda_error(ctx)


def ef_strerror(status: int) -> str:
    return load_library().ef_strerror(status).decode()


def ef_destroy(ctx: int) -> None:
    _check(load_library().ef_destroy(ctx), "ef_destroy")
