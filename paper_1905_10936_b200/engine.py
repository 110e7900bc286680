"""Convenience holder around the C-ABI context: owns the torch workspace tensor and exposes
the device views as torch tensors.  No arithmetic of the method happens here."""
from __future__ import annotations

import ctypes
from typing import Optional

import numpy as np
import torch

from . import binding as ef


def _as_tensor(ptr: int, n: int, dtype: torch.dtype, device: torch.device) -> torch.Tensor:
    """Zero-copy torch view of `n` elements of device memory at `ptr`."""
    itemsize = torch.empty((), dtype=dtype).element_size()

    class _Holder:
        __cuda_array_interface__ = {
            "shape": (n,), "typestr": {torch.float32: "<f4", torch.int32: "<i4",
                                       torch.float64: "<f8"}[dtype],
            "data": (ptr, False), "version": 3, "strides": (itemsize,),
        }
    return torch.as_tensor(_Holder(), device=device)


class EFEngine:
    """One dist-EF-blockSGDM problem on the current CUDA device."""

    def __init__(self, offsets, M: int, mu: float, eta: float, host_staging: bool = False,
                 scale_mode: str = "auto", weight_decay: bool = False, diagnostics: bool = False,
                 stream: Optional[torch.cuda.Stream] = None, device: Optional[torch.device] = None,
                 one_local_worker: bool = False, extra_flags: int = 0,
                 workspace: Optional[torch.Tensor] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("EFEngine needs a CUDA device (there is no CPU path)")
        self.device = torch.device(device if device is not None else f"cuda:{torch.cuda.current_device()}")
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        self.B = len(self.offsets) - 1
        self.d = int(self.offsets[-1])
        self.M = int(M)
        flags = ef.EF_FLAG_HOST_STAGING if host_staging else 0
        flags |= ef.EF_FLAG_WEIGHT_DECAY if weight_decay else 0
        flags |= ef.EF_FLAG_DIAGNOSTICS if diagnostics else 0
        flags |= ef.EF_FLAG_ONE_LOCAL_WORKER if one_local_worker else 0
        flags |= int(extra_flags)
        self.local_workers = 1 if one_local_worker else self.M
        flags |= {"auto": 0, "fused": ef.EF_FLAG_FUSED_SCALE, "split": ef.EF_FLAG_SPLIT_SCALE}[scale_mode]
        nbytes = ef.ef_workspace_bytes(self.d, self.B, self.offsets, self.M, flags)
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            if workspace is None:
                workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            assert workspace.is_cuda and workspace.dtype == torch.uint8 and workspace.is_contiguous()
            assert workspace.numel() >= nbytes and workspace.data_ptr() % 256 == 0
            self.workspace = workspace
            self.stream = stream if stream is not None else torch.cuda.current_stream()
            self.ctx = ef.ef_init(self.d, self.B, self.offsets, self.M, float(mu), float(eta), flags,
                                  self.workspace.data_ptr(), nbytes, self.stream.cuda_stream)
        self.W = ef.ef_num_words(self.ctx)

    def close(self):
        if getattr(self, "ctx", None):
            ef.ef_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- steps ------------------------------------------------------------------------------
    def worker_step(self, i: int, grad: torch.Tensor) -> None:
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.numel() == self.d
        assert grad.is_contiguous()
        ef.ef_worker_step(self.ctx, i, grad.data_ptr())

    def worker_step_all(self, grads: torch.Tensor) -> None:
        """grads: [M, stride] fp32 on the device, row i = gradient of worker i (stride >= d)."""
        assert grads.is_cuda and grads.dtype == torch.float32 and grads.dim() == 2
        assert grads.shape[0] == self.M and grads.shape[1] >= self.d and grads.stride(1) == 1
        ef.ef_worker_step_all(self.ctx, grads.data_ptr(), grads.stride(0))

    def worker_step_host(self, i: int, grad: torch.Tensor) -> None:
        assert (not grad.is_cuda) and grad.dtype == torch.float32 and grad.numel() == self.d
        assert grad.is_contiguous()
        ef.ef_worker_step_host(self.ctx, i, grad.data_ptr())

    def server_step(self) -> None:
        ef.ef_server_step(self.ctx)

    # ---- parameter-server protocol in pieces (block ranges, fused messages) -------------------
    def message_units(self, b0: int, b1: int) -> int:
        return ef.ef_message_units(self.ctx, b0, b1)

    def pack_message(self, who: int, b0: int, b1: int, dst: torch.Tensor) -> None:
        assert dst.is_cuda and dst.dtype == torch.int32 and dst.is_contiguous()
        assert dst.numel() >= self.message_units(b0, b1)
        ef.ef_pack_message(self.ctx, who, b0, b1, dst.data_ptr())

    def worker_step_push(self, i: int, grad: torch.Tensor, block_dst: torch.Tensor) -> None:
        """block_dst: int64 tensor of B device addresses on this device; block b's fused message
        [scale | words] is stored at block_dst[b] (own or peer-mapped memory)."""
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.is_contiguous() and grad.numel() == self.d
        assert block_dst.is_cuda and block_dst.dtype == torch.int64 and block_dst.is_contiguous()
        assert block_dst.numel() == self.B
        ef.ef_worker_step_push(self.ctx, i, grad.data_ptr(), block_dst.data_ptr())

    def push_message(self, who: int, b0: int, b1: int, dst_ptrs) -> None:
        """The fused message of blocks [b0, b1) written to every device address in dst_ptrs."""
        ef.ef_push_message(self.ctx, who, b0, b1, list(dst_ptrs))

    def server_step_range(self, b0: int, b1: int, msgs: Optional[torch.Tensor] = None) -> None:
        """msgs: [M, units] int32 on this device, row i = worker i's fused message for [b0, b1)."""
        if msgs is None:
            ef.ef_server_step_range(self.ctx, b0, b1, None, 0)
        else:
            assert msgs.is_cuda and msgs.dtype == torch.int32 and msgs.dim() == 2
            assert msgs.shape[0] == self.M and msgs.stride(1) == 1
            ef.ef_server_step_range(self.ctx, b0, b1, msgs.data_ptr(), msgs.stride(0))

    def apply_update(self, b0: int, b1: int, update: Optional[torch.Tensor] = None) -> None:
        if update is not None:
            assert update.is_cuda and update.dtype == torch.int32 and update.is_contiguous()
            assert update.numel() >= self.message_units(b0, b1)
        ef.ef_apply_update(self.ctx, b0, b1, update.data_ptr() if update is not None else None)

    # ---- blocks cut across devices ------------------------------------------------------------
    def set_block_divisors(self, full_len) -> None:
        assert len(full_len) == self.B
        ef.ef_set_block_divisors(self.ctx, full_len)

    def block_sums(self, who: int, dst: torch.Tensor) -> None:
        assert dst.is_cuda and dst.dtype == torch.float64 and dst.is_contiguous() and dst.numel() >= self.B
        ef.ef_block_sums(self.ctx, who, dst.data_ptr())

    def complete_scales(self, who: int, totals: torch.Tensor) -> None:
        assert totals.is_cuda and totals.dtype == torch.float64 and totals.is_contiguous()
        assert totals.numel() >= self.B
        ef.ef_complete_scales(self.ctx, who, totals.data_ptr())

    # ---- signum with majority vote (same state, same packed layout) -------------------------
    def vote_worker_step(self, i: int, grad: torch.Tensor) -> None:
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.numel() == self.d
        assert grad.is_contiguous()
        ef.ef_vote_worker_step(self.ctx, i, grad.data_ptr())

    def vote_worker_step_all(self, grads: torch.Tensor) -> None:
        assert grads.is_cuda and grads.dtype == torch.float32 and grads.dim() == 2
        assert grads.shape[0] == self.M and grads.shape[1] >= self.d and grads.stride(1) == 1
        ef.ef_vote_worker_step_all(self.ctx, grads.data_ptr(), grads.stride(0))

    def vote_worker_step_host(self, i: int, grad: torch.Tensor) -> None:
        assert (not grad.is_cuda) and grad.dtype == torch.float32 and grad.numel() == self.d
        assert grad.is_contiguous()
        ef.ef_vote_worker_step_host(self.ctx, i, grad.data_ptr())

    def vote_server_step(self) -> None:
        ef.ef_vote_server_step(self.ctx)

    def worker_diagnostics(self, i: int) -> torch.Tensor:
        """[B, 4] float64 view: ||p_b||_1, ||p_b||_2^2, ||g_b||_1, ||g_b||_2^2 of worker i's last step."""
        return _as_tensor(ef.ef_worker_diagnostics(self.ctx, i), 4 * self.B, torch.float64,
                          self.device).view(self.B, 4)

    def set_eta(self, eta: float) -> None:
        ef.ef_set_eta(self.ctx, float(eta))

    def set_weight_decay(self, lam: float) -> None:
        ef.ef_set_weight_decay(self.ctx, float(lam))

    def decay_momentum(self) -> torch.Tensor:
        return _as_tensor(ef.ef_decay_momentum(self.ctx), self.d, torch.float32, self.device)

    def read_update_host(self, words: torch.Tensor, scales: torch.Tensor) -> None:
        assert words.numel() == self.W and scales.numel() == self.B
        ef.ef_read_update_host(self.ctx, words.data_ptr(), scales.data_ptr())

    # ---- views ------------------------------------------------------------------------------
    def worker_words(self, i: int) -> torch.Tensor:
        return _as_tensor(ef.ef_worker_words(self.ctx, i), self.W, torch.int32, self.device)

    def worker_scales(self, i: int) -> torch.Tensor:
        return _as_tensor(ef.ef_worker_scales(self.ctx, i), self.B, torch.float32, self.device)

    def server_words(self) -> torch.Tensor:
        return _as_tensor(ef.ef_server_words(self.ctx), self.W, torch.int32, self.device)

    def server_scales(self) -> torch.Tensor:
        return _as_tensor(ef.ef_server_scales(self.ctx), self.B, torch.float32, self.device)

    def params(self) -> torch.Tensor:
        return _as_tensor(ef.ef_params(self.ctx), self.d, torch.float32, self.device)

    def momentum(self, i: int) -> torch.Tensor:
        out = torch.empty(self.d, dtype=torch.float32, device=self.device)
        ef.ef_get_momentum(self.ctx, i, out.data_ptr())
        return out

    def residual(self, i: int = -1) -> torch.Tensor:
        out = torch.empty(self.d, dtype=torch.float32, device=self.device)
        ef.ef_get_residual(self.ctx, i, out.data_ptr())
        return out

    def set_state(self, i: int, momentum: Optional[torch.Tensor], residual: torch.Tensor) -> None:
        ef.ef_set_state(self.ctx, i, momentum.data_ptr() if momentum is not None else None,
                        residual.data_ptr())

    @property
    def step_count(self) -> int:
        return ef.ef_step_count(self.ctx)

    @property
    def launch_count(self) -> int:
        return ef.ef_launch_count(self.ctx)
