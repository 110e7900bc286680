"""ctypes loader for the CPU oracles: dist-EF-blockSGDM (Algorithm 4) in ``ef_oracle.cpp``,
signum with majority vote and the top-k compressor in ``vote_topk_oracle.cpp``.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg, never by the CUDA package.  All arithmetic lives in
the two C++ files; this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "ef_oracle.cpp"), os.path.join(_HERE, "vote_topk_oracle.cpp")]
_LIB = os.path.join(_HERE, "libef_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no implicit FMA contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= max(os.path.getmtime(p) for p in _SRCS)):
        return _LIB
    cmd = ["g++", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c++17",
           "-shared", "-fPIC", "-o", _LIB] + _SRCS
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
    lib.efo_init.restype = vp
    lib.efo_init.argtypes = [i64, i32, vp, i32, f32, f32]
    lib.efo_destroy.restype = None
    lib.efo_destroy.argtypes = [vp]
    lib.efo_num_words.restype = i64
    lib.efo_num_words.argtypes = [vp]
    lib.efo_step_count.restype = i64
    lib.efo_step_count.argtypes = [vp]
    lib.efo_worker_step.restype = i64
    lib.efo_worker_step.argtypes = [vp, i32, vp, vp, vp, i64]
    lib.efo_server_step.restype = i64
    lib.efo_server_step.argtypes = [vp, vp, vp, i64]
    lib.efo_set_eta.restype = i32
    lib.efo_set_eta.argtypes = [vp, f32]
    lib.efo_set_weight_decay.restype = i32
    lib.efo_set_weight_decay.argtypes = [vp, f32]
    for name in ("efo_params", "efo_last_p", "efo_decay_momentum"):
        getattr(lib, name).restype = vp
        getattr(lib, name).argtypes = [vp]
    for name in ("efo_momentum", "efo_residual", "efo_words", "efo_scales"):
        getattr(lib, name).restype = vp
        getattr(lib, name).argtypes = [vp, i32]
    lib.efo_set_diagnostics.restype = None
    lib.efo_set_diagnostics.argtypes = [vp, i32]
    lib.efo_diagnostics.restype = vp
    lib.efo_diagnostics.argtypes = [vp, i32]
    # signum with majority vote, top-k
    lib.sgo_init.restype = vp
    lib.sgo_init.argtypes = [i64, i32, vp, i32, f32, f32]
    lib.sgo_destroy.restype = None
    lib.sgo_destroy.argtypes = [vp]
    for name in ("sgo_num_words", "sgo_step_count"):
        getattr(lib, name).restype = i64
        getattr(lib, name).argtypes = [vp]
    lib.sgo_worker_step.restype = i32
    lib.sgo_worker_step.argtypes = [vp, i32, vp]
    lib.sgo_server_step.restype = i32
    lib.sgo_server_step.argtypes = [vp]
    lib.sgo_params.restype = vp
    lib.sgo_params.argtypes = [vp]
    for name in ("sgo_momentum", "sgo_words"):
        getattr(lib, name).restype = vp
        getattr(lib, name).argtypes = [vp, i32]
    lib.tko_compress.restype = i32
    lib.tko_compress.argtypes = [vp, i64, i64, vp, vp, vp]
    _lib = lib
    return lib


def _view(ptr: int, n: int, dtype) -> np.ndarray:
    buf = (ctypes.c_char * (n * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype, count=n)


class Oracle:
    """One optimisation problem held by the oracle (state lives in C++ memory)."""

    ADOPT_CAP = 1 << 16

    def __init__(self, offsets, M: int, mu: float, eta: float, diagnostics: bool = False):
        lib = _load()
        self._lib = lib
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        self.B = len(self.offsets) - 1
        self.d = int(self.offsets[-1]) if len(self.offsets) else 0
        self.M = int(M)
        self._h = lib.efo_init(self.d, self.B, self.offsets.ctypes.data, self.M,
                               float(mu), float(eta))
        if not self._h:
            raise ValueError("efo_init rejected the arguments")
        self.W = int(lib.efo_num_words(self._h))
        if diagnostics:
            lib.efo_set_diagnostics(self._h, 1)
        self._adopt = np.zeros(self.ADOPT_CAP, dtype=np.int64)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.efo_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    # ---- steps --------------------------------------------------------------
    def worker_step(self, i: int, grad: np.ndarray,
                    hint: Optional[np.ndarray] = None) -> np.ndarray:
        """Runs worker i; returns the flat indices of adopted (in-zone, hinted) elements."""
        g = np.ascontiguousarray(grad, dtype=np.float32)
        assert g.shape == (self.d,)
        hp = None
        if hint is not None:
            hint = np.ascontiguousarray(hint, dtype=np.uint32)
            assert hint.shape == (self.W,)
            hp = hint.ctypes.data
        n = self._lib.efo_worker_step(self._h, int(i), g.ctypes.data, hp,
                                      self._adopt.ctypes.data, self.ADOPT_CAP)
        if n < 0:
            raise RuntimeError("efo_worker_step: bad worker index or worker already stepped")
        return self._adopt[:min(n, self.ADOPT_CAP)].copy()

    def server_step(self, hint: Optional[np.ndarray] = None) -> np.ndarray:
        hp = None
        if hint is not None:
            hint = np.ascontiguousarray(hint, dtype=np.uint32)
            assert hint.shape == (self.W,)
            hp = hint.ctypes.data
        n = self._lib.efo_server_step(self._h, hp, self._adopt.ctypes.data, self.ADOPT_CAP)
        if n < 0:
            raise RuntimeError("efo_server_step: not every worker has stepped")
        return self._adopt[:min(n, self.ADOPT_CAP)].copy()

    def set_eta(self, eta: float) -> None:
        if self._lib.efo_set_eta(self._h, float(eta)) != 0:
            raise RuntimeError("efo_set_eta: bad value or called in the middle of an iteration")

    def set_weight_decay(self, lam: float) -> None:
        if self._lib.efo_set_weight_decay(self._h, float(lam)) != 0:
            raise RuntimeError("efo_set_weight_decay: bad value or called in the middle of an iteration")

    @property
    def decay_momentum(self) -> np.ndarray:
        return _view(self._lib.efo_decay_momentum(self._h), self.d, np.float32)

    # ---- views (live; copy if you need a snapshot) ---------------------------
    @property
    def t(self) -> int:
        return int(self._lib.efo_step_count(self._h))

    @property
    def x(self) -> np.ndarray:
        return _view(self._lib.efo_params(self._h), self.d, np.float32)

    @property
    def last_p(self) -> np.ndarray:
        return _view(self._lib.efo_last_p(self._h), self.d, np.float32)

    def momentum(self, i: int) -> np.ndarray:
        return _view(self._lib.efo_momentum(self._h, i), self.d, np.float32)

    def residual(self, i: int = -1) -> np.ndarray:
        return _view(self._lib.efo_residual(self._h, i), self.d, np.float32)

    def words(self, i: int = -1) -> np.ndarray:
        return _view(self._lib.efo_words(self._h, i), self.W, np.uint32)

    def scales(self, i: int = -1) -> np.ndarray:
        return _view(self._lib.efo_scales(self._h, i), self.B, np.float32)

    def diagnostics(self, i: int) -> np.ndarray:
        """[B, 4] float64: ||p_b||_1, ||p_b||_2^2, ||g_b||_1, ||g_b||_2^2 of worker i's last call
        (recorded only by an Oracle created with diagnostics=True)."""
        return _view(self._lib.efo_diagnostics(self._h, i), 4 * self.B, np.float64).reshape(self.B, 4)


class SignumOracle:
    """signum / signSGD with majority vote on one problem (state lives in C++ memory)."""

    def __init__(self, offsets, M: int, mu: float, eta: float):
        lib = _load()
        self._lib = lib
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        self.B = len(self.offsets) - 1
        self.d = int(self.offsets[-1]) if len(self.offsets) else 0
        self.M = int(M)
        self._h = lib.sgo_init(self.d, self.B, self.offsets.ctypes.data, self.M, float(mu), float(eta))
        if not self._h:
            raise ValueError("sgo_init rejected the arguments")
        self.W = int(lib.sgo_num_words(self._h))

    def close(self):
        if getattr(self, "_h", None):
            self._lib.sgo_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def worker_step(self, i: int, grad: np.ndarray) -> None:
        g = np.ascontiguousarray(grad, dtype=np.float32)
        assert g.shape == (self.d,)
        if self._lib.sgo_worker_step(self._h, int(i), g.ctypes.data) != 0:
            raise RuntimeError("sgo_worker_step: bad worker index or worker already stepped")

    def server_step(self) -> None:
        if self._lib.sgo_server_step(self._h) != 0:
            raise RuntimeError("sgo_server_step: not every worker has stepped")

    @property
    def t(self) -> int:
        return int(self._lib.sgo_step_count(self._h))

    @property
    def x(self) -> np.ndarray:
        return _view(self._lib.sgo_params(self._h), self.d, np.float32)

    def momentum(self, i: int) -> np.ndarray:
        return _view(self._lib.sgo_momentum(self._h, i), self.d, np.float32)

    def words(self, i: int = -1) -> np.ndarray:
        return _view(self._lib.sgo_words(self._h, i), self.W, np.uint32)


def topk_compress(v: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Top-k of v: (kept indices in increasing order, their values, residual v - C(v))."""
    v = np.ascontiguousarray(v, dtype=np.float32)
    n = v.shape[0]
    idx = np.empty(k, dtype=np.int64)
    val = np.empty(k, dtype=np.float32)
    resid = np.empty(n, dtype=np.float32)
    if _load().tko_compress(v.ctypes.data, n, int(k), idx.ctypes.data, val.ctypes.data,
                            resid.ctypes.data) != 0:
        raise ValueError("tko_compress rejected the arguments")
    return idx, val, resid
