"""Synthetic workloads: block layouts and seeded gradient generators.

This module is the only code shared by the CUDA path's tests/bench and the CPU
oracle's tests.  It holds no arithmetic of the method (no momentum, no
compression, no packing): only the block partitions ("one block per parameter
tensor", Section 3.2) of the five benchmark layouts and the random gradients
that stand in for the paper's real ResNet-20 / ResNet-50 gradients
(Sections 4.1 and 4.2), whose datasets are not available here.

Gradients are drawn with a seeded ``torch.Generator`` on whatever device the
caller names.  Parity tests draw once and hand the *same buffer* to both sides,
so nothing depends on reproducing a random stream elsewhere.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

BASE_SEED = 190510936


# --------------------------------------------------------------------------
# Block layouts
# --------------------------------------------------------------------------

def _offsets(sizes: Sequence[int]) -> np.ndarray:
    off = np.zeros(len(sizes) + 1, dtype=np.int64)
    np.cumsum(np.asarray(sizes, dtype=np.int64), out=off[1:])
    return off


def flat_sizes(num_blocks: int, block_size: int) -> List[int]:
    return [block_size] * num_blocks


def resnet20_cifar_sizes() -> List[int]:
    """ResNet-20 for CIFAR: 3x3 convolutions, BN gamma/beta vectors, fc 64x10 + bias.

    Network order: stem conv 3->16 with its BN pair, three stages of widths
    16/32/64 with three basic blocks (two 3x3 convs, each followed by a BN pair)
    per stage, then the classifier.  One block per tensor.
    """
    sizes = [3 * 16 * 9, 16, 16]
    inp = 16
    for width in (16, 32, 64):
        for _ in range(3):
            for conv_in in (inp, width):
                sizes += [conv_in * width * 9, width, width]
            inp = width
    sizes += [64 * 10, 10]
    return sizes


def resnet50_sizes() -> List[int]:
    """ResNet-50 (ImageNet): bottleneck stages 3/4/6/3, widths 64..2048, fc 2048x1000."""
    sizes = [3 * 64 * 49, 64, 64]
    inp = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for k in range(blocks):
            out = 4 * planes
            sizes += [inp * planes, planes, planes]
            sizes += [planes * planes * 9, planes, planes]
            sizes += [planes * out, out, out]
            if k == 0:
                sizes += [inp * out, out, out]
            inp = out
    sizes += [2048 * 1000, 1000]
    return sizes


def gpt2_medium_sizes() -> List[int]:
    """GPT-2-medium-shaped: 24 layers, width 1024, token and position embeddings."""
    w = 1024
    sizes = [50257 * w, 1024 * w]
    for _ in range(24):
        sizes += [w, w, w * 3 * w, 3 * w, w * w, w, w, w, w * 4 * w, 4 * w, 4 * w * w, w]
    return sizes


@dataclass
class Workload:
    """One benchmark configuration: layout, worker count, hyper-parameters, gradient law."""
    name: str
    config_id: int
    sizes: List[int]
    M: int
    mu: float
    eta: float
    steps: int
    law: str                       # "normal" | "laplace"
    scale_range: Optional[Tuple[float, float]]   # per-block log-uniform range, None = unit scale
    offsets: np.ndarray = field(init=False)

    def __post_init__(self):
        self.offsets = _offsets(self.sizes)

    @property
    def d(self) -> int:
        return int(self.offsets[-1])

    @property
    def B(self) -> int:
        return len(self.sizes)

    @property
    def num_words(self) -> int:
        return int(sum((s + 31) // 32 for s in self.sizes))

    # ---- gradient generators -------------------------------------------------
    def block_scales(self) -> np.ndarray:
        """Per-block gradient magnitude s_b, drawn once per layout (a property of the
        tensor: shared by all workers and steps)."""
        if self.scale_range is None:
            return np.ones(self.B, dtype=np.float64)
        lo, hi = self.scale_range
        rng = np.random.Generator(np.random.PCG64(BASE_SEED + self.config_id))
        return np.exp(rng.uniform(math.log(lo), math.log(hi), size=self.B))

    def element_scales(self, device) -> Optional[torch.Tensor]:
        """s_b repeated over each block's elements (fp32, length d); None for unit scale."""
        if self.scale_range is None:
            return None
        sb = torch.tensor(self.block_scales(), dtype=torch.float32)
        sz = torch.tensor(self.sizes, dtype=torch.int64)
        return torch.repeat_interleave(sb, sz).to(device)

    def grad_seed(self, step: int, worker: int) -> int:
        return BASE_SEED + 1_000_003 * self.config_id + 1009 * step + worker

    def draw_grad(self, step: int, worker: int, device,
                  elem_scales: Optional[torch.Tensor] = None,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Gradient of worker `worker` at iteration `step`: fp32 vector of length d."""
        gen = torch.Generator(device=device)
        gen.manual_seed(self.grad_seed(step, worker))
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device=device)
        if self.law == "normal":
            out.normal_(0.0, 1.0, generator=gen)
        elif self.law == "laplace":
            # inverse CDF of Laplace(0, 1); |u| is kept strictly below 1/2 so log1p stays finite
            out.uniform_(-0.5, 0.5, generator=gen)
            a = out.abs().clamp_(max=0.5 - 2.0 ** -25)
            mag = torch.log1p(-2.0 * a).neg_()
            out.copy_(torch.where(out < 0, -mag, mag))
        else:
            raise ValueError(self.law)
        if self.scale_range is not None:
            if elem_scales is None:
                elem_scales = self.element_scales(device)
            out.mul_(elem_scales)
        return out


def make_workload(config_id: int) -> Workload:
    """The five benchmark configurations (1-based ids)."""
    if config_id == 1:
        return Workload("C1-flat-2^20", 1, flat_sizes(16, 65536), M=2, mu=0.9, eta=0.1,
                        steps=10, law="normal", scale_range=None)
    if config_id == 2:
        return Workload("C2-resnet20-cifar", 2, resnet20_cifar_sizes(), M=8, mu=0.9, eta=0.1,
                        steps=10, law="normal", scale_range=(1e-3, 1e-1))
    if config_id == 3:
        return Workload("C3-resnet50", 3, resnet50_sizes(), M=7, mu=0.9, eta=0.1,
                        steps=10, law="laplace", scale_range=(1e-4, 1e-1))
    if config_id == 4:
        return Workload("C4-flat-2^28", 4, flat_sizes(256, 1 << 20), M=7, mu=0.9, eta=0.1,
                        steps=20, law="normal", scale_range=None)
    if config_id == 5:
        return Workload("C5-gpt2-medium", 5, gpt2_medium_sizes(), M=4, mu=0.9, eta=0.1,
                        steps=10, law="normal", scale_range=(1e-5, 1e-2))
    raise ValueError(f"unknown config {config_id}")


def custom_workload(name: str, sizes: Sequence[int], M: int, mu: float = 0.9, eta: float = 0.1,
                    steps: int = 10, law: str = "normal",
                    scale_range: Optional[Tuple[float, float]] = None,
                    config_id: int = 99) -> Workload:
    return Workload(name, config_id, list(sizes), M, mu, eta, steps, law, scale_range)


# --------------------------------------------------------------------------
# Sharding of a layout over ranks (whole blocks per rank; no exchange needed
# because every operation of the method is per element or per block)
# --------------------------------------------------------------------------

def shard_blocks(sizes: Sequence[int], world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous range of whole blocks [b0, b1) owned by `rank`.

    Greedy split by cumulative element count so that shards are balanced; every
    rank gets a (possibly empty) contiguous range and the ranges tile [0, B).
    """
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    off = _offsets(sizes)
    d = int(off[-1])
    cuts = [0]
    for r in range(1, world_size):
        target = d * r / world_size
        # first block boundary at or after the target, but never before the previous cut
        b = int(np.searchsorted(off, target, side="left"))
        b = min(max(b, cuts[-1]), len(sizes))
        cuts.append(b)
    cuts.append(len(sizes))
    return cuts[rank], cuts[rank + 1]


@dataclass
class ElementShard:
    """One rank's share of a layout cut by ELEMENT count (blocks may be cut): the pieces it
    holds, as a layout of its own."""
    elem_lo: int                   # first element (flat index in the whole vector)
    elem_hi: int
    local_sizes: List[int]         # sizes of the local blocks (whole blocks and pieces)
    full_sizes: List[int]          # size of the whole block each local block belongs to
    global_block: List[int]        # index of that block in the whole layout
    offset_in_block: List[int]     # where the local block starts inside it


def shard_elements(sizes: Sequence[int], world_size: int, rank: int, granule: int = 4096) -> ElementShard:
    """Contiguous element range owned by `rank` when the flat vector is cut into `world_size`
    nearly equal parts.  A cut may fall inside a block, but only at a multiple of `granule`
    elements from the block's start (granule must be a multiple of 32, so that every piece
    starts on a packed-word boundary of the whole block's message).  The ranges tile [0, d).

    A rank then holds each block it intersects as a local block of its own; for a piece the
    scale needs the sum of all pieces' L1 norms (one number per cut block, see
    ef_set_block_divisors / ef_block_sums / ef_complete_scales)."""
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    if granule % 32 != 0 or granule <= 0:
        raise ValueError("granule must be a positive multiple of 32")
    off = _offsets(sizes)
    d = int(off[-1])

    def cut(r: int) -> int:
        if r <= 0:
            return 0
        if r >= world_size:
            return d
        target = d * r // world_size
        b = int(np.searchsorted(off, target, side="right")) - 1      # block that holds the target
        b = min(max(b, 0), len(sizes) - 1)
        return int(off[b]) + (target - int(off[b])) // granule * granule

    lo, hi = cut(rank), cut(rank + 1)
    shard = ElementShard(lo, hi, [], [], [], [])
    for b, size in enumerate(sizes):
        s, e = max(lo, int(off[b])), min(hi, int(off[b + 1]))
        if e > s:
            shard.local_sizes.append(e - s)
            shard.full_sizes.append(int(size))
            shard.global_block.append(b)
            shard.offset_in_block.append(s - int(off[b]))
    return shard
