"""Seeded synthetic inputs and workload shapes for rolling-KV chunk attention.

This module only draws random numbers, rounds them to bf16 bit patterns and
names shapes.  It holds none of the attention or cache arithmetic, so both the
CUDA path and the CPU oracle can be fed from it without sharing method code.

Value recipe: every tensor is i.i.d. N(0, 1) drawn from numpy's Philox
counter-based generator keyed by ``seed``, produced in float32 and rounded to
bf16 with round-to-nearest-even.  Tensors travel as uint16 bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (nearest, ties to even); returns uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def normal_bf16(seed: int, shape) -> np.ndarray:
    """i.i.d. N(0,1) tensor as bf16 bit patterns (uint16), reproducible from ``seed``."""
    gen = np.random.Generator(np.random.Philox(key=int(seed)))
    x = gen.standard_normal(size=tuple(int(s) for s in shape), dtype=np.float32)
    return f32_to_bf16_bits(x)


def tensor_seed(config: int, tensor_index: int) -> int:
    """Seed convention: 1000 * workload number + index of the tensor inside it."""
    return 1000 * int(config) + int(tensor_index)


@dataclass(frozen=True)
class Workload:
    """Shape of one synthetic workload (names follow the rolling-cache notation).

    batch B, cache_batch B_c (B or 1), heads H, head_dim D, tokens_per_frame T,
    chunk_frames c, sink_frames S, window_frames L (slots of the sliding window),
    held_frames = frames resident in the cache while the chunk is attended.
    """
    name: str
    batch: int
    cache_batch: int
    heads: int
    head_dim: int
    tokens_per_frame: int
    chunk_frames: int
    sink_frames: int
    window_frames: int
    held_frames: int

    @property
    def chunk_tokens(self) -> int:
        return self.chunk_frames * self.tokens_per_frame

    @property
    def ctx_tokens(self) -> int:
        return self.held_frames * self.tokens_per_frame

    @property
    def total_keys(self) -> int:
        return self.ctx_tokens + self.chunk_tokens

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    def fwd_flops(self) -> float:
        return 4.0 * self.batch * self.heads * self.chunk_tokens * self.total_keys * self.head_dim

    def bwd_flops(self) -> float:
        return (self.batch * self.heads * self.chunk_tokens * self.head_dim
                * (6.0 * self.total_keys + 4.0 * self.chunk_tokens))


# The five synthetic workloads.  Capacity S+L counts every attended frame, the
# chunk included, so the caller evicts down to S+L-c held frames before a chunk.
TINY = Workload("tiny", 1, 1, 2, 64, 16, 3, 0, 6, 3)
LAYER_FWD = Workload("layer_fwd", 1, 1, 12, 128, 1560, 3, 3, 18, 18)
ROLLOUT = Workload("rollout", 4, 4, 12, 128, 1560, 3, 3, 12, 12)
RL_UPDATE = Workload("rl_update", 2, 2, 12, 128, 1560, 3, 3, 18, 18)
SWEEP_KEYS = (1560, 4680, 16380, 32760, 65520)
