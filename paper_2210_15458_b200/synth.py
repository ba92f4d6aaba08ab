"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path.

This module holds no arithmetic of the sampling method itself: it only draws
random logits, tables, start tokens and shifts with numpy's PCG64 generator and
rounds them to the storage dtype.  Both sides read the *materialised* arrays it
returns (bf16 arrays are returned as uint16 bit patterns), so they see exactly
the same stored values.

The five workloads follow the shapes and value distributions of the synthetic
configurations this library is measured on:

  c1  bigram table 512x512 fp32 ~ N(0, 2^2), 4 start tokens x 32 codes, T=16
  c2  256 lanes x V=32000 bf16 ~ N(0, 3^2) + Zipf-like bias, temp 0.7, top_k=40
  c3  1024 lanes x V=128256 fp32 ~ N(0, 4^2) + bias, temp 1.0, top_p=0.9
  c4  bigram table 32128x32128 bf16 ~ N(0, 2.5^2) + column bias, 64 x 32 codes,
      T<=128, EOS id 1, temp 0.8
  c5  L lanes x V=256000 bf16 ~ N(0, 3^2) + bias, temp 0.8, top_k=64, top_p=0.95

"Zipf-like bias" is bias_j = -1.5 * ln(rank_j + 1) with rank a seeded random
permutation of 0..V-1 shared by every lane (row) of the tensor.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

F32 = 0
BF16 = 1


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = a.view(np.uint32)
    rounded = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def stored_as_f64(arr: np.ndarray, dtype: int) -> np.ndarray:
    """The stored values widened exactly to fp64 (for tests that need plain numbers)."""
    if dtype == BF16:
        return bf16_bits_to_f32(arr).astype(np.float64)
    return np.asarray(arr, dtype=np.float32).astype(np.float64)


def zipf_bias(V: int, seed: int, scale: float = 1.5) -> np.ndarray:
    rank = np.random.default_rng(seed).permutation(V)
    return (-scale * np.log(rank.astype(np.float64) + 1.0)).astype(np.float32)


def logits_rows(rows: int, V: int, sigma: float, dtype: int, seed: int,
                bias: Optional[np.ndarray] = None, block_rows: int = 256) -> np.ndarray:
    """rows x V logits ~ N(0, sigma^2) (+ bias per column), stored in `dtype`.

    Generated in row blocks from one generator, so the result does not depend on
    block_rows.  Returns float32 [rows, V] for F32, uint16 [rows, V] for BF16.
    """
    rng = np.random.default_rng(seed)
    out = np.empty((rows, V), dtype=np.float32 if dtype == F32 else np.uint16)
    for r0 in range(0, rows, block_rows):
        r1 = min(rows, r0 + block_rows)
        x = rng.standard_normal((r1 - r0, V), dtype=np.float32)
        x *= np.float32(sigma)
        if bias is not None:
            x += bias[None, :]
        out[r0:r1] = x if dtype == F32 else f32_to_bf16_bits(x)
    return out


def uniform_shift(seed: int) -> float:
    return float(np.random.default_rng(seed).random())


def iid_codes(n: int, seed: int) -> np.ndarray:
    """Independent U[0,1) codes (ordinary ancestral sampling through the same path)."""
    return np.random.default_rng(seed).random(n)


def start_tokens(S: int, lo: int, hi: int, seed: int) -> np.ndarray:
    """S start tokens uniform on [lo, hi] inclusive."""
    return np.random.default_rng(seed).integers(lo, hi + 1, size=S).astype(np.int32)


@dataclass
class StepWorkload:
    name: str
    lanes: int
    V: int
    dtype: int
    sigma: float
    temp: float
    top_k: int
    top_p: float
    seed_logits: int
    seed_perm: int
    seed_shift: int
    N: int = 0  # lattice size (defaults to lanes)

    def __post_init__(self):
        if self.N == 0:
            self.N = self.lanes

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == F32 else 2

    def shift(self) -> float:
        return uniform_shift(self.seed_shift)

    def logits(self, lanes: Optional[int] = None, seed_offset: int = 0) -> np.ndarray:
        """First `lanes` rows of the workload's logits (rows come from one stream, so a
        prefix of the rows equals the prefix of the full tensor)."""
        n = self.lanes if lanes is None else lanes
        bias = zipf_bias(self.V, self.seed_perm)
        return logits_rows(n, self.V, self.sigma, self.dtype, self.seed_logits + 1000 * seed_offset, bias)


@dataclass
class BigramWorkload:
    name: str
    V: int
    dtype: int
    sigma: float
    S: int
    N: int
    T: int
    eos: int
    temp: float
    top_k: int
    top_p: float
    seed_table: int
    seed_perm: Optional[int]
    seed_starts: int
    seed_shift: int
    start_lo: int = 1
    eos_bias: Optional[float] = None  # if set, overrides the EOS column's bias
    extra: dict = field(default_factory=dict)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == F32 else 2

    @property
    def lanes(self) -> int:
        return self.S * self.N

    def shift(self) -> float:
        return uniform_shift(self.seed_shift)

    def starts(self) -> np.ndarray:
        return start_tokens(self.S, self.start_lo, self.V - 1, self.seed_starts)

    def column_bias(self) -> Optional[np.ndarray]:
        if self.seed_perm is None:
            return None
        b = zipf_bias(self.V, self.seed_perm)
        if self.eos_bias is not None:
            b[self.eos] = np.float32(self.eos_bias)
        return b

    def table(self, rows: Optional[int] = None) -> np.ndarray:
        n = self.V if rows is None else rows
        return logits_rows(n, self.V, self.sigma, self.dtype, self.seed_table, self.column_bias())


def c1() -> BigramWorkload:
    return BigramWorkload("c1", V=512, dtype=F32, sigma=2.0, S=4, N=32, T=16, eos=0, temp=1.0,
                          top_k=0, top_p=1.0, seed_table=0, seed_perm=None, seed_starts=2,
                          seed_shift=1, start_lo=1)


def c2() -> StepWorkload:
    return StepWorkload("c2", lanes=256, V=32000, dtype=BF16, sigma=3.0, temp=0.7, top_k=40,
                        top_p=1.0, seed_logits=20, seed_perm=21, seed_shift=22)


def c3(lanes: int = 1024) -> StepWorkload:
    return StepWorkload("c3", lanes=lanes, V=128256, dtype=F32, sigma=4.0, temp=1.0, top_k=0,
                        top_p=0.9, seed_logits=30, seed_perm=31, seed_shift=32, N=1024)


def c4(eos_bias: Optional[float] = None, V: int = 32128, S: int = 64, T: int = 128) -> BigramWorkload:
    return BigramWorkload("c4", V=V, dtype=BF16, sigma=2.5, S=S, N=32, T=T, eos=1, temp=0.8,
                          top_k=0, top_p=1.0, seed_table=40, seed_perm=41, seed_starts=42,
                          seed_shift=43, start_lo=2, eos_bias=eos_bias)


def c5(lanes: int = 1024) -> StepWorkload:
    return StepWorkload("c5", lanes=lanes, V=256000, dtype=BF16, sigma=3.0, temp=0.8, top_k=64,
                        top_p=0.95, seed_logits=50, seed_perm=51, seed_shift=52, N=lanes)


def reward_table(V: int, seed: int) -> np.ndarray:
    """Per-token rewards r[v] ~ N(0, 1) for the additive sequence reward of the estimator runs."""
    return np.random.default_rng(seed).normal(0.0, 1.0, V)
