"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests.

This module holds no attention arithmetic: it draws Gaussian samples, rounds
them once to bf16 (round to nearest even) and hands out bit patterns, plus the
row-sampling helper used when a full-size comparison is too large.  It imports
neither the oracle nor the CUDA binding, so both sides can use it.

The workloads mirror the paper's evaluation, which uses synthetic shapes only
(single head, L in {4096 .. 32768}, d = 128, Section "Results"); there is no
dataset behind them.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class AttnCase:
    """One attention workload: shapes, input standard deviations and stream id."""
    name: str
    B: int
    H: int
    L: int
    d: int
    sigma_qk: float = 1.0
    sigma_v: float = 1.0
    cfg_id: int = 0

    @property
    def flops(self) -> float:
        return 4.0 * self.B * self.H * float(self.L) ** 2 * self.d

    @property
    def elems(self) -> int:
        return self.B * self.H * self.L * self.d


_SQRT3 = float(np.sqrt(3.0))

# The five benchmark configurations.  "N(0,3)" in the sequence sweep is read as
# variance 3 (standard deviation sqrt(3)): with standard deviation 3 the outputs
# exceed 4 in magnitude, where half a bf16 ulp (1.56e-2) is already above the
# 1e-2 max-abs tolerance, so no bf16-output implementation could pass.
CONFIGS = {
    "cfg1": AttnCase("cfg1", 1, 1, 256, 64, cfg_id=1),
    "cfg2": AttnCase("cfg2", 1, 8, 2048, 128, cfg_id=2),
    "cfg3": AttnCase("cfg3", 1, 1, 16384, 128, cfg_id=3),
    **{f"cfg4_L{L}": AttnCase(f"cfg4_L{L}", 1, 4, L, 128, sigma_qk=_SQRT3, cfg_id=4)
       for L in (1024, 2048, 4096, 8192, 16384, 32768)},
    "cfg5a": AttnCase("cfg5a", 4, 32, 4096, 128, cfg_id=5),
    "cfg5b": AttnCase("cfg5b", 4, 32, 8192, 64, cfg_id=6),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 with round-to-nearest-even; returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    bits = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        bits[nan] = np.uint16(0x7FC0)
    return bits


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def gaussian_bf16(shape, sigma: float, seed: int, cfg_id: int, tensor_id: int) -> np.ndarray:
    """i.i.d. N(0, sigma^2) in fp32, rounded once to bf16; one stream per (seed, cfg, tensor)."""
    rng = np.random.default_rng([seed, cfg_id, tensor_id])
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    return f32_to_bf16_bits(x)


def make_qkv(case: AttnCase, seed: int = 0):
    """Q, K, V as uint16 bf16 bit patterns, contiguous [B][H][L][d]."""
    shape = (case.B, case.H, case.L, case.d)
    q = gaussian_bf16(shape, case.sigma_qk, seed, case.cfg_id, 0)
    k = gaussian_bf16(shape, case.sigma_qk, seed, case.cfg_id, 1)
    v = gaussian_bf16(shape, case.sigma_v, seed, case.cfg_id, 2)
    return q, k, v


def sample_rows(L: int, min_rows: int = 256, tile: int = 128, seed: int = 0) -> np.ndarray:
    """Stratified row sample: at least two rows from every `tile`-row block.

    In-block offsets cycle over 0..tile-1 so that every lane position is hit,
    and the block-boundary rows 0, tile-1, tile, L-tile, L-1 are always
    included.  Returns a sorted, duplicate-free int32 array; all rows when
    L <= min_rows.
    """
    if L <= min_rows:
        return np.arange(L, dtype=np.int32)
    n_blocks = (L + tile - 1) // tile
    per_block = max(2, -(-min_rows // n_blocks))
    rng = np.random.default_rng([seed, L, 977])
    start = int(rng.integers(0, tile))
    rows = {0, min(tile - 1, L - 1), min(tile, L - 1), max(L - tile, 0), L - 1}
    for b in range(n_blocks):
        width = min(tile, L - b * tile)
        first = (start + 37 * b) % width                 # cycles over the in-block positions
        others = rng.choice(width, size=min(width, per_block + 1), replace=False)
        picked = [first] + [int(o) for o in others if int(o) != first][: per_block - 1]
        rows.update(b * tile + off for off in picked)
    return np.array(sorted(rows), dtype=np.int32)
