"""TEST INFRASTRUCTURE, NOT PRODUCT CODE: fp64 CPU oracle for the dense matrix
product and for the unfused attention path built from it.

Only tests, the smoke check and the benchmark's CPU-baseline arm may import
this module. It imports nothing from the CUDA package.

* ``matmul_rows``   -- the definition C[i, j] = sum_k A[i, k] B[k, j] (the
  paper's Section "GEMM", C = A B) for chosen rows i, in fp64 over the
  bf16-rounded inputs; the sum over k is a numpy fp64 matrix product (a
  library routine used as one step, nothing blocked or reordered around it).
  ``b_layout`` says how B is stored: "kn" = [K][N] row-major (C = A B),
  "nk" = [N][K] row-major (C = A B^T, the layout of K in Q K^T).
* ``matmul_loops``  -- the same definition as three plain Python loops; tiny
  shapes only; it pins ``matmul_rows``.
* ``softmax_rows``  -- row softmax of scale * S with the running statistics
  of the paper's Section "Online Softmax": maximum m, denominator
  sum exp(s - m); evaluated directly (two passes) in fp64.
* ``unfused_attention_rows`` -- the three separate steps of the paper's
  unfused baseline (Section "Results": S = Q K^T materialised, row softmax,
  then P V), each rounded to the storage type the GPU path materialises
  (bf16 S and bf16 P), so that the GPU's unfused path can be compared step
  for step.

Parity of the paper's own numeric outputs: unpinned (the paper prints none
for these operators).
"""
from __future__ import annotations

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_f64(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to bf16 (nearest even, via fp32) and return them as fp64."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint32) << 16
    return rounded.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def matmul_rows(a_bits, b_bits, M: int, N: int, K: int, rows, b_layout: str = "kn") -> np.ndarray:
    """C[rows, :] of C = A B (b_layout "kn": B is [K][N]) or C = A B^T ("nk": B is [N][K]), fp64."""
    a = bf16_bits_to_f64(a_bits).reshape(M, K)
    if b_layout == "kn":
        b = bf16_bits_to_f64(b_bits).reshape(K, N)
    elif b_layout == "nk":
        b = bf16_bits_to_f64(b_bits).reshape(N, K).T
    else:
        raise ValueError(b_layout)
    rows = np.asarray(rows, dtype=np.int64)
    return a[rows, :] @ b


def matmul_loops(a_bits, b_bits, M: int, N: int, K: int, b_layout: str = "kn") -> np.ndarray:
    """The definition written out: three loops, fp64 accumulation in index order."""
    a = bf16_bits_to_f64(a_bits).reshape(M, K)
    b = bf16_bits_to_f64(b_bits).reshape((K, N) if b_layout == "kn" else (N, K))
    c = np.zeros((M, N), dtype=np.float64)
    for i in range(M):
        for j in range(N):
            acc = 0.0
            for k in range(K):
                acc += a[i, k] * (b[k, j] if b_layout == "kn" else b[j, k])
            c[i, j] = acc
    return c


def softmax_rows(s: np.ndarray, scale: float) -> np.ndarray:
    """Row softmax of scale * s in fp64: exp(x - m) / sum exp(x - m) with m the row maximum."""
    x = np.asarray(s, dtype=np.float64) * scale
    m = x.max(axis=-1, keepdims=True)
    e = np.exp(x - m)
    return e / e.sum(axis=-1, keepdims=True)


def unfused_attention_rows(q_bits, k_bits, v_bits, L: int, d: int, rows) -> dict:
    """One head of the unfused path for chosen query rows: S = Q K^T (stored as bf16), P = softmax(S / sqrt(d))
    (stored as bf16), O = P V.  Returns the three arrays in fp64 (S and P after their bf16 rounding)."""
    rows = np.asarray(rows, dtype=np.int64)
    s = f64_to_bf16_f64(matmul_rows(q_bits, k_bits, L, L, d, rows, "nk"))
    p = f64_to_bf16_f64(softmax_rows(s, 1.0 / np.sqrt(float(d))))
    v = bf16_bits_to_f64(v_bits).reshape(L, d)
    return {"s": s, "p": p, "o": p @ v}
