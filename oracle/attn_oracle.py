"""TEST INFRASTRUCTURE, NOT PRODUCT CODE: fp64 CPU oracle for fused attention.

Only tests, the smoke check and the benchmark's CPU-baseline / reference arm
may import this module. It imports nothing from the CUDA package.

Three independent statements of the same result live here:

* ``attention_rows``      -- ctypes front end of ``attn_oracle.c``: the plain
  definition (the paper's attention equation, Section "Fused Attention")
  evaluated row by row in fp64 with OpenMP over rows.
* ``attention_definition`` -- the same definition through library routines
  (``scipy.special.softmax`` and a numpy fp64 matmul); small shapes only.
* ``attention_streaming`` -- Algorithm 1 of the paper (one Q tile, K/V tiles
  streamed, running maximum ``m`` and denominator ``delta``) in fp64 with an
  arbitrary ``tile_kv`` (the last tile padded with -inf as the paper's
  boundary note requires) and ``merge_partials`` -- the associative merge
  operator of Section "Online Softmax" extended to carry the un-normalised
  output, applied in an arbitrary tree order.

Parity of the paper's own numeric outputs: unpinned (the paper prints none).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_LIB_PATH = _HERE / "libattn_oracle.so"
_SRC_PATH = _HERE / "attn_oracle.c"
_lib = None


def build(force: bool = False) -> Path:
    """Compile attn_oracle.c into libattn_oracle.so with gcc (-O2, OpenMP)."""
    if force or not _LIB_PATH.exists() or _LIB_PATH.stat().st_mtime < _SRC_PATH.stat().st_mtime:
        tmp = _LIB_PATH.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(tmp), str(_SRC_PATH), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB_PATH))
        lib.attn_oracle_rows.restype = ctypes.c_int
        lib.attn_oracle_rows.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 4 + [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        lib.attn_oracle_rows_causal.restype = ctypes.c_int
        lib.attn_oracle_rows_causal.argtypes = lib.attn_oracle_rows.argtypes
        lib.attn_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the C oracle will use."""
    return int(_load().attn_oracle_threads())


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def attention_rows(q_bits, k_bits, v_bits, B, H, L, d, rows, want_psum=False, causal=False):
    """Definition of attention for the given rows of every head (C, fp64).

    causal=True: row i attends to keys 0..i only (later keys have score -inf).

    q_bits, k_bits, v_bits: uint16 bf16 bit patterns, contiguous [B][H][L][d].
    rows: 1-D int array of row indices (same for every head).
    Returns fp64 [B*H, len(rows), d] (and the softmax row sums if asked).
    """
    lib = _load()
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    n = B * H * L * d
    if not (q_bits.size == k_bits.size == v_bits.size == n):
        raise ValueError("q/k/v sizes do not match B*H*L*d")
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    out = np.empty((B * H, rows.size, d), dtype=np.float64)
    psum = np.empty((B * H, rows.size), dtype=np.float64) if want_psum else None
    fn = lib.attn_oracle_rows_causal if causal else lib.attn_oracle_rows
    rc = fn(
        q_bits.ctypes.data, k_bits.ctypes.data, v_bits.ctypes.data, B, H, L, d,
        rows.ctypes.data, int(rows.size), out.ctypes.data,
        psum.ctypes.data if want_psum else None)
    if rc != 0:
        raise RuntimeError(f"attn_oracle_rows failed with code {rc}")
    return (out, psum) if want_psum else out


def attention_definition(q: np.ndarray, k: np.ndarray, v: np.ndarray, causal: bool = False) -> np.ndarray:
    """softmax(Q K^T / sqrt(d)) V for one head, fp64, via scipy + numpy.

    causal=True masks the scores of keys after the query's position with -inf."""
    from scipy.special import softmax

    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    s = (q @ k.T) * (1.0 / np.sqrt(np.float64(q.shape[1])))
    if causal:
        s = np.where(np.tril(np.ones(s.shape, dtype=bool)), s, -np.inf)
    return softmax(s, axis=1) @ v


def streaming_partial(q, k, v, tile_kv, kv_begin=0, kv_end=None):
    """Algorithm 1 over keys [kv_begin, kv_end): returns (m, delta, O_unnormalised).

    Follows the paper's loop: m <- -inf, delta <- 0, O <- 0; per tile
    S_t = Q K_t^T / sqrt(d); m_new = max(m, rowmax S_t); s = exp(m - m_new);
    E_t = exp(S_t - m_new); delta = delta*s + rowsum E_t; O = O*s + E_t V_t.
    A ragged last tile is padded to tile_kv with -inf scores (never zeros).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n_q, d = q.shape
    kv_end = k.shape[0] if kv_end is None else kv_end
    m = np.full(n_q, -np.inf)
    delta = np.zeros(n_q)
    o = np.zeros((n_q, d))
    inv = 1.0 / np.sqrt(np.float64(d))
    for t0 in range(kv_begin, kv_end, tile_kv):
        t1 = min(t0 + tile_kv, kv_end)
        s_t = np.full((n_q, tile_kv), -np.inf)
        s_t[:, : t1 - t0] = (q @ k[t0:t1].T) * inv
        v_t = np.zeros((tile_kv, d))
        v_t[: t1 - t0] = v[t0:t1]
        m_new = np.maximum(m, s_t.max(axis=1))
        with np.errstate(invalid="ignore"):
            corr = np.where(np.isneginf(m), 0.0, np.exp(m - m_new))
        e_t = np.exp(s_t - m_new[:, None])
        delta = delta * corr + e_t.sum(axis=1)
        o = o * corr[:, None] + e_t @ v_t
        m = m_new
    return m, delta, o


def merge_partials(a, b):
    """(m, delta, O)_a (+) (m, delta, O)_b -- the associative merge operator."""
    m_a, d_a, o_a = a
    m_b, d_b, o_b = b
    m_new = np.maximum(m_a, m_b)
    with np.errstate(invalid="ignore"):
        w_a = np.where(np.isneginf(m_a), 0.0, np.exp(m_a - m_new))
        w_b = np.where(np.isneginf(m_b), 0.0, np.exp(m_b - m_new))
    return m_new, d_a * w_a + d_b * w_b, o_a * w_a[:, None] + o_b * w_b[:, None]


def attention_streaming(q, k, v, tile_kv, splits=1, tree="left"):
    """Algorithm 1 + merge: split the keys into `splits` ranges, merge, normalise."""
    L = np.asarray(k).shape[0]
    bounds = [(L * i) // splits for i in range(splits + 1)]
    parts = [streaming_partial(q, k, v, tile_kv, bounds[i], bounds[i + 1])
             for i in range(splits) if bounds[i + 1] > bounds[i]]
    if tree == "left":
        acc = parts[0]
        for p in parts[1:]:
            acc = merge_partials(acc, p)
    elif tree == "right":
        acc = parts[-1]
        for p in reversed(parts[:-1]):
            acc = merge_partials(p, acc)
    else:  # balanced binary reduction
        while len(parts) > 1:
            nxt = [merge_partials(parts[i], parts[i + 1]) for i in range(0, len(parts) - 1, 2)]
            if len(parts) % 2:
                nxt.append(parts[-1])
            parts = nxt
        acc = parts[0]
    m, delta, o = acc
    return o / delta[:, None]
