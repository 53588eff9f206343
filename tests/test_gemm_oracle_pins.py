"""Pins of the matrix-product / softmax / unfused-attention oracle against things other than itself:
brute-force loops, closed forms, invariants, a library routine and the attention oracle."""
import math

import numpy as np
import pytest
import scipy.special

from oracle import attn_oracle as orc
from oracle import gemm_oracle as go
from paper_2609_10937_b200 import synth


def _bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


@pytest.mark.parametrize("M,N,K", [(3, 5, 7), (8, 8, 8), (1, 9, 4), (6, 1, 11)])
@pytest.mark.parametrize("layout", ["kn", "nk"])
def test_matmul_rows_equals_three_plain_loops(M, N, K, layout):
    rng = np.random.default_rng([M, N, K])
    a = _bits(rng.standard_normal((M, K)))
    b = _bits(rng.standard_normal((K, N) if layout == "kn" else (N, K)))
    ref = go.matmul_loops(a, b, M, N, K, layout)
    got = go.matmul_rows(a, b, M, N, K, np.arange(M), layout)
    assert np.abs(got - ref).max() <= 1e-13 * max(1.0, np.abs(ref).max())


def test_identity_ones_and_an_integer_closed_form():
    rng = np.random.default_rng(5)
    M, K = 12, 16
    a = _bits(rng.standard_normal((M, K)))
    eye = _bits(np.eye(K))
    assert np.array_equal(go.matmul_rows(a, eye, M, K, K, np.arange(M)), go.bf16_bits_to_f64(a).reshape(M, K))
    ones = _bits(np.ones((K, 3)))
    c = go.matmul_rows(a, ones, M, 3, K, np.arange(M))
    af = go.bf16_bits_to_f64(a).reshape(M, K)
    for i in range(M):
        assert c[i, 0] == pytest.approx(math.fsum(af[i].tolist()), abs=1e-14)
        assert c[i, 0] == c[i, 1] == c[i, 2]
    # A[i,k] = i, B[k,j] = j (small integers, exact in bf16)  =>  C[i,j] = K * i * j
    ai = _bits(np.repeat(np.arange(8, dtype=np.float32)[:, None], K, axis=1))
    bj = _bits(np.repeat(np.arange(6, dtype=np.float32)[None, :], K, axis=0))
    c = go.matmul_rows(ai, bj, 8, 6, K, np.arange(8))
    assert np.array_equal(c, K * np.outer(np.arange(8), np.arange(6)).astype(np.float64))
    # a transposed operand would not survive this one: A = e_2 e_5^T (single one at [2,5]) picks row 5 of B
    a1 = np.zeros((M, K), np.float32)
    a1[2, 5] = 1.0
    b = _bits(rng.standard_normal((K, 7)))
    c = go.matmul_rows(_bits(a1), b, M, 7, K, np.arange(M))
    assert np.array_equal(c[2], go.bf16_bits_to_f64(b).reshape(K, 7)[5]) and not c[[0, 1, 3]].any()


def test_the_two_storage_layouts_of_b_agree():
    rng = np.random.default_rng(6)
    M, N, K = 5, 9, 13
    a = _bits(rng.standard_normal((M, K)))
    b = rng.standard_normal((K, N)).astype(np.float32)
    c_kn = go.matmul_rows(a, _bits(b), M, N, K, np.arange(M), "kn")
    c_nk = go.matmul_rows(a, _bits(np.ascontiguousarray(b.T)), M, N, K, np.arange(M), "nk")
    assert np.array_equal(c_kn, c_nk)
    assert np.array_equal(go.matmul_rows(a, _bits(b), M, N, K, [3, 1], "kn"), c_kn[[3, 1]])


def test_bf16_rounding_helper_against_known_values():
    # ties go to the even mantissa: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6; representable values are kept
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 1.0 + 2.0 ** -7, 0.0])
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -6, -2.5, 1.0 + 2.0 ** -7, 0.0])
    assert np.array_equal(go.f64_to_bf16_f64(x), want)
    # agrees with the input generator's conversion on random values
    r = np.random.default_rng(7).standard_normal(1000).astype(np.float32)
    assert np.array_equal(go.f64_to_bf16_f64(r.astype(np.float64)), go.bf16_bits_to_f64(synth.f32_to_bf16_bits(r)))


def test_softmax_rows_invariants_and_library():
    rng = np.random.default_rng(8)
    s = rng.standard_normal((7, 33)) * 4.0
    p = go.softmax_rows(s, 0.5)
    assert np.abs(p.sum(axis=1) - 1.0).max() <= 1e-14 and (p > 0).all()
    assert np.abs(go.softmax_rows(s + 123.0, 0.5) - p).max() <= 1e-13          # shift invariance
    e = np.exp(0.5 * s)                                                         # no max subtraction (small values)
    assert np.abs(e / e.sum(axis=1, keepdims=True) - p).max() <= 1e-14
    assert np.abs(go.softmax_rows(np.zeros((2, 10)), 3.0) - 0.1).max() == 0.0
    assert np.abs(scipy.special.softmax(0.5 * s, axis=1) - p).max() <= 1e-15
    # the paper's running statistics: m is the row maximum, the denominator is sum exp(x - m)
    m = (0.5 * s).max(axis=1)
    d = np.exp(0.5 * s - m[:, None]).sum(axis=1)
    assert np.abs(np.exp(0.5 * s - m[:, None]) / d[:, None] - p).max() <= 1e-15


def test_unfused_path_agrees_with_the_attention_definition_up_to_its_bf16_roundings():
    L, d = 192, 64
    case = synth.AttnCase("pin", 1, 1, L, d)
    q, k, v = synth.make_qkv(case, seed=3)
    rows = np.arange(0, L, 5)
    u = go.unfused_attention_rows(q, k, v, L, d, rows)
    ref = orc.attention_rows(q, k, v, 1, 1, L, d, rows.astype(np.int32)).reshape(len(rows), d)
    err = np.abs(u["o"] - ref)
    # S and P each carry one bf16 rounding (2^-9 relative): a few 1e-3 on outputs of size ~0.1-1
    assert err.max() <= 2e-2 and np.linalg.norm(err) / np.linalg.norm(ref) <= 1e-2
    assert np.abs(u["p"].sum(axis=1) - 1.0).max() <= 2e-2
    # the first step is the plain product Q K^T, rounded once
    qf, kf = go.bf16_bits_to_f64(q).reshape(L, d), go.bf16_bits_to_f64(k).reshape(L, d)
    assert np.array_equal(u["s"], go.f64_to_bf16_f64(qf[rows] @ kf.T))
