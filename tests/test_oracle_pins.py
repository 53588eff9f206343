"""Pins for the fp64 oracle: closed forms, invariants, brute force, library routes.

None of these tests touches the CUDA path.  Each is chosen so that a plausible
slip in the oracle (dropped 1/sqrt(d), transposed operand, wrong normaliser,
wrong reduction axis, K/V swapped) makes at least one of them fail.
"""
import math

import numpy as np
import pytest

from oracle import attn_oracle as orc
from paper_2609_10937_b200 import synth


def _rand_bits(shape, sigma, seed, tid):
    return synth.gaussian_bf16(shape, sigma, seed, 900, tid)


def _f64(bits):
    return orc.bf16_bits_to_f64(bits)


def _rows(L):
    return np.arange(L, dtype=np.int32)


def test_bf16_widening_is_exact():
    vals = np.array([0.0, 1.0, -2.5, 0.0078125, 3.140625, -65280.0], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(vals)
    assert np.array_equal(_f64(bits), vals.astype(np.float64))
    # round-to-nearest-even at the halfway point: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6
    half = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    assert np.array_equal(_f64(synth.f32_to_bf16_bits(half)), [1.0, 1.0 + 2.0 ** -6])


def test_identical_v_rows_return_that_row():
    B, H, L, d = 1, 2, 96, 32
    q = _rand_bits((B, H, L, d), 1.0, 1, 0)
    k = _rand_bits((B, H, L, d), 1.0, 1, 1)
    row = _rand_bits((d,), 1.0, 1, 2)
    v = np.broadcast_to(row, (B, H, L, d)).copy()
    out = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))
    np.testing.assert_allclose(out, np.broadcast_to(_f64(row), out.shape), rtol=1e-14, atol=0)


@pytest.mark.parametrize("zero", ["q", "k"])
def test_zero_q_or_k_gives_column_mean_of_v(zero):
    B, H, L, d = 2, 1, 200, 16
    q = _rand_bits((B, H, L, d), 1.0, 2, 0)
    k = _rand_bits((B, H, L, d), 1.0, 2, 1)
    v = _rand_bits((B, H, L, d), 1.0, 2, 2)
    if zero == "q":
        q[:] = 0
    else:
        k[:] = 0
    out = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))
    vf = _f64(v).reshape(B * H, L, d)
    mean = np.array([[math.fsum(vf[b, :, c]) / L for c in range(d)] for b in range(B * H)])
    np.testing.assert_allclose(out, np.broadcast_to(mean[:, None, :], out.shape), rtol=0, atol=1e-13)


def test_softmax_rows_sum_to_one():
    B, H, L, d = 1, 3, 333, 64
    q, k, v = (_rand_bits((B, H, L, d), 2.0, 3, t) for t in range(3))
    _, psum = orc.attention_rows(q, k, v, B, H, L, d, _rows(L), want_psum=True)
    np.testing.assert_allclose(psum, 1.0, rtol=0, atol=1e-13)


@pytest.mark.parametrize("L,d", [(1, 8), (2, 8), (7, 4), (33, 16), (64, 64)])
def test_tiny_brute_force_without_max_shift(L, d):
    """Pure-Python exp/normalise with no max subtraction (the schematic form of
    the paper's per-tile equation) must agree on tiny inputs."""
    q, k, v = (_rand_bits((1, 1, L, d), 1.0, 4, t) for t in range(3))
    out = orc.attention_rows(q, k, v, 1, 1, L, d, _rows(L))[0]
    qf, kf, vf = (_f64(x).reshape(L, d) for x in (q, k, v))
    inv = 1.0 / math.sqrt(d)
    for i in range(L):
        w = [math.exp(inv * math.fsum(qf[i, c] * kf[j, c] for c in range(d))) for j in range(L)]
        den = math.fsum(w)
        for c in range(d):
            ref = math.fsum(w[j] * vf[j, c] for j in range(L)) / den
            assert out[i, c] == pytest.approx(ref, rel=1e-12, abs=1e-14)


def test_length_one_and_two_closed_forms():
    d = 16
    q, k, v = (_rand_bits((1, 1, 1, d), 1.0, 5, t) for t in range(3))
    out = orc.attention_rows(q, k, v, 1, 1, 1, d, _rows(1))
    assert np.array_equal(out[0, 0], _f64(v).reshape(d))
    q, k, v = (_rand_bits((1, 1, 2, d), 1.0, 6, t) for t in range(3))
    out = orc.attention_rows(q, k, v, 1, 1, 2, d, _rows(2))[0]
    qf, kf, vf = (_f64(x).reshape(2, d) for x in (q, k, v))
    for i in range(2):
        s = (qf[i] @ kf.T) / math.sqrt(d)
        w0 = 1.0 / (1.0 + math.exp(s[1] - s[0]))     # logistic of the score difference
        np.testing.assert_allclose(out[i], w0 * vf[0] + (1 - w0) * vf[1], rtol=1e-14, atol=1e-15)


def test_invariants_permutation_keyshift_linearity_hull():
    B, H, L, d = 1, 1, 150, 32
    q, k, v = (_rand_bits((B, H, L, d), 1.0, 7, t) for t in range(3))
    base = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))[0]
    # joint permutation of the (K, V) rows
    perm = np.random.default_rng(7).permutation(L)
    out = orc.attention_rows(q, k[:, :, perm], v[:, :, perm], B, H, L, d, _rows(L))[0]
    np.testing.assert_allclose(out, base, rtol=1e-12, atol=1e-14)
    # permuting K alone must change the result (catches an oracle that ignores K)
    out_k = orc.attention_rows(q, k[:, :, perm], v, B, H, L, d, _rows(L))[0]
    assert np.abs(out_k - base).max() > 1e-3
    # every output lies in the per-column hull of V
    vf = _f64(v).reshape(L, d)
    assert (base <= vf.max(axis=0) + 1e-12).all() and (base >= vf.min(axis=0) - 1e-12).all()
    # linear in V: V -> 2V (exact in bf16) doubles the output
    v2 = synth.f32_to_bf16_bits(2.0 * synth.bf16_bits_to_f32(v))
    out2 = orc.attention_rows(q, k, v2, B, H, L, d, _rows(L))[0]
    np.testing.assert_allclose(out2, 2.0 * base, rtol=1e-14, atol=0)
    # adding the same vector u to every key row shifts each score row by q.u: no effect.
    # Small integers keep k + u exactly representable in bf16.
    ki = np.random.default_rng(8).integers(-3, 4, size=(B, H, L, d)).astype(np.float32)
    u = np.random.default_rng(9).integers(-2, 3, size=(d,)).astype(np.float32)
    a = orc.attention_rows(q, synth.f32_to_bf16_bits(ki), v, B, H, L, d, _rows(L))[0]
    b = orc.attention_rows(q, synth.f32_to_bf16_bits(ki + u), v, B, H, L, d, _rows(L))[0]
    np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)


def test_structured_identity_layouts():
    """Structured cases in the spirit of the paper's fragment-layout test:
    Q = sqrt(d) I gives S = K^T, V = I gives O = the softmax matrix."""
    d = L = 16
    eye = np.eye(L, dtype=np.float32)
    qb = synth.f32_to_bf16_bits(4.0 * eye).reshape(1, 1, L, d)      # sqrt(16) = 4, exact
    k = _rand_bits((1, 1, L, d), 1.0, 10, 1)
    vb = synth.f32_to_bf16_bits(eye).reshape(1, 1, L, d)
    out = orc.attention_rows(qb, k, vb, 1, 1, L, d, _rows(L))[0]
    kf = _f64(k).reshape(L, d)
    s = kf.T                                                          # S[i, j] = K[j, i]
    p = np.exp(s - s.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(out, p, rtol=1e-13, atol=1e-15)
    assert np.abs(out - out.T).max() > 1e-3      # a transposed score matrix would be caught
    # one dominant key: the output row is that key's value row
    L2 = 40
    q = np.zeros((L2, d), np.float32)
    q[:, 0] = 64.0
    kk = np.zeros((L2, d), np.float32)
    kk[17, 0] = 64.0                                                  # logit 64*64/4 = 1024
    v = _rand_bits((1, 1, L2, d), 1.0, 11, 2)
    out = orc.attention_rows(synth.f32_to_bf16_bits(q).reshape(1, 1, L2, d),
                             synth.f32_to_bf16_bits(kk).reshape(1, 1, L2, d), v, 1, 1, L2, d, _rows(L2))[0]
    np.testing.assert_allclose(out, np.broadcast_to(_f64(v).reshape(L2, d)[17], out.shape), rtol=0, atol=1e-15)


@pytest.mark.parametrize("B,H,L,d,sigma", [(1, 1, 256, 64, 1.0), (2, 3, 320, 128, math.sqrt(3.0))])
def test_c_oracle_matches_library_definition(B, H, L, d, sigma):
    q = _rand_bits((B, H, L, d), sigma, 12, 0)
    k = _rand_bits((B, H, L, d), sigma, 12, 1)
    v = _rand_bits((B, H, L, d), 1.0, 12, 2)
    out = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))
    qf, kf, vf = (_f64(x).reshape(B * H, L, d) for x in (q, k, v))
    for bh in range(B * H):
        ref = orc.attention_definition(qf[bh], kf[bh], vf[bh])
        np.testing.assert_allclose(out[bh], ref, rtol=1e-12, atol=1e-14)
    # heads must not be mixed up: head 0 of the batch differs from head 1
    if B * H > 1:
        assert np.abs(out[0] - out[1]).max() > 1e-3


def test_c_oracle_matches_torch_fp64():
    import torch

    B, H, L, d = 1, 2, 192, 64
    q, k, v = (_rand_bits((B, H, L, d), 1.0, 13, t) for t in range(3))
    out = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))
    tq, tk, tv = (torch.from_numpy(_f64(x).reshape(B * H, L, d)) for x in (q, k, v))
    ref = torch.softmax(tq @ tk.transpose(1, 2) / math.sqrt(d), dim=-1) @ tv
    np.testing.assert_allclose(out, ref.numpy(), rtol=1e-12, atol=1e-14)


def test_row_subset_matches_full():
    B, H, L, d = 1, 2, 300, 32
    q, k, v = (_rand_bits((B, H, L, d), 1.0, 14, t) for t in range(3))
    full = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))
    rows = np.array([0, 5, 127, 128, 299], dtype=np.int32)
    sub = orc.attention_rows(q, k, v, B, H, L, d, rows)
    assert np.array_equal(sub, full[:, rows])


@pytest.mark.parametrize("tile_kv", [16, 64, 100, 128])
@pytest.mark.parametrize("splits,tree", [(1, "left"), (3, "left"), (3, "right"), (5, "tree")])
def test_streaming_algorithm_and_merge_equal_the_definition(tile_kv, splits, tree):
    """Algorithm 1 with any KV tile (ragged tail padded with -inf) and the merge
    operator in any tree order reproduce the definition."""
    L, d = 330, 32
    q, k, v = (_f64(_rand_bits((L, d), math.sqrt(3.0), 15, t)) for t in range(3))
    ref = orc.attention_definition(q, k, v)
    got = orc.attention_streaming(q, k, v, tile_kv, splits=splits, tree=tree)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)


def test_zero_padding_would_be_wrong():
    """The paper's boundary note: padding a ragged tile with zero scores adds
    spurious weight.  The -inf padding used by the streaming routine does not."""
    L, d, tile = 100, 16, 64
    q, k, v = (_f64(_rand_bits((L, d), 1.0, 16, t)) for t in range(3))
    ref = orc.attention_definition(q, k, v)
    kz = np.vstack([k, np.zeros((28, d))])
    vz = np.vstack([v, np.zeros((28, d))])
    bad = orc.attention_definition(q, kz, vz)          # zero-padded keys take part
    assert np.abs(bad - ref).max() > 1e-3
    good = orc.attention_streaming(q, k, v, tile)
    np.testing.assert_allclose(good, ref, rtol=1e-12, atol=1e-14)


def test_sample_rows_properties():
    for L in (256, 1024, 4096, 32768):
        rows = synth.sample_rows(L)
        assert len(np.unique(rows)) == len(rows) and rows.min() >= 0 and rows.max() < L
        if L > 256:
            assert len(rows) >= 256
            counts = np.bincount(rows // 128, minlength=L // 128)
            assert counts.min() >= 2
            for r in (0, 127, 128, L - 128, L - 1):
                assert r in rows


# ----------------------------------------------------------------------------- causal variant
def test_causal_row_equals_noncausal_attention_over_its_prefix():
    """Brute force through the already pinned non-causal oracle: row i of the causal result is the
    last row of plain attention over the first i+1 keys and values."""
    B, H, L, d = 1, 2, 70, 16
    q, k, v = (_rand_bits((B, H, L, d), 1.5, 21, t) for t in range(3))
    got = orc.attention_rows(q, k, v, B, H, L, d, _rows(L), causal=True)
    for i in (0, 1, 2, 31, 32, 63, 64, 69):
        ref = orc.attention_rows(q[:, :, : i + 1].copy(), k[:, :, : i + 1].copy(), v[:, :, : i + 1].copy(),
                                 B, H, i + 1, d, np.array([i], dtype=np.int32))
        np.testing.assert_allclose(got[:, i], ref[:, 0], rtol=1e-13, atol=1e-15)
    # row 0 sees one key only: the output is V[0] exactly
    assert np.array_equal(got[:, 0], _f64(v).reshape(B * H, L, d)[:, 0])


def test_causal_rows_ignore_later_keys_and_values():
    B, H, L, d = 1, 1, 50, 8
    q, k, v = (_rand_bits((B, H, L, d), 1.0, 22, t) for t in range(3))
    base = orc.attention_rows(q, k, v, B, H, L, d, _rows(L), causal=True)[0]
    k2, v2 = k.copy(), v.copy()
    k2[:, :, 30:] = _rand_bits((B, H, 20, d), 3.0, 23, 1)
    v2[:, :, 30:] = _rand_bits((B, H, 20, d), 3.0, 23, 2)
    out = orc.attention_rows(q, k2, v2, B, H, L, d, _rows(L), causal=True)[0]
    assert np.array_equal(out[:30], base[:30])            # rows before the change are untouched
    assert np.abs(out[30:] - base[30:]).max() > 1e-3      # rows that can see it do change
    # and the causal result differs from the non-causal one (a mask that does nothing would be caught)
    full = orc.attention_rows(q, k, v, B, H, L, d, _rows(L))[0]
    assert np.abs(full[:-1] - base[:-1]).max() > 1e-3
    np.testing.assert_allclose(full[-1], base[-1], rtol=1e-13)   # the last row sees every key either way


def test_causal_c_oracle_matches_library_definition():
    B, H, L, d = 2, 2, 200, 64
    q, k, v = (_rand_bits((B, H, L, d), math.sqrt(3.0), 24, t) for t in range(3))
    out, psum = orc.attention_rows(q, k, v, B, H, L, d, _rows(L), want_psum=True, causal=True)
    np.testing.assert_allclose(psum, 1.0, rtol=0, atol=1e-13)
    qf, kf, vf = (_f64(x).reshape(B * H, L, d) for x in (q, k, v))
    for bh in range(B * H):
        np.testing.assert_allclose(out[bh], orc.attention_definition(qf[bh], kf[bh], vf[bh], causal=True),
                                   rtol=1e-12, atol=1e-14)
