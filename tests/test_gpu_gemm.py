"""GPU parity of the unfused path (matrix product, row softmax, three-kernel attention) against the fp64 oracle."""
import math

import numpy as np
import pytest

from paper_2609_10937_b200 import synth
from tests.gpu_util import to_cuda_bf16, to_host_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch

    from oracle import gemm_oracle as go
    from paper_2609_10937_b200 import binding, build

    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    build.build()
    binding.lib()
    return torch, go, binding


def _rand_bits(rng, shape, sigma=1.0):
    return synth.f32_to_bf16_bits((rng.standard_normal(shape) * sigma).astype(np.float32))


def _check_product(env, batch, M, N, K, layout, seed, rows_per_batch=None, **tiles):
    torch, go, binding = env
    rng = np.random.default_rng([seed, M, N, K])
    a = _rand_bits(rng, (batch, M, K))
    b = _rand_bits(rng, (batch, K, N) if layout == "kn" else (batch, N, K))
    c = binding.gemm(to_cuda_bf16(a), to_cuda_bf16(b), b_layout=layout, **tiles)
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    got = to_host_f64(c).reshape(batch, M, N)
    for bi in range(batch):
        rows = np.arange(M) if rows_per_batch is None or rows_per_batch >= M else \
            np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, rows_per_batch)]))
        ref = go.matmul_rows(a[bi], b[bi], M, N, K, rows, layout)
        # fp32 accumulation of K products of size ~1, then one bf16 rounding of a value of size ~sqrt(K)
        tol = 2.0 ** -8 * np.maximum(np.abs(ref), 1.0) + 1e-5 * math.sqrt(K)
        err = np.abs(got[bi][rows] - ref)
        assert (err <= tol).all(), (layout, batch, M, N, K, float(err.max()), float(np.abs(ref).max()))


@pytest.mark.parametrize("layout", ["kn", "nk"])
@pytest.mark.parametrize("batch,M,N,K", [
    (1, 256, 256, 64), (1, 256, 256, 256), (1, 512, 768, 192), (2, 384, 520, 136), (1, 1, 8, 8), (3, 130, 264, 72),
    (1, 1000, 1000, 1000), (1, 2048, 128, 2048)])
def test_matrix_product_matches_oracle(env, layout, batch, M, N, K):
    _check_product(env, batch, M, N, K, layout, seed=1)


@pytest.mark.parametrize("layout", ["kn", "nk"])
@pytest.mark.parametrize("batch,M,N,K", [
    (1, 512, 512, 256), (1, 520, 264, 264), (2, 300, 1000, 328), (1, 129, 136, 256), (1, 4096, 768, 320), (5, 257, 257 + 7, 1024),
    (1, 2560, 2304, 256), (1, 4000, 4096 - 56, 264), (1, 1280, 4096 - 8, 1096),
    (1, 512, 520, 64), (2, 300, 1000, 72), (1, 2560, 2304, 128), (1, 384, 264, 8), (1, 8192, 8200, 64)])
def test_cta_pairs_and_lone_ctas_agree_with_the_oracle_and_each_other(env, layout, batch, M, N, K):
    """The two tilings of the same product: CTA pairs (one matrix instruction over two CTAs, two accumulators in tensor
    memory, per-warp stores) and lone CTAs.  Ragged M, N and K, several tiles per pair (more than the accumulators,
    so that buffers are reused), batches, and shapes whose last wave runs as half-width work items (the last two: 256 and
    80 tiles on 74 pairs leave 34 and 6), one or two ring stages of products per tile, and an output larger than the
    cache (the last: its stores carry an eviction priority).  All sum the K products of an element in the same order:
    same bits."""
    torch, go, binding = env
    desc = binding.hw_desc_query(0)
    assert binding.gemm_plan(desc, batch, M, N, K).cta_pair == 2
    if M >= 1280 and N > 4000:
        assert binding.gemm_plan(desc, batch, M, N, K).tail_split > 0
    _check_product(env, batch, M, N, K, layout, seed=4, rows_per_batch=300)                 # closed-form default: pairs
    _check_product(env, batch, M, N, K, layout, seed=4, rows_per_batch=300, cta_pair=1)
    _check_product(env, batch, M, N, K, layout, seed=4, rows_per_batch=300, cta_pair=2, tile_n=128)
    _check_product(env, batch, M, N, K, layout, seed=4, rows_per_batch=300, tail_split=-1)   # whole tiles in the last wave
    rng = np.random.default_rng([9, M, N, K])
    a = to_cuda_bf16(_rand_bits(rng, (batch, M, K)))
    b = to_cuda_bf16(_rand_bits(rng, (batch, K, N) if layout == "kn" else (batch, N, K)))
    pair, lone = binding.gemm(a, b, b_layout=layout), binding.gemm(a, b, b_layout=layout, cta_pair=1)
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    assert torch.equal(pair.view(torch.int16), lone.view(torch.int16))


@pytest.mark.parametrize("layout", ["kn", "nk"])
def test_structured_products(env, layout):
    """Identity, a single one, and an index pattern: operand order and the two storage layouts of B."""
    torch, go, binding = env
    M = N = K = 320
    rng = np.random.default_rng(4)
    a = _rand_bits(rng, (M, K))
    eye = synth.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    c = to_host_f64(binding.gemm(to_cuda_bf16(a), to_cuda_bf16(eye), b_layout=layout)).reshape(M, N)
    assert np.array_equal(c, go.bf16_bits_to_f64(a).reshape(M, K))
    # B[k][j] (as a matrix, whatever its storage) = 1 if k == 2 j' pattern: picks columns of A
    bm = np.zeros((K, N), np.float32)
    bm[(np.arange(N) * 7) % K, np.arange(N)] = 1.0
    b_store = bm if layout == "kn" else np.ascontiguousarray(bm.T)
    c = to_host_f64(binding.gemm(to_cuda_bf16(a), to_cuda_bf16(synth.f32_to_bf16_bits(b_store)), b_layout=layout)).reshape(M, N)
    assert np.array_equal(c, go.bf16_bits_to_f64(a).reshape(M, K)[:, (np.arange(N) * 7) % K])
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0


def test_matrix_product_full_size_sampled(env):
    """The paper's 4096^3 shape, rows sampled."""
    _check_product(env, 1, 4096, 4096, 4096, "kn", seed=2, rows_per_batch=48)


@pytest.mark.parametrize("rows,cols", [(4, 8), (7, 256), (33, 2048), (5, 2056), (3, 16384), (2, 32768), (9, 1000),
                                       (3, 16392), (2, 20000), (5, 32760)])   # the last three: staged in shared memory
def test_row_softmax_matches_oracle(env, rows, cols):
    torch, go, binding = env
    rng = np.random.default_rng([rows, cols])
    s = _rand_bits(rng, (rows, cols), sigma=6.0)
    scale = 0.37
    ref = go.softmax_rows(go.bf16_bits_to_f64(s).reshape(rows, cols), scale)
    st = to_cuda_bf16(s)
    p = binding.softmax_rows(st, scale)
    got = to_host_f64(p).reshape(rows, cols)
    assert np.abs(got - ref).max() <= 2.0 ** -8 * ref.max() + 1e-6
    assert np.abs(got.sum(axis=1) - 1.0).max() <= 1e-2
    p2 = binding.softmax_rows(st, scale, out=st)                 # in place
    assert torch.equal(p2, p)


@pytest.mark.parametrize("B,H,L,d", [(1, 1, 256, 64), (1, 2, 1024, 128), (2, 2, 520, 64), (1, 1, 4096, 128), (1, 1, 16384, 128)])
def test_unfused_attention_matches_its_oracle_and_the_fused_kernel(env, B, H, L, d):
    torch, go, binding = env
    from oracle import attn_oracle as orc

    case = synth.AttnCase("unfused", B, H, L, d)
    q, k, v = synth.make_qkv(case, seed=5)
    tq, tk, tv = (to_cuda_bf16(x) for x in (q, k, v))
    scores = torch.empty(B * H * L * L, dtype=torch.bfloat16, device="cuda")
    o = binding.forward_unfused(tq, tk, tv, scores)
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    got = to_host_f64(o).reshape(B * H, L, d)
    rows = np.unique(np.concatenate([[0, L - 1], np.random.default_rng(L).integers(0, L, 40)]))
    qh, kh, vh = (x.reshape(B * H, L, d) for x in (q, k, v))
    for bh in range(B * H):
        u = go.unfused_attention_rows(qh[bh], kh[bh], vh[bh], L, d, rows)
        err = np.abs(got[bh][rows] - u["o"])
        # same three steps and the same two bf16 roundings; what remains is fp32 accumulation, exp2 and the
        # final bf16 rounding of the output
        assert err.max() <= 1e-2 and np.linalg.norm(err) / np.linalg.norm(u["o"]) <= 5e-3
    # and the definition itself (the fused kernel's oracle), at the looser bound the two extra roundings cost
    ref = orc.attention_rows(q, k, v, B, H, L, d, rows.astype(np.int32)).reshape(B * H, len(rows), d)
    assert np.abs(got[:, rows] - ref).max() <= 3e-2


def test_unfused_entry_points_refuse_bad_arguments(env):
    torch, _, binding = env
    a = torch.zeros(64, 72, dtype=torch.bfloat16, device="cuda")
    b = torch.zeros(72, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.AttnError) as err:                       # K = 70 is not a multiple of 8
        binding.gemm(a[:, :70].contiguous(), b[:70].contiguous())
    assert err.value.code == -2
    with pytest.raises(binding.AttnError) as err:                       # c overlaps a
        L = binding.lib()
        rc = L.gemm_forward(a.data_ptr(), b.data_ptr(), a.data_ptr(), 1, 64, 64, 72, 0, None)
        binding._check(rc, "gemm_forward")
    assert err.value.code == -4
    flat = torch.zeros(64 * 72 + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.AttnError) as err:                       # pointer not 16-byte aligned
        rc = binding.lib().gemm_forward(flat.data_ptr() + 2, b.data_ptr(), torch.empty(64, 64, dtype=torch.bfloat16, device="cuda").data_ptr(),
                                        1, 64, 64, 72, 0, None)
        binding._check(rc, "gemm_forward")
    assert err.value.code == -3
    s = torch.zeros(4, 100, dtype=torch.bfloat16, device="cuda")        # 100 columns: not a multiple of 8
    with pytest.raises(binding.AttnError) as err:
        binding.softmax_rows(s, 1.0)
    assert err.value.code == -2
    ok = torch.zeros(4, 128, dtype=torch.bfloat16, device="cuda")
    for bad_scale in (0.0, -0.5, float("inf"), float("nan")):           # the row maximum is taken before scaling
        with pytest.raises(binding.AttnError) as err:
            binding.softmax_rows(ok, bad_scale)
        assert err.value.code == -1
    q = torch.zeros(1, 1, 256, 64, dtype=torch.bfloat16, device="cuda")
    small = torch.empty(10, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.AttnError) as err:                       # score buffer too small
        binding.forward_unfused(q, q.clone(), q.clone(), small)
    assert err.value.code == -1
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
