"""GPU parity tests: the CUDA path (through the C ABI) against the fp64 oracle.

Tolerance (stated by the build target): fp32 accumulation, max-abs error <= 1e-2
and relative L2 <= 5e-3 on bf16 outputs.  Small cases are compared element by
element on every row; full-size cases on a stratified sample of >= 256 rows per
head (at least two rows in every 128-row block) plus whole-output properties.
"""
import math

import numpy as np
import pytest

from paper_2609_10937_b200 import synth
from tests.gpu_util import assert_close, errors, to_cuda_bf16, to_host_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from oracle import attn_oracle as orc
    from paper_2609_10937_b200 import binding

    binding.lib()   # must load: there is no fallback
    return torch, orc, binding


def _case(name, B, H, L, d, sigma_qk=1.0, cfg_id=50):
    return synth.AttnCase(name, B, H, L, d, sigma_qk=sigma_qk, cfg_id=cfg_id)


def _run_and_compare(env, case, runner, rows=None, what="", causal=False):
    torch, orc, binding = env
    q, k, v = synth.make_qkv(case, seed=0)
    tq, tk, tv = (to_cuda_bf16(x) for x in (q, k, v))
    out = runner(tq, tk, tv)
    torch.cuda.synchronize()
    code, detail = binding.last_device_status()
    assert code == 0, f"{what}: device status {code} detail {detail}"
    got = to_host_f64(out).reshape(case.B * case.H, case.L, case.d)
    rows = np.arange(case.L, dtype=np.int32) if rows is None else rows
    ref = orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, rows, causal=causal)
    stats = assert_close(got[:, rows], ref, what or case.name)
    # whole-output properties that hold at any size: finite, inside the per-column hull of V
    vf = to_host_f64(tv).reshape(case.B * case.H, case.L, case.d)
    assert np.isfinite(got).all()
    assert (got <= vf.max(axis=1, keepdims=True) + 1e-2).all() and (got >= vf.min(axis=1, keepdims=True) - 1e-2).all()
    return got, stats


# ------------------------------------------------------------ layout / structured
@pytest.mark.parametrize("d,tile_kv", [(128, 128), (128, 64), (64, 128), (64, 64)])
def test_score_tile_layout(env, d, tile_kv):
    """Raw S = Q_0 K_0^T read back from tensor memory must equal the fp64 product:
    catches a wrong shared-memory descriptor, swizzle or tensor-memory lane mapping."""
    torch, orc, binding = env
    case = _case("scores", 1, 1, 256, d)
    q, k, v = synth.make_qkv(case, seed=1)
    s_out = torch.zeros(128 * tile_kv, dtype=torch.float32, device="cuda")
    binding.forward_simple(*(to_cuda_bf16(x) for x in (q, k, v)), tile_kv=tile_kv, scores_out=s_out)
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    qf = orc.bf16_bits_to_f64(q).reshape(256, d)
    kf = orc.bf16_bits_to_f64(k).reshape(256, d)
    ref = qf[:128] @ kf[:tile_kv].T
    got = s_out.cpu().numpy().reshape(128, tile_kv).astype(np.float64)
    assert np.abs(got - ref).max() <= 1e-4 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("variant", ["simple", "pipelined"])
@pytest.mark.parametrize("d", [64, 128])
def test_structured_inputs(env, variant, d):
    """Structured cases in the spirit of the paper's fragment-layout test."""
    torch, orc, binding = env
    L = 256
    run = (lambda a, b, c: binding.forward_simple(a, b, c)) if variant == "simple" else binding.forward
    rng = np.random.default_rng(3)
    rnd = lambda: synth.f32_to_bf16_bits(rng.standard_normal((1, 1, L, d), dtype=np.float32))
    # (a) identical V rows -> every output row is that row (exactly representable)
    row = synth.f32_to_bf16_bits(rng.standard_normal(d, dtype=np.float32))
    v = np.broadcast_to(row, (1, 1, L, d)).copy()
    out = to_host_f64(run(to_cuda_bf16(rnd()), to_cuda_bf16(rnd()), to_cuda_bf16(v))).reshape(L, d)
    assert np.abs(out - orc.bf16_bits_to_f64(row)).max() <= 1e-2
    # (b) Q = 0 -> column mean of V
    vb = rnd()
    out = to_host_f64(run(to_cuda_bf16(np.zeros((1, 1, L, d), np.uint16)), to_cuda_bf16(rnd()), to_cuda_bf16(vb)))
    mean = orc.bf16_bits_to_f64(vb).reshape(L, d).mean(axis=0)
    assert np.abs(out.reshape(L, d) - mean).max() <= 1e-2
    # (c) V carries the key index in column 0 and a column-dependent pattern: checks the
    #     key-axis and column-axis ordering of the second product against the oracle
    vf = np.zeros((L, d), np.float32)
    vf[:, 0] = np.arange(L) / 32.0
    vf[:, 1:] = (np.arange(L)[:, None] % 7) * 0.25 + (np.arange(1, d)[None, :] % 5) * 0.5
    qb, kb, vb = rnd(), rnd(), synth.f32_to_bf16_bits(vf).reshape(1, 1, L, d)
    out = to_host_f64(run(to_cuda_bf16(qb), to_cuda_bf16(kb), to_cuda_bf16(vb))).reshape(1, L, d)
    ref = orc.attention_rows(qb, kb, vb, 1, 1, L, d, np.arange(L, dtype=np.int32))
    assert_close(out, ref, "structured V")
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0


# ---------------------------------------------------------------- small, every row
@pytest.mark.parametrize("B,H,L,d,tile_kv", [(1, 1, 128, 128, 128), (1, 1, 256, 64, 128), (2, 3, 384, 128, 64),
                                             (1, 2, 640, 64, 64), (1, 1, 1024, 128, 128)])
def test_simple_kernel_matches_oracle(env, B, H, L, d, tile_kv):
    _, _, binding = env
    _run_and_compare(env, _case("simple", B, H, L, d), lambda a, b, c: binding.forward_simple(a, b, c, tile_kv=tile_kv))


@pytest.mark.parametrize("B,H,L,d", [(1, 1, 128, 128), (1, 1, 256, 64), (1, 1, 384, 128), (2, 3, 640, 128),
                                     (1, 5, 1152, 64), (3, 2, 1024, 128)])
def test_pipelined_kernel_matches_oracle_small(env, B, H, L, d):
    """Several tiles, an odd number of 128-row blocks (one sub-tile of the last CTA idle),
    sequences shorter than the K/V ring."""
    _, _, binding = env
    _run_and_compare(env, _case("small", B, H, L, d), binding.forward)


@pytest.mark.parametrize("d,n_q,kv_splits,L,cluster", [
    (128, 2, 2, 2100, 2),     # two parts: landing in the Q buffer, ready one step before the end; ragged L
    (128, 2, 3, 1408, 3),     # three and four parts: landing in the K/V ring
    (128, 2, 4, 2048, 4),
    (128, 2, 5, 2560, 0),     # five parts of a two-sub-tile CTA do not fit the ring: through the workspace
    (64, 2, 2, 1408, 2), (64, 2, 3, 1500, 3), (64, 2, 4, 2048, 4),
    (64, 2, 5, 1280, 5), (64, 2, 8, 1024, 8),      # half the bytes per part at d = 64: up to eight parts fit the ring
    (128, 1, 2, 1408, 2), (128, 1, 4, 1408, 4), (64, 1, 3, 777, 3),
    (128, 1, 5, -1408, 5), (64, 1, 8, -1100, 8)])  # (one head) more CTAs than 32-row groups: the last ranks only publish
def test_uniform_split_through_clusters(env, d, n_q, kv_splits, L, cluster):
    """Uniform key splits: the CTAs of a Q tile run as one thread-block cluster and exchange their partial results
    through distributed shared memory where the landing areas fit; the result is the oracle's either way, the
    same bits run to run, and the same bits as with one CTA per tile merged nowhere (up to the merge's rounding)."""
    torch, _, binding = env
    case = _case("cluster", 1, 3 if L > 0 else 1, abs(L), d, sigma_qk=math.sqrt(3.0))
    seen = []

    def run(a, b, c):
        o = binding.forward_tiles(a, b, c, n_q=n_q, kv_splits=kv_splits)
        seen.append(binding.last_cluster_size())
        return o

    _run_and_compare(env, case, run)
    # (a device with fewer resident clusters of that size than this problem has tiles goes through the workspace)
    tiles = case.B * case.H * -(-case.L // (128 * n_q))
    resident = list(binding.hw_desc_query(0).max_clusters)
    assert seen == [cluster if cluster == 0 or resident[cluster - 1] >= tiles else 0]
    q, k, v = (to_cuda_bf16(x) for x in synth.make_qkv(case, seed=0))
    o1 = binding.forward_tiles(q, k, v, n_q=n_q, kv_splits=kv_splits)
    o2 = binding.forward_tiles(q, k, v, n_q=n_q, kv_splits=kv_splits)
    whole = binding.forward_tiles(q, k, v, n_q=n_q, kv_splits=1)
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    assert float((o1.float() - whole.float()).abs().max()) <= 2e-2


def _device_desc_dict(binding):
    d = binding.hw_desc_query(0)
    return {n: (list(getattr(d, n)) if n == "max_clusters" else getattr(d, n)) for n, _ in d._fields_}


@pytest.mark.parametrize("B,H,L,d,clustered", [
    (1, 4, 1024, 128, True), (1, 1, 2048, 128, True), (1, 1, 4096, 128, True), (1, 3, 3000, 128, True), (1, 2, 8192, 128, True),
    (1, 7, 1024, 64, True), (1, 1, 2048, 64, True), (2, 3, 1500, 64, True), (1, 1, 520, 128, False), (1, 12, 1100, 128, True),
    (1, 5, 333, 128, False)])
def test_default_plan_of_under_occupied_shapes(env, B, H, L, d, clustered):
    """Fewer Q tiles than SMs: the closed-form plan picks k CTAs per tile as one cluster (k from this device's
    resident-cluster counts: the plan oracle's restatement on the queried descriptor); the launch follows it."""
    torch, _, binding = env
    from oracle import plan_oracle as po

    t = binding.plan(binding.hw_desc_query(0), B, H, L, d)
    want = po.derive_tiles_tmem_machine(_device_desc_dict(binding), B, H, L, d)
    assert t.tiles < 148 and (t.tiles, t.ctas) == (want["tiles"], want["ctas"]) and t.ctas % t.tiles == 0
    k = t.ctas // t.tiles
    assert (k >= 2) == clustered
    rows = None if L <= 2048 else np.unique(np.concatenate([[0, L - 1], np.random.default_rng(L).integers(0, L, 96)])).astype(np.int32)
    _run_and_compare(env, _case("under", B, H, L, d, sigma_qk=math.sqrt(3.0)), binding.forward, rows=rows)
    assert binding.last_cluster_size() == (k if k > 1 else 0)


@pytest.mark.parametrize("n_q,tile_kv,kv_stages,kv_splits", [
    (2, 128, 0, 1), (2, 128, 2, 1), (2, 128, 3, 3), (2, 64, 0, 1), (2, 64, 4, 5),
    (1, 128, 0, 1), (1, 64, 0, 2), (1, 128, 3, 7)])
@pytest.mark.parametrize("d", [64, 128])
def test_tile_variants_match_oracle(env, d, n_q, tile_kv, kv_stages, kv_splits):
    """Every compiled tile variant, ring depth and key split (uneven splits included)."""
    _, _, binding = env
    run = lambda a, b, c: binding.forward_tiles(a, b, c, n_q=n_q, tile_kv=tile_kv, kv_stages=kv_stages,
                                                kv_splits=kv_splits)
    _run_and_compare(env, _case("variant", 1, 2, 1408, d, sigma_qk=math.sqrt(3.0)), run)


@pytest.mark.parametrize("L", [1, 2, 17, 64, 100, 127, 129, 200, 255, 257, 333, 1000, 1111, 2049])
@pytest.mark.parametrize("d", [64, 128])
def test_ragged_sequence_lengths(env, d, L):
    """Any L >= 1: the last key tile is ragged (its out-of-range scores are -inf, never zero-padded,
    as the paper's boundary note requires) and the last Q tile is clipped."""
    _, _, binding = env
    case = _case("ragged", 1, 3, L, d, sigma_qk=1.5)
    _run_and_compare(env, case, binding.forward)
    _run_and_compare(env, case, lambda a, b, c: binding.forward_simple(a, b, c, tile_kv=64))


@pytest.mark.parametrize("kw", [dict(tile_kv=64), dict(n_q=1), dict(kv_splits=3), dict(ctas=23), dict(n_q=1, tile_kv=64, ctas=41)])
def test_ragged_length_with_tile_variants_and_key_splits(env, kw):
    _, _, binding = env
    case = _case("ragged_variants", 2, 2, 1100, 128, sigma_qk=math.sqrt(3.0))
    _run_and_compare(env, case, lambda a, b, c: binding.forward_tiles(a, b, c, **kw))


def test_zero_padding_would_show(env):
    """A kernel that treated the zero-filled keys of a ragged tile as real keys would pull every output
    toward zero-weighted garbage: with all true scores very negative the padded keys would dominate."""
    torch, orc, binding = env
    L, d = 130, 64
    rng = np.random.default_rng(11)
    q = np.full((1, 1, L, d), 4.0, np.float32)
    k = np.full((1, 1, L, d), -4.0, np.float32)          # every true score is -16*64/8 = -128
    v = rng.standard_normal((1, 1, L, d), dtype=np.float32) + 3.0
    qb, kb, vb = (synth.f32_to_bf16_bits(x) for x in (q, k, v))
    out = to_host_f64(binding.forward(to_cuda_bf16(qb), to_cuda_bf16(kb), to_cuda_bf16(vb))).reshape(1, L, d)
    ref = orc.attention_rows(qb, kb, vb, 1, 1, L, d, np.arange(L, dtype=np.int32))
    assert_close(out, ref, "zero padding")
    assert np.abs(ref).mean() > 2.0        # the correct answer is the mean of V (~3), not ~0


@pytest.mark.parametrize("ctas", [1, 3, 5, 12, 13, 17, 29, 64, 131])
@pytest.mark.parametrize("d,n_q,tile_kv", [(128, 2, 128), (64, 2, 128), (128, 1, 64)])
def test_balanced_key_ranges_any_grid_size(env, d, n_q, tile_kv, ctas):
    """Grid sizes that cut the (Q tile, KV step) line at arbitrary places: ranges that straddle tile
    boundaries (several segments per CTA, whole tiles in the middle), tiles shared by two to many CTAs,
    tiles owned by a single CTA, one CTA doing everything."""
    _, _, binding = env
    case = _case("ranges", 1, 2, 1408, d, sigma_qk=math.sqrt(3.0))
    run = lambda a, b, c: binding.forward_tiles(a, b, c, n_q=n_q, tile_kv=tile_kv, ctas=ctas)
    _run_and_compare(env, case, run)


# --------------------------------------------------------------------------- causal
@pytest.mark.parametrize("L", [1, 3, 64, 128, 129, 200, 256, 257, 640, 1000, 1408, 2049])
@pytest.mark.parametrize("d", [64, 128])
def test_causal_matches_oracle(env, d, L):
    """Row i attends to keys 0..i: diagonal tiles masked with -inf, key steps after a Q tile skipped."""
    _, _, binding = env
    case = _case("causal", 1, 3, L, d, sigma_qk=1.5)
    _run_and_compare(env, case, lambda a, b, c: binding.forward(a, b, c, causal=True), causal=True)


@pytest.mark.parametrize("B,H,L,d", [(1, 8, 2048, 128), (1, 4, 1000, 128), (2, 5, 1408, 64), (1, 16, 1024, 128),
                                     (1, 3, 300, 64), (1, 1, 4096, 128), (1, 3, 2500, 128), (1, 5, 1800, 64)])
def test_causal_short_shapes_run_as_clusters(env, B, H, L, d):
    """Few short tiles: k CTAs per tile as one cluster, each with a share of the tile's own key steps (the tiles
    at the start of a head have fewer key steps than the cluster has CTAs: some CTAs then have nothing to do)."""
    torch, _, binding = env
    from oracle import plan_oracle as po

    t = binding.plan(binding.hw_desc_query(0), B, H, L, d, causal=True)
    want = po.derive_tiles_tmem_machine(_device_desc_dict(binding), B, H, L, d, causal=True)
    assert (t.tiles, t.ctas) == (want["tiles"], want["ctas"]) and t.ctas % t.tiles == 0
    k = t.ctas // t.tiles
    assert 2 <= k <= 4
    run = lambda a, b, c: binding.forward(a, b, c, causal=True)
    _run_and_compare(env, _case("causal_pairs", B, H, L, d, sigma_qk=math.sqrt(3.0)), run, causal=True)
    assert binding.last_cluster_size() == k
    q, kk, v = (to_cuda_bf16(x) for x in synth.make_qkv(_case("causal_pairs", B, H, L, d), seed=3))
    o1, o2 = binding.forward(q, kk, v, causal=True), binding.forward(q, kk, v, causal=True)
    ranges = binding.forward_tiles(q, kk, v, ctas=t.tiles + 1, causal=True)                  # equal ranges, merged elsewhere
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    assert float((o1.float() - ranges.float()).abs().max()) <= 2e-2


@pytest.mark.parametrize("kw", [dict(ctas=1), dict(ctas=2), dict(ctas=7), dict(ctas=37), dict(ctas=101),
                                dict(tile_kv=64), dict(n_q=1), dict(n_q=1, tile_kv=64, ctas=53), dict(kv_stages=2)])
def test_causal_tile_variants_and_grid_sizes(env, kw):
    _, _, binding = env
    case = _case("causal_variants", 2, 2, 1100, 128, sigma_qk=math.sqrt(3.0))
    _run_and_compare(env, case, lambda a, b, c: binding.forward_tiles(a, b, c, causal=True, **kw), causal=True)


def test_causal_structured_and_reproducible(env):
    torch, orc, binding = env
    L, d = 512, 128
    rng = np.random.default_rng(5)
    rnd = lambda: synth.f32_to_bf16_bits(rng.standard_normal((1, 1, L, d), dtype=np.float32))
    qb, kb, vb = rnd(), rnd(), rnd()
    q, k, v = (to_cuda_bf16(x) for x in (qb, kb, vb))
    a = binding.forward(q, k, v, causal=True)
    b = binding.forward(q, k, v, causal=True)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    out = to_host_f64(a).reshape(L, d)
    # row 0 sees only key 0: the output is V[0] exactly (one weight, equal to 1)
    assert np.array_equal(out[0], orc.bf16_bits_to_f64(vb).reshape(L, d)[0])
    # changing keys/values after position 300 must not change rows 0..300
    kb2, vb2 = kb.copy(), vb.copy()
    kb2[:, :, 301:] = rnd()[:, :, 301:]
    vb2[:, :, 301:] = rnd()[:, :, 301:]
    c = to_host_f64(binding.forward(q, to_cuda_bf16(kb2), to_cuda_bf16(vb2), causal=True)).reshape(L, d)
    assert np.array_equal(c[:301], out[:301]) and np.abs(c[301:] - out[301:]).max() > 1e-3


def test_causal_full_size_sampled_rows(env):
    _, _, binding = env
    case = synth.CONFIGS["cfg3"]
    _run_and_compare(env, case, lambda a, b, c: binding.forward(a, b, c, causal=True),
                     rows=synth.sample_rows(case.L), causal=True)
    case = synth.CONFIGS["cfg5a"]
    _run_and_compare(env, case, lambda a, b, c: binding.forward(a, b, c, causal=True),
                     rows=synth.sample_rows(case.L), causal=True)


def test_two_kernels_agree_and_runs_are_bitwise_reproducible(env):
    torch, _, binding = env
    case = _case("agree", 1, 4, 2048, 128)
    q, k, v = (to_cuda_bf16(x) for x in synth.make_qkv(case, seed=2))
    a = binding.forward(q, k, v)
    b = binding.forward(q, k, v)
    c = binding.forward_simple(q, k, v)
    s = binding.forward_tiles(q, k, v, kv_splits=4)
    s2 = binding.forward_tiles(q, k, v, kv_splits=4)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert torch.equal(s.view(torch.int16), s2.view(torch.int16))
    # balanced key ranges (the headline shape): which CTA merges a tile depends on timing, the bits must not
    big = synth.CONFIGS["cfg3"]
    qb, kb, vb = (to_cuda_bf16(x) for x in synth.make_qkv(big, seed=0))
    first = binding.forward(qb, kb, vb).clone()
    for _ in range(4):
        again = binding.forward(qb, kb, vb)
        assert torch.equal(first.view(torch.int16), again.view(torch.int16))
    fa, fc, fs = (to_host_f64(x) for x in (a, c, s))
    assert errors(fa, fc)[0] <= 1e-2 and errors(fa, fc)[1] <= 5e-3
    assert errors(fa, fs)[0] <= 1e-2 and errors(fa, fs)[1] <= 5e-3


# -------------------------------------------------------- benchmark configurations
def test_cfg1_every_row(env):
    _, _, binding = env
    _run_and_compare(env, synth.CONFIGS["cfg1"], binding.forward)


def test_cfg2_every_row(env):
    _, _, binding = env
    _run_and_compare(env, synth.CONFIGS["cfg2"], binding.forward)


def test_cfg3_headline_shape_sampled_rows(env):
    """The launch configuration the benchmark times (closed-form default tiles)."""
    _, _, binding = env
    case = synth.CONFIGS["cfg3"]
    _run_and_compare(env, case, binding.forward, rows=synth.sample_rows(case.L))


@pytest.mark.parametrize("L", [1024, 2048, 4096, 8192, 16384, 32768])
def test_cfg4_large_logit_sweep(env, L):
    """Q, K ~ N(0, 3): frequent maximum updates and rescale factors over many binades."""
    _, _, binding = env
    case = synth.CONFIGS[f"cfg4_L{L}"]
    _run_and_compare(env, case, binding.forward, rows=synth.sample_rows(L))


def test_cfg4_sigma3_extra_stress(env):
    """Standard deviation 3 (logit std 9): outputs above 4 in magnitude are judged by one bf16 ulp."""
    _, _, binding = env
    _run_and_compare(env, _case("sigma3", 1, 4, 4096, 128, sigma_qk=3.0, cfg_id=44), binding.forward,
                     rows=synth.sample_rows(4096))


@pytest.mark.parametrize("name", ["cfg5a", "cfg5b"])
def test_cfg5_prefill_batches_sampled_rows(env, name):
    _, _, binding = env
    case = synth.CONFIGS[name]
    _run_and_compare(env, case, binding.forward, rows=synth.sample_rows(case.L))


def test_host_buffer_entry_point(env):
    torch, orc, binding = env
    case = _case("host", 1, 2, 512, 128)
    q, k, v = synth.make_qkv(case, seed=4)
    hq, hk, hv = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in (q, k, v))
    ho = torch.empty_like(hq).pin_memory()
    scratch = torch.empty(4 * hq.numel() * 2, dtype=torch.uint8, device="cuda")
    binding.forward_host(hq, hk, hv, ho, scratch)
    torch.cuda.synchronize()
    got = (ho.view(torch.int16).numpy().view(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ref = orc.attention_rows(q, k, v, 1, 2, 512, 128, np.arange(512, dtype=np.int32))
    assert_close(got.reshape(2, 512, 128), ref, "host entry")


@pytest.mark.parametrize("L,d", [(8192, 128), (8192 + 72, 64), (16384 + 8, 128)])
def test_host_buffer_entry_point_pipelined_long_head(env, L, d):
    """One long head goes through the host entry point as blocks of query rows whose copies overlap the kernels:
    the result must match the oracle on sampled rows of every block and on the rows either side of each block
    boundary, on three calls in a row (the streams and events are reused), two of them on a stream of the caller's
    that alone is waited for."""
    torch, orc, binding = env
    case = _case("hostpipe", 1, 1, L, d)
    q, k, v = synth.make_qkv(case, seed=5)
    hq, hk, hv = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in (q, k, v))
    scratch = torch.empty(4 * hq.numel() * 2, dtype=torch.uint8, device="cuda")
    blocks = 2
    per = (-(-L // blocks) + 255) // 256 * 256
    edges = [e for i in range(1, blocks) for e in (i * per - 1, i * per) if e < L]
    rows = np.unique(np.concatenate([synth.sample_rows(L)[::max(1, L // 2048)], edges, [0, L - 1]])).astype(np.int32)
    ref = orc.attention_rows(q, k, v, 1, 1, L, d, rows)
    side = torch.cuda.Stream()
    for it in range(3):
        ho = torch.full_like(hq, float("nan")).pin_memory()
        if it == 0:
            binding.forward_host(hq, hk, hv, ho, scratch)
            torch.cuda.synchronize()
        else:
            # the caller waits for its own stream only: the library's copy streams must have been joined into it
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                binding.forward_host(hq, hk, hv, ho, scratch)
            side.synchronize()
        assert binding.last_device_status()[0] == 0
        got = (ho.view(torch.int16).numpy().view(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        assert np.isfinite(got).all()
        assert_close(got.reshape(1, L, d)[:, rows], ref, "pipelined host entry")
        scratch.zero_()


def test_missing_or_small_workspace_is_reported_and_nothing_runs(env):
    """A plan that shares Q tiles between CTAs needs the caller's workspace: with none registered, or one smaller than
    attn_workspace_bytes, the call returns NEED_WORKSPACE before any launch and the output is untouched."""
    import ctypes

    torch, _, binding = env
    lib = binding.lib()
    dev = torch.cuda.current_device()
    B, H, L, d = 1, 1, 4096, 128
    case = _case("needws", B, H, L, d)
    tq, tk, tv = (to_cuda_bf16(x) for x in synth.make_qkv(case, seed=7))
    o = torch.full_like(tq, float("nan"))
    need = binding.workspace_bytes(binding.plan(binding.hw_desc_query(dev), B, H, L, d), B, H, L, d)
    assert need > 65536
    binding.ensure_workspace(dev, need)                  # the buffer the binding keeps registered; restored below
    kept = binding._workspaces[dev]
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    call = lambda: lib.attn_forward(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), o.data_ptr(), B, H, L, d, stream)
    small = torch.empty(need - 16, dtype=torch.uint8, device="cuda")
    try:
        assert lib.attn_set_workspace(dev, None, 0) == 0
        assert call() == binding.ERR_NEED_WORKSPACE
        assert lib.attn_set_workspace(dev, small.data_ptr(), small.numel()) == 0
        assert call() == binding.ERR_NEED_WORKSPACE
        assert binding.lib().attn_last_launch_count() == 0
        torch.cuda.synchronize()
        assert bool(torch.isnan(o).all())
    finally:
        assert lib.attn_set_workspace(dev, kept.data_ptr(), kept.numel()) == 0
    assert call() == 0
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0 and bool(torch.isfinite(o).all())
    assert "workspace" in binding.status_string(binding.ERR_NEED_WORKSPACE)


def test_bounded_wait_expiry_is_reported_and_the_context_survives(env):
    """The library's self-test queues one warp that waits, with the kernels' bounded wait, on a barrier nothing arrives
    at.  The wait must run out by itself (about half a second), the expiry must be reported once with the place that
    gave up, and the device must go on computing correct results afterwards."""
    import ctypes
    import time

    torch, _, binding = env
    lib = binding.lib()
    assert binding.last_device_status()[0] == 0
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    t0 = time.perf_counter()
    assert lib.attn_selftest_wait_expiry(stream) == 0
    code, detail = binding.last_device_status()              # synchronises the stream
    waited = time.perf_counter() - t0
    assert code == binding.ERR_DEVICE_TIMEOUT
    assert detail[0] == 1 and detail[1] == (5 << 24) | (10 << 16) | 0x7E57 and detail[2] == 0
    assert 0.2 < waited < 5.0, f"the wait took {waited:.2f} s"
    assert binding.last_device_status()[0] == 0              # reported once, then cleared
    _run_and_compare(env, _case("after_expiry", 1, 2, 512, 128), binding.forward)
    _run_and_compare(env, _case("after_expiry_split", 1, 1, 4096, 128), binding.forward, rows=synth.sample_rows(4096))


def test_shared_tile_counters_bound_the_grid(env):
    """Grids whose CTAs share Q tiles keep two counters per warp of every (CTA, sub-tile) in the 64 KB counter block:
    more than 1024 such CTAs are refused, not run."""
    torch, _, binding = env
    case = _case("limit", 1, 1, 8192, 64)                # 32 Q tiles x 128 steps of 64 keys = 4096 units
    q, k, v = (to_cuda_bf16(x) for x in synth.make_qkv(case, 0))
    with pytest.raises(binding.AttnError) as err:
        binding.forward_tiles(q, k, v, ctas=1500, tile_kv=64)
    assert err.value.code == binding.ERR_BAD_TILES
    rows = synth.sample_rows(case.L)
    _run_and_compare(env, case, lambda a, b, c: binding.forward_tiles(a, b, c, ctas=1024, tile_kv=64), rows=rows)


@pytest.mark.parametrize("field,value,expect", [
    ("num_units", 74, dict(ctas=64)),                                  # half the SMs: two CTAs per Q tile instead of four
    ("local_mem_bytes", 166912, dict(tile_kv=64, binding_constraint=1)),   # less shared memory: smaller K/V tiles
    ("acc_mem_columns", 256, dict(n_q=1)),                             # half the tensor memory: one Q sub-tile per CTA
    ("cache_bytes", 0, dict()),                                        # no cache model
])
def test_other_descriptors_run_with_no_code_change(env, field, value, expect):
    """The paper's portability claim carried to the launch: a changed descriptor re-runs the derivation and the same
    kernels run with the tiles it gives (here: descriptors of smaller machines, on the B200 itself)."""
    torch, _, binding = env
    desc = binding.hw_desc_query(0)
    setattr(desc, field, value)
    case = _case("desc", 1, 2, 4096, 128)
    plan = binding.plan(desc, case.B, case.H, case.L, case.d)
    assert plan.feasible
    for key, want in expect.items():
        assert getattr(plan, key) == want, (key, getattr(plan, key))
    _run_and_compare(env, case, lambda a, b, c: binding.forward_desc(desc, a, b, c), rows=synth.sample_rows(case.L))
    _run_and_compare(env, case, lambda a, b, c: binding.forward_desc(desc, a, b, c, causal=True),
                     rows=synth.sample_rows(case.L), causal=True)


def test_changed_cost_constants_change_the_grid_and_the_launch_follows(env):
    """The occupancy step reads its cost constants from the descriptor: with the two ways of splitting a tile made
    expensive and equal ranges made cheap, eight heads of 2048 keys no longer run as 64 clusters of two but as one
    range per SM through the workspace -- same kernels, same result within tolerance."""
    torch, _, binding = env
    case = _case("ovh", 1, 8, 2048, 128)
    desc = binding.hw_desc_query(0)
    base = binding.plan(desc, case.B, case.H, case.L, case.d)
    assert base.ctas == 2 * base.tiles == 128
    _run_and_compare(env, case, lambda a, b, c: binding.forward_desc(desc, a, b, c), rows=synth.sample_rows(case.L))
    assert binding.last_cluster_size() == 2
    desc.ovh_cluster, desc.ovh_workspace, desc.ovh_ranges = 40, 40, 10
    plan = binding.plan(desc, case.B, case.H, case.L, case.d)
    assert plan.ctas == desc.num_units and plan.cost_steps == -(-64 * 16 // desc.num_units) + 10
    _run_and_compare(env, case, lambda a, b, c: binding.forward_desc(desc, a, b, c), rows=synth.sample_rows(case.L))
    assert binding.last_cluster_size() == 0


def test_uniform_split_larger_than_the_machine_is_merged_by_the_last_finisher(env):
    """Fixed merge roles make a merging warp wait for the other CTAs of its tile, so they need every CTA resident.  A
    uniform split with more CTAs than SMs (an override; the closed form never asks for one) runs the instantiation in
    which the last CTA of a tile to finish merges: correct, and no wait runs out."""
    torch, _, binding = env
    case = _case("big_uniform", 1, 8, 2048, 128)                 # 64 Q tiles
    for k in (3, 4):                                             # 192 and 256 CTAs on 148 SMs
        _run_and_compare(env, case, lambda a, b, c: binding.forward_tiles(a, b, c, kv_splits=k),
                         rows=synth.sample_rows(case.L), what=f"{k} CTAs per tile")
        assert binding.last_cluster_size() == 0


def test_per_call_workspaces_let_two_streams_run_split_plans_at_once(env):
    """attn_forward_ws: two streams of one device, each with its own workspace and status words, run plans that share
    Q tiles at the same time; results equal the ordinary entry point bit for bit and the oracle within tolerance."""
    torch, orc, binding = env
    desc = binding.hw_desc_query(0)
    # one range per SM (the last CTA of a tile to finish merges) and three CTAs per tile that cannot run as clusters
    cases = [_case("ws_a", 1, 1, 16384, 128, cfg_id=81), _case("ws_b", 1, 3, 4096, 128, cfg_id=82)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    work = []
    for case, st in zip(cases, streams):
        plan = binding.plan(desc, case.B, case.H, case.L, case.d)
        need = binding.workspace_bytes(plan, case.B, case.H, case.L, case.d)
        assert need > 65536
        q, k, v = synth.make_qkv(case, seed=3)
        t = [to_cuda_bf16(x) for x in (q, k, v)]
        ws = torch.empty(need, dtype=torch.uint8, device="cuda").fill_(0xAB)       # dirty: the init call must clear it
        status = torch.full((4,), 7, dtype=torch.int32, device="cuda")
        work.append(dict(case=case, host=(q, k, v), dev=t, ws=ws, status=status, stream=st,
                         out=torch.full_like(t[0], float("nan"))))
    torch.cuda.synchronize()
    for w in work:
        with torch.cuda.stream(w["stream"]):
            binding.workspace_init(w["ws"], w["status"])
    for rep in range(3):                                         # interleaved launches on the two streams
        for w in work:
            with torch.cuda.stream(w["stream"]):
                binding.forward_ws(*w["dev"], w["out"], workspace=w["ws"], status=w["status"])
                assert binding.last_cluster_size() == 0
    for w in work:
        with torch.cuda.stream(w["stream"]):
            code, detail = binding.status_read(w["status"], w["ws"])
        assert code == 0 and detail == [0, 0, 0, 0]
    torch.cuda.synchronize()
    for w in work:
        case = w["case"]
        want = binding.forward(*w["dev"])
        torch.cuda.synchronize()
        assert torch.equal(w["out"].view(torch.int16), want.view(torch.int16))
        rows = synth.sample_rows(case.L)
        ref = orc.attention_rows(*w["host"], case.B, case.H, case.L, case.d, rows)
        got = to_host_f64(w["out"]).reshape(case.B * case.H, case.L, case.d)
        assert_close(got[:, rows], ref, case.name)
    # too small a buffer is refused before any launch; no workspace is fine for a plan that needs none
    w = work[0]
    with pytest.raises(binding.AttnError) as err:
        binding.forward_ws(*w["dev"], w["out"], workspace=w["ws"][:70000], status=w["status"])
    assert err.value.code == binding.ERR_NEED_WORKSPACE and binding.last_launch_count() == 0
    small = _case("ws_none", 4, 40, 512, 64)
    tq, tk, tv = (to_cuda_bf16(x) for x in synth.make_qkv(small, 0))
    a = binding.forward_ws(tq, tk, tv)
    b = binding.forward(tq, tk, tv)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_bounded_wait_expiry_is_recorded_in_the_callers_status_words(env):
    """A launch given its own status words reports an expired wait there, not in the device-wide record.  The wait that
    runs out is the self-test's (one warp on a barrier nothing arrives at; it ends by itself at the cycle limit)."""
    torch, _, binding = env
    assert binding.last_device_status()[0] == 0
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    other = torch.zeros(4, dtype=torch.int32, device="cuda")
    case = _case("ws_status", 1, 1, 4096, 128)
    plan = binding.plan(binding.hw_desc_query(0), case.B, case.H, case.L, case.d)
    ws = torch.zeros(binding.workspace_bytes(plan, case.B, case.H, case.L, case.d), dtype=torch.uint8, device="cuda")
    tq, tk, tv = (to_cuda_bf16(x) for x in synth.make_qkv(case, 0))
    stream = torch.cuda.current_stream().cuda_stream
    rc = binding.lib().attn_selftest_wait_expiry_to(status.data_ptr(), stream)
    assert rc == 0
    out = binding.forward_ws(tq, tk, tv, workspace=ws, status=other)        # a normal launch with other status words
    code, detail = binding.status_read(status, None)
    assert code == binding.ERR_DEVICE_TIMEOUT
    assert detail[0] == 1 and detail[1] == (5 << 24) | (10 << 16) | 0x7E57 and detail[2] == 0
    assert binding.status_read(status, None) == (0, [0, 0, 0, 0])            # reported once, then cleared
    assert binding.status_read(other, ws) == (0, [0, 0, 0, 0])               # the other launch saw nothing
    assert binding.last_device_status()[0] == 0                              # nor did the device-wide record
    want = binding.forward(tq, tk, tv)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("B,H,L,d,causal", [(2, 40, 2048, 64, False), (4, 32, 8192, 64, False), (1, 8, 2048, 64, False),
                                            (2, 40, 2048, 128, False), (2, 40, 2048, 64, True)])
def test_many_launches_no_wait_expires_and_the_bits_repeat(env, B, H, L, d, causal):
    """Launch-to-launch repeatability under many launches.  At d = 64 the next step's scores are produced before this
    step's P V is issued; arrivals on the per-step barriers are anonymous, so a protocol that lets a fast warp arrive
    for step g+1 before a slow warp has arrived for step g fails once in ~10^4 launches of the large prefill shape (an
    expired wait, or a product issued before its rows were rescaled).  Every launch must leave the device status clean
    and reproduce the first launch's output bits."""
    torch, _, binding = env
    case = _case("many", B, H, L, d, cfg_id=88)
    q, k, v = (to_cuda_bf16(x) for x in synth.make_qkv(case, 0))
    first = binding.forward(q, k, v, causal=causal).clone()
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    out = torch.empty_like(q)
    launches = 300 if case.flops > 1e12 else 3000
    for it in range(launches):
        binding.forward(q, k, v, out, causal=causal)
        if it % 50 == 49 or it == launches - 1:
            code, detail = binding.last_device_status()
            assert code == 0, (it, detail)
            assert torch.equal(out.view(torch.int16), first.view(torch.int16)), f"launch {it} differs from the first"


def test_descriptor_of_a_larger_machine_is_refused(env):
    torch, _, binding = env
    desc = binding.hw_desc_query(0)
    desc.num_units += 1
    case = _case("desc", 1, 1, 512, 64)
    with pytest.raises(binding.AttnError) as err:
        binding.forward_desc(desc, *(to_cuda_bf16(x) for x in synth.make_qkv(case, 0)))
    assert err.value.code == -1


@pytest.mark.parametrize("B,H,L,d", [(1, 20, 2000, 128), (2, 40, 2047, 64), (1, 37, 1025, 128), (3, 50, 777, 64)])
def test_persistent_grid_with_ragged_lengths(env, B, H, L, d):
    """More Q tiles than SMs and little K/V per head: one persistent CTA per SM walks whole tiles and shares the ones at
    its range ends; the ragged last Q tile is clipped by the staged TMA stores, the ragged last KV tile masked."""
    _, _, binding = env
    plan = binding.plan(binding.hw_desc_query(0), B, H, L, d)
    assert plan.tiles > plan.ctas == binding.hw_desc_query(0).num_units
    case = _case("persistent", B, H, L, d)
    _run_and_compare(env, case, binding.forward)
    _run_and_compare(env, case, lambda a, b, c: binding.forward(a, b, c, causal=True), causal=True)


def test_random_shapes_every_grid_mode_agrees_with_an_unsplit_run(env):
    """Seeded random shapes, causal and not: whatever grid the plan picks (one CTA per tile, clusters of 2 to 8,
    equal ranges, persistent), the output equals that of a launch that shares no Q tile between CTAs, up to the
    merge's rounding; the modes met are counted so that a change of the plan that stops exercising one shows."""
    torch, _, binding = env
    import random

    rng = random.Random(2024)
    desc = binding.hw_desc_query(0)
    modes = {}
    for it in range(120):
        d = rng.choice([64, 128])
        causal = rng.random() < 0.5
        L = rng.choice([rng.randint(1, 300), rng.randint(300, 2500), rng.randint(2500, 7000)])
        B = rng.randint(1, 2)
        H = rng.randint(1, max(1, min(40, 50000 // L) // B))
        g = torch.Generator(device="cuda").manual_seed(it)
        q, k, v = (torch.randn(B, H, L, d, device="cuda", generator=g).mul_(1.3).to(torch.bfloat16) for _ in range(3))
        t = binding.plan(desc, B, H, L, d, causal=causal)
        o = binding.forward(q, k, v, causal=causal)
        cl = binding.last_cluster_size()
        ref = binding.forward_tiles(q, k, v, ctas=1 if causal else t.tiles, causal=causal)
        torch.cuda.synchronize()
        assert binding.last_device_status()[0] == 0, (B, H, L, d, causal)
        assert bool(torch.isfinite(o.float()).all())
        assert float((o.float() - ref.float()).abs().max()) <= 2e-2, (B, H, L, d, causal, t.ctas, t.tiles, cl)
        mode = ("causal " if causal else "") + ("cluster" if cl else "tiles" if t.ctas == t.tiles else "ranges")
        modes[mode] = modes.get(mode, 0) + 1
    assert all(modes.get(m, 0) >= 3 for m in ("cluster", "tiles", "ranges", "causal cluster", "causal ranges")), modes


@pytest.mark.parametrize("B,H,Lq,Lk,d", [(1, 2, 300, 1408, 128), (2, 3, 1000, 2500, 64), (1, 1, 4096, 16384, 128),
                                          (1, 2, 1500, 700, 128), (1, 5, 1, 333, 64), (1, 1, 2048, 8192, 128)])
def test_separate_query_and_key_lengths(env, B, H, Lq, Lk, d):
    """attn_forward_qk: Lq query rows against Lk keys.  The oracle is the self-attention oracle of length Lk whose
    first query rows are a block of the Lq rows (every query row attends to all keys, so blocks are independent)."""
    torch, orc, binding = env
    rng = np.random.default_rng([B, H, Lq, Lk, d])
    bits = lambda *shape: synth.f32_to_bf16_bits((rng.standard_normal(shape) * 1.2).astype(np.float32))
    q, k, v = bits(B * H, Lq, d), bits(B * H, Lk, d), bits(B * H, Lk, d)
    out = binding.forward_qk(to_cuda_bf16(q).view(B, H, Lq, d), to_cuda_bf16(k).view(B, H, Lk, d),
                             to_cuda_bf16(v).view(B, H, Lk, d))
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    got = to_host_f64(out).reshape(B * H, Lq, d)
    blocks = [(r0, min(Lq, r0 + Lk)) for r0 in range(0, Lq, Lk)]
    if Lq > 2048:                                            # sampled rows of the large case
        blocks = [(r0, r0 + 32) for r0 in (0, 1000, Lq - 32)]
    for r0, r1 in blocks:
        q_pad = np.zeros((B * H, Lk, d), dtype=q.dtype)
        q_pad[:, : r1 - r0] = q[:, r0:r1]
        ref = orc.attention_rows(q_pad.reshape(-1), k.reshape(-1), v.reshape(-1), B, H, Lk, d,
                                 np.arange(r1 - r0, dtype=np.int32))
        assert_close(got[:, r0:r1], ref, f"qk rows {r0}:{r1}")
    # the same through the self-attention entry point when the lengths agree
    if Lq <= 2048:
        o_self = binding.forward(to_cuda_bf16(k).view(B, H, Lk, d), to_cuda_bf16(k).view(B, H, Lk, d), to_cuda_bf16(v).view(B, H, Lk, d))
        o_qk = binding.forward_qk(to_cuda_bf16(k).view(B, H, Lk, d), to_cuda_bf16(k).view(B, H, Lk, d), to_cuda_bf16(v).view(B, H, Lk, d))
        assert torch.equal(o_self.view(torch.int16), o_qk.view(torch.int16))


@pytest.mark.parametrize("L,d,heads", [(512, 128, 33024), (520, 64, 64640)])
def test_tensors_beyond_two_to_the_31_elements(env, L, d, heads):
    """Each of Q, K, V, O holds more than 2^31 elements (4.3 GB): byte offsets and element indices past the 32-bit range.
    64 seeded heads are laid out `heads / 64` times one after the other (a device-side copy of the same host data).
    Every element of every group is compared with the oracle's result for those 64 heads (on the device, max-abs bar),
    the first and the last group -- the one past the 2^31st element -- with both bars on the host, and all but the few
    heads whose tiles straddle a boundary between two CTAs' ranges (computed in two pieces and merged) must reproduce the
    first group's bits exactly."""
    torch, orc, binding = env
    base = 64
    assert heads % base == 0 and heads * L * d > 2 ** 31
    free, _ = torch.cuda.mem_get_info()
    if free < 5 * heads * L * d * 2:
        pytest.skip("not enough free device memory for four 4.3 GB tensors")
    case = _case("big", 1, base, L, d)
    q, k, v = synth.make_qkv(case, seed=6)
    groups = heads // base
    tq, tk, tv = (to_cuda_bf16(x).reshape(1, base, L, d).repeat(1, groups, 1, 1).contiguous() for x in (q, k, v))
    assert tq.numel() > 2 ** 31
    out = torch.full_like(tq, float("nan"))
    binding.forward(tq, tk, tv, out)
    torch.cuda.synchronize()
    assert binding.last_device_status()[0] == 0
    rows = np.arange(L, dtype=np.int32)
    ref = orc.attention_rows(q, k, v, 1, base, L, d, rows)
    ref_dev = torch.from_numpy(ref.reshape(base, L, d)).cuda()
    bits = out.view(torch.int16).reshape(groups, base, L, d)
    grouped = out.reshape(groups, base, L, d)
    differing_heads, worst = 0, 0.0
    for g0 in range(0, groups, 16):
        blk = grouped[g0:g0 + 16]
        assert bool(torch.isfinite(blk).all()), f"non-finite output in groups {g0}.."
        worst = max(worst, float((blk.double() - ref_dev).abs().max()))
        differing_heads += int((bits[g0:g0 + 16] != bits[:1]).flatten(2).any(dim=2).sum())
    print(f"L={L} d={d} heads={heads}: max_abs over all groups {worst:.3e}, heads differing bitwise {differing_heads}")
    assert worst <= 1e-2, f"max_abs {worst:.3e} over all groups"
    plan = binding.plan(binding.hw_desc_query(torch.cuda.current_device()), 1, heads, L, d)
    assert differing_heads <= plan.ctas, f"{differing_heads} heads differ from their copy in the first group"
    for g in (0, groups - 1):
        got = to_host_f64(out.reshape(groups, base, L, d)[g]).reshape(base, L, d)
        assert_close(got, ref, f"head group {g}")
    del tq, tk, tv, out, bits
    torch.cuda.empty_cache()


@pytest.mark.parametrize("L,d", [(131072 + 40, 128), (262144, 64)])
def test_very_long_single_head(env, L, d):
    """One head of 131,112 (ragged) and 262,144 keys: 1025 and 2048 key steps per Q tile, row sums of that many terms
    carried through as many rescales; a stratified sample of rows against the oracle plus the whole-output properties."""
    torch, orc, binding = env
    case = _case("long", 1, 1, L, d)
    rows = synth.sample_rows(L)[:: max(1, L // 16384)]
    rows = np.unique(np.concatenate([rows, [0, 127, 128, L - 129, L - 1]])).astype(np.int32)
    assert len(rows) >= 256
    _run_and_compare(env, case, binding.forward, rows=rows)
    _run_and_compare(env, case, lambda q, k, v: binding.forward(q, k, v, causal=True), rows=rows[::4], causal=True)
