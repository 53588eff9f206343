"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol,
its planner equals the oracle-side restatement, and argument errors are reported
before any CUDA call.  No kernel is launched here."""
import ctypes
import itertools
import os
import re

import pytest

from oracle import plan_oracle as po
from tests.conftest import ROOT, read_golden


@pytest.fixture(scope="module")
def binding():
    from paper_2609_10937_b200 import binding as b
    from paper_2609_10937_b200 import build

    build.build()
    b.lib()
    return b


def _declared_functions():
    names = set()
    for header in ("attn.h", "gemm.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b((?:attn|gemm|softmax)_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(binding):
    names = _declared_functions()
    assert len(names) >= 16
    L = binding.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/*.h but not exported"
    assert set(names) == set(binding.EXPORTED_SYMBOLS)


def test_gemm_plan_closed_form(binding):
    """Tile derivation of the matrix product (Eq. 2, Eq. 3 re-read for tensor memory), retyped from the header's formula
    with the B200 constants, and its reaction to a changed descriptor."""
    desc = binding.hw_desc_b200()
    t = binding.gemm_plan(desc, 1, 4096, 4096, 4096)
    # CTA pairs: a pair owns 256 x 256; per CTA a stage is (128 + 128) * 64 * 2 = 32768 bytes, staging 8 warps x 2 x 4096
    assert (t.tile_m, t.tile_n, t.tile_k, t.n_sub, t.cta_pair, t.acc_buffers) == (256, 256, 64, 2, 2, 2)
    assert t.stages == (232448 - 65536 - 1024) // 32768 == 5 and t.smem_bytes == 5 * 32768 + 65536 + 1024
    assert (t.tiles, t.ctas, t.feasible, t.tmem_columns) == (256, 148, 1, 512)
    # last wave: 256 = 3 * 74 + 34 tiles, 2 * 34 <= 74: the 34 run as 68 half-width items (0.64 of a tile's time each)
    assert t.tail_split == 34 and t.wave_efficiency == pytest.approx(256 / ((3 + 0.64) * 74))
    t8 = binding.gemm_plan(desc, 1, 8192, 8192, 8192)          # 1024 = 13 * 74 + 62 tiles: 124 halves do not fit one wave
    assert t8.tail_split == 0 and t8.wave_efficiency == pytest.approx(1024 / (14 * 74))
    # pairs occupy as many CTAs as lone 128-row tiles would (3 * 4 * 3 = 36 pairs against 3 * 8 * 3 = 72 CTAs)
    t = binding.gemm_plan(desc, 3, 1000, 520, 256)
    assert (t.cta_pair, t.tile_m, t.tiles, t.ctas) == (2, 256, 36, 72)
    # ... whatever K is (one ring stage of products per tile: the scores of the unfused path at d = 64)
    t = binding.gemm_plan(desc, 3, 1000, 520, 64)
    assert (t.cta_pair, t.tile_m, t.tiles, t.ctas) == (2, 256, 36, 72)
    # M within one sub-tile: nothing for a second CTA to hold
    t = binding.gemm_plan(desc, 3, 128, 520, 64)
    assert (t.cta_pair, t.n_sub, t.tile_m, t.tiles) == (1, 1, 128, 9)
    # an output no wider than half the atom's N stays with lone CTAs (P V of the unfused path: 64 blocks -> 128)
    t = binding.gemm_plan(desc, 1, 16384, 128, 16384)
    assert (t.cta_pair, t.n_sub, t.tile_n, t.tiles, t.ctas) == (1, 1, 128, 128, 128)
    # a machine that cannot run pairs: the lone-CTA derivation (two sub-tiles share every B tile)
    desc.max_clusters[1] = 0
    t = binding.gemm_plan(desc, 1, 4096, 4096, 4096)
    assert (t.tile_m, t.tile_n, t.tile_k, t.n_sub, t.cta_pair, t.acc_buffers) == (256, 256, 64, 2, 1, 1)
    # stage = (256 + 256) * 64 * 2 = 65536; staging 2 * 128 * 128
    assert t.stages == (232448 - 32768 - 1024) // 65536 == 3 and t.smem_bytes == 3 * 65536 + 32768 + 1024
    assert (t.tiles, t.ctas, t.feasible, t.tmem_columns) == (256, 148, 1, 512)
    assert t.wave_efficiency == pytest.approx(256 / (2 * 148))
    # fewer two-sub-tile blocks than SMs (3 * 4 * 3 = 36 < 148): one sub-tile per block, twice as many blocks
    t = binding.gemm_plan(desc, 3, 1000, 520, 64)
    assert (t.n_sub, t.tile_m, t.tiles, t.ctas) == (1, 128, 3 * 8 * 3, 72)
    desc = binding.hw_desc_b200()
    desc.acc_mem_columns = 256                      # half the tensor memory: no second accumulator, one sub-tile
    t = binding.gemm_plan(desc, 1, 4096, 4096, 4096)
    assert (t.cta_pair, t.n_sub, t.tile_m, t.stages) == (1, 1, 128, (232448 - 16384 - 1024) // 49152)
    desc.local_mem_bytes = 101376                   # a small shared memory: the ring no longer fits twice
    t = binding.gemm_plan(desc, 1, 4096, 4096, 4096)
    assert t.feasible == 0 or t.stages >= 2


def test_plan_for_separate_query_and_key_lengths(binding):
    """attn_plan_qk: Q tiles from the query rows, key steps from the keys; equal to the oracle's restatement, and to
    attn_plan when the two lengths agree."""
    desc = binding.hw_desc_b200()
    dd = _desc_dict(desc)
    for B, H, Lq, Lk, d in [(1, 1, 4096, 16384, 128), (1, 1, 8192, 16384, 128), (2, 3, 300, 5000, 64), (1, 4, 5000, 300, 128),
                            (1, 1, 100, 4096, 128), (1, 200, 1000, 2000, 64)]:
        got = binding.plan_qk(desc, B, H, Lq, Lk, d)
        ref = po.derive_tiles_tmem_machine(dd, B, H, Lq, d, Lk=Lk)
        assert got.feasible and (got.tile_q, got.tile_kv, got.n_q, got.kv_stages, got.tiles, got.ctas) == \
            (ref["tile_q"], ref["tile_kv"], ref["n_q"], ref["kv_stages"], ref["tiles"], ref["ctas"])
        assert got.tiles == B * H * -(-Lq // got.tile_q)
    a, b = binding.plan_qk(desc, 1, 8, 2048, 2048, 128), binding.plan(desc, 1, 8, 2048, 128)
    assert a.as_dict() == b.as_dict()


def test_struct_sizes_match_the_header(binding):
    d = binding.hw_desc_b200()
    assert d.struct_bytes == ctypes.sizeof(binding.AttnHwDesc) == 136
    assert ctypes.sizeof(binding.AttnTiles) == 84
    assert binding.AttnTiles.causal.offset == 68 and binding.AttnTiles.predicted_us.offset == 80
    assert binding.AttnHwDesc.hbm_gbps.offset == 120


def _desc_dict(d):
    return {n: (list(getattr(d, n)) if n == "max_clusters" else getattr(d, n)) for n, _ in d._fields_}


def test_b200_plan_equals_oracle_restatement(binding):
    desc = binding.hw_desc_b200()
    dd = _desc_dict(desc)
    shapes = itertools.product([1, 4], [1, 8, 32], [128, 256, 1024, 2048, 4096, 16384, 32768], [64, 128, 256, 72])
    for B, H, L, d in shapes:
        got = binding.plan(desc, B, H, L, d)
        ref = po.derive_tiles_tmem_machine(dd, B, H, L, d)
        assert bool(got.feasible) == ref["feasible"], (B, H, L, d)
        assert got.binding_constraint == ref["binding"]
        if not ref["feasible"]:
            continue
        for key in ("tile_q", "tile_kv", "n_q", "n_s", "kv_stages", "kv_splits", "smem_bytes", "tmem_columns",
                    "regs_softmax", "threads", "tiles", "ctas", "cost_steps"):
            assert getattr(got, key) == ref[key], (key, B, H, L, d)
        assert bool(got.under_occupied) == ref["under_occupied"]
        assert got.wave_efficiency == pytest.approx(ref["wave_efficiency"], rel=1e-6)
        assert got.ctas_per_unit == pytest.approx(ref["ctas_per_unit"], rel=1e-6)
        gc = binding.plan(desc, B, H, L, d, causal=True)
        rc = po.derive_tiles_tmem_machine(dd, B, H, L, d, causal=True)
        assert (gc.feasible, gc.causal, gc.tile_q, gc.tile_kv, gc.kv_stages, gc.ctas, gc.cost_steps) == (
            1, 1, rc["tile_q"], rc["tile_kv"], rc["kv_stages"], rc["ctas"], rc["cost_steps"]), (B, H, L, d)


def test_occupancy_step_follows_the_descriptor_cost_constants(binding):
    """The occupancy step of the C planner against the oracle's candidate table for descriptors whose cost constants,
    unit counts and resident-cluster counts are drawn at random: the grid and its cost must be the first cheapest
    eligible candidate whatever the constants are -- the rule, not the B200 values, is what is compared here."""
    import numpy as np

    rng = np.random.default_rng(11)
    ovh = ("ovh_whole_tile", "ovh_cluster", "ovh_workspace", "ovh_ranges", "ovh_persistent", "ovh_tile_change",
           "ovh_causal_ranges", "ovh_causal_cluster")
    for _ in range(40):
        desc = binding.hw_desc_b200()
        desc.num_units = int(rng.integers(8, 200))
        for k in range(8):
            desc.max_clusters[k] = max(0, desc.num_units // (k + 1) - int(rng.integers(0, 3)))
        desc.cache_bytes = int(rng.integers(0, 3)) * (63 << 20)
        for name in ovh:
            setattr(desc, name, int(rng.integers(0, 24)))
        dd = _desc_dict(desc)
        for B, H, L, d in [(1, 1, 1024, 128), (1, 8, 2048, 128), (1, 1, 16384, 128), (2, 3, 1500, 64), (1, 40, 4096, 128),
                           (4, 32, 4096, 64), (1, 2, 8192, 128), (1, 5, 640, 64), (1, 3, 3000, 128)]:
            for causal in (False, True):
                got = binding.plan(desc, B, H, L, d, causal=causal)
                ref = po.derive_tiles_tmem_machine(dd, B, H, L, d, causal=causal)
                assert (got.ctas, got.cost_steps, got.kv_splits) == (ref["ctas"], ref["cost_steps"], ref["kv_splits"]), \
                    (B, H, L, d, causal, dd)
    # a constant changed in the descriptor changes the grid: the B200 pick for eight heads of 2048 keys is 64 clusters of 2
    desc = binding.hw_desc_b200()
    assert binding.plan(desc, 1, 8, 2048, 128).ctas == 128
    desc.ovh_cluster = desc.ovh_workspace = 40          # both ways of splitting a tile made expensive:
    assert binding.plan(desc, 1, 8, 2048, 128).ctas == 64      # whole tiles (16 + 2) beat equal ranges (7 + 12)
    desc.ovh_ranges = 10
    assert binding.plan(desc, 1, 8, 2048, 128).ctas == 148     # ... until equal ranges get cheaper (7 + 10)


def test_predicted_time_and_bound(binding):
    """attn_plan's predicted time: the longest CTA's path at the per-unit share of the descriptor's tensor peak against
    the compulsory HBM traffic at its bandwidth (the roofline the derivation's hardware model implies)."""
    desc = binding.hw_desc_b200()
    t = binding.plan(desc, 1, 1, 16384, 128)
    step_flops = 4.0 * t.tile_q * t.tile_kv * 128
    want = t.cost_steps * step_flops / (desc.peak_tflops / desc.num_units * 1e6)
    assert t.bound == 0 and t.predicted_us == pytest.approx(want, rel=1e-5)
    assert t.predicted_us >= 4.0 * 16384 ** 2 * 128 / (desc.peak_tflops * 1e6)      # never below the whole-machine roofline
    desc.hbm_gbps = 1.0                                                             # a machine with almost no bandwidth
    t = binding.plan(desc, 1, 1, 16384, 128)
    assert t.bound == 1 and t.predicted_us == pytest.approx(4 * 16384 * 128 * 2 / 1e3, rel=1e-5)
    desc.peak_tflops = 0.0
    assert binding.plan(desc, 1, 1, 16384, 128).predicted_us == 0.0


def test_other_descriptors_rerun_the_same_derivation(binding):
    """Changing the descriptor re-runs the derivation with no code change (the paper's portability claim)."""
    desc = binding.hw_desc_b200()
    for field, value in (("local_mem_bytes", 101376), ("num_units", 74), ("acc_mem_columns", 256),
                         ("regs_per_unit", 32768)):
        setattr(desc, field, value)
        for B, H, L, d in [(1, 1, 16384, 128), (4, 32, 4096, 64), (1, 8, 2048, 128)]:
            got = binding.plan(desc, B, H, L, d)
            ref = po.derive_tiles_tmem_machine(_desc_dict(desc), B, H, L, d)
            assert bool(got.feasible) == ref["feasible"]
            if ref["feasible"]:
                assert (got.tile_q, got.tile_kv, got.kv_stages, got.kv_splits, got.smem_bytes) == (
                    ref["tile_q"], ref["tile_kv"], ref["kv_stages"], ref["kv_splits"], ref["smem_bytes"])
                assert got.smem_bytes <= desc.local_mem_bytes
            assert got.binding_constraint == ref["binding"]


def _cdna_desc(binding, num_cus):
    d = binding.AttnHwDesc()
    d.struct_bytes = ctypes.sizeof(binding.AttnHwDesc)
    d.num_units, d.local_mem_bytes, d.max_regs_per_thread, d.simd_width = num_cus, 64 * 1024, 256, 64
    d.atom_m, d.atom_n, d.atom_k, d.atom_n_max, d.elem_bytes = 16, 16, 4, 16, 4
    return d


def test_register_machine_plan_reproduces_the_paper_table(binding):
    """The C planner fed the paper's CDNA descriptor returns the tiles of its Table 2."""
    for d, t_kv, t_q, regs, feasible in ([int(x) for x in r] for r in read_golden("paper_table2_tiles.txt")):
        if not feasible:
            continue
        got = binding.plan(_cdna_desc(binding, 120), 1, 1, 16384, d)
        assert (got.feasible, got.tile_kv, got.tile_q, got.regs_softmax) == (1, t_kv, t_q, regs)
        assert got.binding_constraint == po.BIND_REG
    for num_cus, t_q, t_kv, _ in read_golden("paper_derive_tiles_listing.txt"):
        got = binding.plan(_cdna_desc(binding, int(num_cus)), 1, 1, 16384, 128)
        assert (got.tile_q, got.tile_kv, got.tiles) == (int(t_q), int(t_kv), 512)


def test_plan_argument_errors(binding):
    desc = binding.hw_desc_b200()
    t = binding.AttnTiles()
    L = binding.lib()
    assert L.attn_plan(None, 1, 1, 128, 64, ctypes.byref(t)) == binding.ERR_INVALID_ARG
    desc.struct_bytes = 12
    assert L.attn_plan(ctypes.byref(desc), 1, 1, 128, 64, ctypes.byref(t)) == binding.ERR_INVALID_ARG
    desc = binding.hw_desc_b200()
    assert L.attn_plan(ctypes.byref(desc), 1, 1, 0, 64, ctypes.byref(t)) == 0 and t.feasible == 0
    assert t.binding_constraint == po.BIND_SHAPE


def test_workspace_bytes(binding):
    desc = binding.hw_desc_b200()
    t = binding.plan(desc, 1, 1, 16384, 128)
    assert (t.tiles, t.ctas) == (64, 148)
    assert binding.workspace_bytes(t, 1, 1, 16384, 128) == 65536 + 2 * t.ctas * 2 * (128 * 128 + 256) * 4
    t1 = binding.plan(desc, 4, 32, 4096, 128)
    assert binding.workspace_bytes(t1, 4, 32, 4096, 128) == 0


def test_forward_argument_errors_come_before_any_cuda_call(binding):
    L = binding.lib()
    p = ctypes.c_void_p
    a, b, c, o = 0x10000, 0x20000000, 0x40000000, 0x60000000    # never dereferenced: checks fail first
    assert L.attn_forward(None, p(b), p(c), p(o), 1, 1, 128, 64, None) == binding.ERR_INVALID_ARG
    assert L.attn_forward(p(a), p(b), p(c), p(o), 0, 1, 128, 64, None) == binding.ERR_INVALID_ARG
    assert L.attn_forward(p(a), p(b), p(c), p(o), 1, 1, 128, 96, None) == binding.ERR_UNSUPPORTED_SHAPE
    assert L.attn_forward(p(a), p(b), p(c), p(o), 1, 1, 100, 80, None) == binding.ERR_UNSUPPORTED_SHAPE
    assert L.attn_forward(p(a + 8), p(b), p(c), p(o), 1, 1, 128, 64, None) == binding.ERR_MISALIGNED
    assert L.attn_forward(p(a), p(b), p(c), p(a + 1024), 1, 1, 128, 64, None) == binding.ERR_ALIASING
    assert L.attn_forward_simple(p(a), p(b), p(c), p(b), 1, 1, 128, 64, 128, None, None) == binding.ERR_ALIASING
    assert L.attn_forward_host(p(a), p(b), p(c), p(o), 1, 1, 128, 64, p(0x7000000), 16, None) == binding.ERR_INVALID_ARG
    assert "aligned" in binding.status_string(binding.ERR_MISALIGNED)
    assert binding.status_string(12345) == "unknown status"


def test_host_entry_workspace_covers_both_query_blocks(binding):
    """One long head runs through the host entry point as blocks of query rows: its workspace figure is the
    largest of the unsplit plan's and the blocks' plans; other shapes need what attn_forward needs."""
    L = binding.lib()
    desc = binding.hw_desc_b200()
    need = lambda B, H, n, d: int(L.attn_forward_host_workspace_bytes(ctypes.byref(desc), B, H, n, d))
    for (B, H, n, d) in [(1, 1, 16384, 128), (1, 1, 8192 + 72, 64), (1, 1, 8192, 128), (1, 1, 32768 + 8, 128)]:
        blocks = 2
        per = (-(-n // blocks) + 255) // 256 * 256
        sizes = {min(per, n - i * per) for i in range(blocks) if n - i * per > 0}
        want = binding.workspace_bytes(binding.plan(desc, B, H, n, d), B, H, n, d)
        for r in sizes:
            want = max(want, binding.workspace_bytes(binding.plan_qk(desc, B, H, r, n, d), B, H, r, d))
        assert need(B, H, n, d) == want > 0
    for (B, H, n, d) in [(1, 2, 16384, 128), (1, 1, 4096, 128), (4, 32, 4096, 128)]:
        assert need(B, H, n, d) == binding.workspace_bytes(binding.plan(desc, B, H, n, d), B, H, n, d)
    assert need(1, 1, 128, 96) == 0


def test_product_does_not_reach_the_oracle():
    """The product package must not import, read or execute anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_2609_10937_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                for pat in (r"import\s+oracle", r"from\s+oracle", r"oracle[/\\.]", r"attn_oracle", r"plan_oracle"):
                    assert not re.search(pat, text), f"{f} reaches into oracle/ ({pat})"


def test_traffic_model_matches_the_paper_figures():
    """The benchmark's traffic calculator against the figures the paper prints."""
    import bench as traffic

    g = {row[0]: (int(row[1]), float(row[2])) for row in read_golden("paper_hbm_traffic.txt")}
    L = g["fused_mb"][0]
    assert round(traffic.fused_bytes(1, 1, L, 128, 4) / 1e6) == g["fused_mb"][1]
    assert round(traffic.unfused_bytes(1, 1, L, 128, 4, 4) / 1e6) == g["unfused_mb"][1]
    assert round(traffic.unfused_bytes(1, 1, L, 128, 4, 4) / traffic.fused_bytes(1, 1, L, 128, 4)) == g["ratio"][1]
    assert round(traffic.unfused_bytes(1, 1, g["unfused_gb"][0], 128, 4, 4) / 1e9) == g["unfused_gb"][1]
    assert traffic.unfused_bytes(1, 1, L, 128, 4, 4) == po.traffic_unfused(1, 1, L, 128, 4, 4)
