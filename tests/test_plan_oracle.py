"""Pins for the tile-derivation and traffic restatements under oracle/.

The register-machine derivation is pinned by the numbers the paper prints
(Table 2, the descriptor listing, the HBM-traffic paragraph).  The tensor-memory
derivation has no printed numbers: its capacity part is pinned by capacity
invariants, its occupancy part by what the arithmetic fixes -- brute-force
enumeration of the CTAs' shares on small grids, optimality and first-minimum of
the choice over the candidate table, floors on the steps per CTA, landing areas
inside the ring -- for the built-in descriptor and for descriptors with random
cost constants.
"""
import itertools
import math

import numpy as np

import pytest

from oracle import plan_oracle as po
from tests.conftest import read_golden

CDNA = dict(lds_bytes=64 * 1024, regs_per_thread=256, wavefront=64, atom_m=16, atom_n=16, elem_bytes=4)

B200 = dict(num_units=148, local_mem_bytes=232448, regs_per_unit=65536, max_regs_per_thread=255,
            simd_width=32, acc_mem_lanes=128, acc_mem_columns=512, atom_m=128, atom_n=16, atom_k=16,
            atom_n_max=256, elem_bytes=2, cache_bytes=126 << 20,
            max_clusters=[148, 74, 45, 33, 26, 22, 15, 15],
            # start and end of a CTA's work under each way of sharing out the key axis, in KV steps
            ovh_whole_tile=2, ovh_cluster=5, ovh_workspace=8, ovh_ranges=12, ovh_persistent=6, ovh_tile_change=1,
            ovh_causal_ranges=15, ovh_causal_cluster=6)


def test_table2_register_use_and_feasibility():
    for d, t_kv, t_q, regs, feasible in ((int(x) for x in row) for row in read_golden("paper_table2_tiles.txt")):
        assert po.register_file_use(t_q, t_kv, d, 64) == regs
        assert (regs <= 256) == bool(feasible)


def test_table2_tiles_are_what_the_derivation_returns():
    feasible_rows = [[int(x) for x in r] for r in read_golden("paper_table2_tiles.txt") if r[4] == "1"]
    for d, t_kv, t_q, regs, _ in feasible_rows:
        got = po.derive_tiles_register_machine(num_units=120, B=1, H=1, L=16384, d=d, **CDNA)
        assert (got["tile_kv"], got["tile_q"], got["regs"], got["feasible"]) == (t_kv, t_q, regs, True)
        # one atom step larger must not fit (the infeasible rows of the table)
        assert po.register_file_use(t_q + 16, t_kv, d, 64) > 256


def test_descriptor_listing_same_tiles_different_occupancy():
    for num_cus, t_q, t_kv, printed in read_golden("paper_derive_tiles_listing.txt"):
        got = po.derive_tiles_register_machine(num_units=int(num_cus), B=1, H=1, L=16384, d=128, **CDNA)
        assert (got["tile_q"], got["tile_kv"]) == (int(t_q), int(t_kv))
        assert got["tiles"] == 512
        # the printed per-CU figure is the blocks-per-CU ratio (its fractional part for 120 CUs)
        ratio = got["ctas_per_unit"]
        assert min(abs(ratio - float(printed)), abs(ratio - math.floor(ratio) - float(printed))) < 0.01


def test_traffic_figures_printed_in_the_paper():
    g = {row[0]: (int(row[1]), float(row[2])) for row in read_golden("paper_hbm_traffic.txt")}
    mb, gb = 1e6, 1e9
    L, val = g["fused_mb"]
    assert round(po.traffic_fused(1, 1, L, 128, 4) / mb) == val
    L, val = g["unfused_mb"]
    assert round(po.traffic_unfused(1, 1, L, 128, 4, 4) / mb) == val
    L, val = g["score_mb"]
    assert round(L * L * 4 / mb) == val
    L, val = g["ratio"]
    assert round(po.traffic_unfused(1, 1, L, 128, 4, 4) / po.traffic_fused(1, 1, L, 128, 4)) == val
    L, val = g["unfused_gb"]
    assert round(po.traffic_unfused(1, 1, L, 128, 4, 4) / gb) == val
    L, val = g["savings"]
    assert po.savings_ratio(L, 128) == val


@pytest.mark.parametrize("B,H,L,d", [(1, 1, 256, 64), (1, 8, 2048, 128), (1, 1, 16384, 128), (1, 4, 32768, 128),
                                     (4, 32, 4096, 128), (4, 32, 8192, 64), (1, 1, 128, 128), (2, 2, 1024, 256)])
def test_tmem_machine_capacity_invariants(B, H, L, d):
    t = po.derive_tiles_tmem_machine(B200, B, H, L, d)
    assert t["feasible"]
    n_q = t["n_q"]
    assert t["tile_q"] == 128 * n_q and t["tile_kv"] % 16 == 0 and 32 <= t["tile_kv"] <= 256
    assert n_q * (t["tile_kv"] + d) <= 512 <= 512 and t["tmem_columns"] <= 512       # tensor memory
    assert t["smem_bytes"] <= B200["local_mem_bytes"]                                  # shared memory
    assert t["smem_bytes"] == n_q * 128 * d * 2 + t["kv_stages"] * t["tile_kv"] * d * 2 + 3072 + n_q * 128 * 128
    assert 4 <= t["kv_stages"] <= 8
    regs_total = 128 * n_q * t["regs_softmax"] + 128 * 64 + 128 * 64                   # register file
    assert regs_total <= 65536 and t["regs_softmax"] <= 248
    assert t["tile_kv"] + t["tile_kv"] // 4 + 32 <= t["regs_softmax"]
    # one CTA per tile, several per tile (key split), or one persistent CTA per unit
    assert t["tiles"] <= t["ctas"] <= t["tiles"] * t["kv_splits"] or (t["ctas"] == 148 and t["tiles"] > 148)
    tc = po.derive_tiles_tmem_machine(B200, B, H, L, d, causal=True)
    assert tc["feasible"] and 1 <= tc["ctas"] <= 148 and tc["tile_kv"] == t["tile_kv"] and tc["tile_q"] == t["tile_q"]
    assert 0 < t["wave_efficiency"] <= 1.0
    if t["ctas"] > t["tiles"]:
        assert t["under_occupied"] and t["ctas"] <= 148
        k = t["ctas"] // t["tiles"]
        clustered = t["ctas"] % t["tiles"] == 0 and B200["max_clusters"][k - 1] >= t["tiles"]
        # at least 4 KV steps per CTA; 2 where the CTAs of a tile form a cluster
        assert t["tiles"] * math.ceil(L / t["tile_kv"]) // t["ctas"] >= (2 if clustered else 4)
        assert t["ctas"] % t["tiles"] == 0 or t["ctas"] == 148                   # uniform split or one range per SM


def test_tmem_machine_expected_defaults_for_the_benchmark_shapes():
    t = po.derive_tiles_tmem_machine(B200, 1, 1, 16384, 128)
    assert (t["tile_q"], t["tile_kv"], t["kv_stages"], t["kv_splits"], t["ctas"]) == (256, 128, 4, 3, 148)   # 65536 Q + 4 x 32768 ring + 32768 output staging + 3072 = 232448
    assert t["under_occupied"] and abs(t["wave_efficiency"] - 1.0) < 1e-12
    t = po.derive_tiles_tmem_machine(B200, 4, 32, 8192, 64)
    assert (t["tile_q"], t["tile_kv"], t["kv_stages"], t["kv_splits"]) == (256, 128, 8, 1)
    assert not t["under_occupied"]
    # more tiles than SMs: a persistent grid of 148 CTAs when it saves partial waves and CTA starts and the
    # K/V of the heads in flight fit two thirds of the L2 (4 heads x 8.4 MB), else one CTA per tile
    t = po.derive_tiles_tmem_machine(B200, 1, 4, 16384, 128)
    assert (t["tiles"], t["ctas"], t["kv_splits"]) == (256, 148, 1)
    t = po.derive_tiles_tmem_machine(B200, 4, 32, 4096, 128)                             # 128 heads x 2.1 MB
    assert (t["tiles"], t["ctas"]) == (2048, 2048)
    t = po.derive_tiles_tmem_machine(B200, 1, 42, 4096, 128)                             # 42 x 2 MiB = 84 MiB = 2/3 of 126 MiB
    assert (t["tiles"], t["ctas"]) == (672, 148)
    t = po.derive_tiles_tmem_machine(B200, 1, 43, 4096, 128)                             # 86 MiB: over
    assert (t["tiles"], t["ctas"]) == (688, 688)
    assert po.derive_tiles_tmem_machine(dict(B200, cache_bytes=0), 1, 4, 16384, 128)["ctas"] == 256
    # Fewer tiles than SMs.  Costs in KV steps per CTA: one CTA per tile steps + 2; k CTAs per tile as a cluster
    # ceil(steps / k) + 5 (k <= 8, at least 2 steps each, that many clusters resident, landing areas fit);
    # through the workspace ceil(steps / k) + 8 + k // 2 (at least 4 steps each); equal ranges ceil(total / g) + 12.
    ctas = lambda B, H, L, d, desc=B200: po.derive_tiles_tmem_machine(desc, B, H, L, d)["ctas"]
    assert ctas(1, 8, 2048, 128) == 128        # 64 tiles x 16 steps: clusters of 2 (8 + 5) against ranges (7 + 12)
    assert ctas(1, 4, 1024, 128) == 64         # 16 tiles x 8 steps: clusters of 4, two steps each (2 + 5)
    assert ctas(1, 1, 4096, 128) == 64         # 16 tiles x 32: clusters of 4 (8 + 5); 16 clusters of 8 are not resident (15)
    assert ctas(1, 1, 2048, 128) == 64         # 8 tiles x 16: clusters of 8 fit the ring (1 group x 7 parts) and 15 >= 8 are resident
    assert ctas(1, 3, 3000, 128) == 108        # 36 tiles: 36 clusters of 4 are not resident (33), 36 of 3 are
    assert ctas(1, 2, 8192, 128) == 128        # 64 tiles x 64: clusters of 2 (32 + 5) against ranges (28 + 12)
    assert ctas(1, 1, 16384, 128) == 148       # 64 tiles x 128: ranges (56 + 12) against clusters of 2 (64 + 5)
    assert ctas(1, 4, 8192, 128) == 128        # 128 tiles: whole tiles (64 + 2) against ranges (56 + 12)
    # causal: equal ranges, ceil((units + 3 tiles) / G) + 15, against k = 2..4 CTAs per tile as a cluster,
    # ceil(steps / k) + 6 (k * tiles <= 148, that many clusters resident, the longest part at least two steps)
    cc = lambda B, H, L, d, desc=B200: po.derive_tiles_tmem_machine(desc, B, H, L, d, causal=True)["ctas"]
    assert cc(1, 8, 2048, 128) == 128          # 64 tiles x <= 16 steps: pairs (8 + 6) against ranges (6 + 15)
    assert cc(1, 4, 4096, 128) == 128          # 64 tiles x <= 32: pairs (16 + 6) against ranges (9 + 15)
    assert cc(1, 1, 4096, 128) == 64           # 16 tiles: clusters of 4 (8 + 6) against ranges over 68 CTAs (5 + 15)
    assert cc(1, 1, 8192, 128) == 128          # 32 tiles x <= 64: clusters of 4 (16 + 6) against ranges (8 + 15)
    assert cc(1, 3, 300, 64) == 12             # 3 steps: pairs (2 + 6); three parts would be one step each
    assert cc(1, 1, 16384, 128) == 148 and cc(1, 2, 8192, 128) == 148
    assert cc(1, 8, 2048, 128, dict(B200, max_clusters=[0] * 8)) == 144
    no_clusters = dict(B200, max_clusters=[0] * 8)
    assert ctas(1, 8, 2048, 128, no_clusters) == 128   # workspace split in two: 8 + 8 + 1 against ranges 7 + 12
    assert ctas(1, 1, 4096, 128, no_clusters) == 128   # 16 tiles x 32: eight parts through the workspace (4 + 8 + 4) = ranges (4 + 12): tie
    assert not po.derive_tiles_tmem_machine(B200, 1, 1, 1024, 72)["feasible"]          # d not a multiple of 16
    assert not po.derive_tiles_tmem_machine(B200, 1, 1, 1024, 512)["feasible"]         # d beyond the atom's N


# ---------------------------------------------------------------------------------------------------------
# Occupancy step: the candidate table and the choice (Section "Tile Derivation", blocks against compute units)
# ---------------------------------------------------------------------------------------------------------
def _random_descriptors(n, seed=7):
    """The B200 capacities with other cost constants, unit counts and resident-cluster counts."""
    rng = np.random.default_rng(seed)
    out = [B200, dict(B200, max_clusters=[0] * 8), dict(B200, num_units=74, max_clusters=[74, 37, 22, 16, 13, 11, 7, 7])]
    for _ in range(n):
        units = int(rng.integers(8, 200))
        d = dict(B200, num_units=units, max_clusters=[units // k - int(rng.integers(0, 3)) for k in range(1, 9)],
                 cache_bytes=int(rng.integers(0, 3)) * (63 << 20))
        for key in ("ovh_whole_tile", "ovh_cluster", "ovh_workspace", "ovh_ranges", "ovh_persistent", "ovh_tile_change",
                    "ovh_causal_ranges", "ovh_causal_cluster"):
            d[key] = int(rng.integers(0, 24))
        out.append(d)
    return out


_SHAPES = [(B, H, L, d) for B, H, L, d in itertools.product([1, 2], [1, 3, 8, 40], [128, 300, 1024, 2048, 4096, 16384],
                                                            [64, 128])]


@pytest.mark.parametrize("causal", [False, True])
def test_occupancy_choice_is_the_first_cheapest_eligible_candidate(causal):
    for desc in _random_descriptors(12):
        units = desc["num_units"]
        for B, H, L, d in _SHAPES:
            t = po.derive_tiles_tmem_machine(desc, B, H, L, d, causal=causal)
            rows = t["candidates"]
            ok = [r for r in rows if r["eligible"]]
            assert ok, "some way of running the problem is always eligible"
            pick = next(r for r in ok if r["ctas"] == t["ctas"] and r["cost"] == t["cost_steps"] and r["mode"] == t["mode"])
            assert all(pick["cost"] <= r["cost"] for r in ok)                        # cheapest
            assert not any(r["cost"] == pick["cost"] for r in ok[:ok.index(pick)])   # and the first of the cheapest
            tiles, steps = t["tiles"], t["steps"]
            total = tiles * steps if not causal else B * H * po.causal_head_units(-(-L // t["tile_q"]), steps,
                                                                                  t["tile_q"] // t["tile_kv"])
            assert 1 <= t["ctas"] <= max(tiles, units) and t["kv_splits"] == -(-t["ctas"] // tiles)
            if t["under_occupied"] or causal:
                assert t["ctas"] <= units or (causal and t["mode"] == "cluster")
            # nobody's path is shorter than an even share of the work over the CTAs that exist
            assert pick["path"] >= -(-total // max(units, t["ctas"]))
            if not causal and t["under_occupied"]:
                whole = next(r for r in rows if r["mode"] == "whole_tiles")
                assert whole["eligible"] and t["cost_steps"] <= steps + desc["ovh_whole_tile"]
            # floors on what one CTA gets, and the room for what it receives
            if pick["mode"] == "cluster":
                k = pick["k"]
                assert tiles * k <= units and desc["max_clusters"][k - 1] >= tiles
                assert (-(-steps // k) if causal else steps // k) >= 2
                if k > 2:
                    assert -(-(4 * t["n_q"]) // k) * (k - 1) * (32 * 4 * d + 256) <= t["ring_bytes"]
            if pick["mode"] == "workspace":
                assert pick["k"] >= 2 and steps // pick["k"] >= 4 and tiles * pick["k"] <= units
            if pick["mode"] == "ranges" and not causal:
                assert tiles < t["ctas"] <= units and total // t["ctas"] >= 4
            if pick["mode"] == "persistent":
                heads = min(B * H, units)
                assert t["ctas"] == units and 3 * heads * 2 * L * d * 2 <= 2 * desc["cache_bytes"]


def test_candidate_paths_equal_the_brute_force_shares():
    """The `path` column against the shares counted CTA by CTA: equal ranges [c*T/G, (c+1)*T/G) of the unit line,
    equal shares [p*s/k, (p+1)*s/k) of a tile's steps; causal tiles have min(steps, (q+1)*ratio) steps."""
    for desc in (B200, dict(B200, num_units=40, max_clusters=[40, 20, 13, 10, 8, 6, 5, 5])):
        for (B, H, L, d), causal in itertools.product([(1, 1, 1024, 128), (1, 3, 1500, 128), (2, 2, 2048, 64),
                                                       (1, 5, 768, 64), (1, 1, 4096, 128), (1, 9, 640, 128)], [False, True]):
            t = po.derive_tiles_tmem_machine(desc, B, H, L, d, causal=causal)
            steps, q_tiles, ratio = t["steps"], -(-L // t["tile_q"]), t["tile_q"] // t["tile_kv"]
            per_tile = [min(steps, (q + 1) * ratio) if causal else steps for q in range(q_tiles)] * (B * H)
            assert sum(per_tile) == (B * H * po.causal_head_units(q_tiles, steps, ratio) if causal else t["tiles"] * steps)
            for r in t["candidates"]:
                if r["mode"] == "ranges":
                    T = sum(per_tile) + (3 * len(per_tile) if causal else 0)     # causal: 3 cost units lead every tile
                    G = r["ctas"]
                    assert r["path"] == max((c + 1) * T // G - c * T // G for c in range(G))
                elif r["mode"] in ("cluster", "workspace") and r["k"] >= 1:
                    k = r["k"]
                    share = lambda s: max((p + 1) * s // min(k, s) - p * s // min(k, s) for p in range(min(k, s)))
                    assert r["path"] == max(share(s) for s in per_tile)
                    assert r["ctas"] == k * len(per_tile)
                elif r["mode"] == "persistent":
                    T, G = sum(per_tile), r["ctas"]
                    assert r["path"] == max((c + 1) * T // G - c * T // G for c in range(G))


def test_cost_constants_steer_the_choice():
    """A way of sharing out the keys that is made expensive in the descriptor is no longer chosen, and with every
    cost constant zero the choice is a candidate of the shortest path."""
    t = po.derive_tiles_tmem_machine(B200, 1, 8, 2048, 128)
    assert t["mode"] == "cluster" and t["k"] == 2
    assert po.derive_tiles_tmem_machine(dict(B200, ovh_cluster=40), 1, 8, 2048, 128)["mode"] != "cluster"
    t = po.derive_tiles_tmem_machine(B200, 1, 1, 16384, 128)
    assert t["mode"] == "ranges" and t["ctas"] == 148
    t = po.derive_tiles_tmem_machine(dict(B200, ovh_ranges=14), 1, 1, 16384, 128)
    assert (t["mode"], t["k"], t["ctas"]) == ("cluster", 2, 128)
    free = dict(B200, **{k: 0 for k in B200 if k.startswith("ovh_")})
    for B, H, L, d in _SHAPES:
        t = po.derive_tiles_tmem_machine(free, B, H, L, d)
        assert t["cost_steps"] == min(r["path"] for r in t["candidates"] if r["eligible"])


def test_closed_form_grid_is_the_measured_fastest():
    """The B200 cost constants against measurements: for every shape of the grid sweep kept under profiles/ (times of
    all candidate grids on a B200), the grid the C planner derives from the built-in descriptor must be within 5 % of
    the fastest measured one.  A wrong constant or tie-break moves some pick to a measurably slower grid."""
    import os

    from paper_2609_10937_b200 import binding, build
    from tests.conftest import ROOT

    build.build()
    desc = binding.hw_desc_b200()
    shapes = {}
    with open(os.path.join(ROOT, "profiles", "grid_sweep_b200.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            B, H, L, d, q_tiles, steps, ctas, k, cluster, us, picked = line.split()
            shapes.setdefault((int(B), int(H), int(L), int(d)), {})[int(ctas)] = float(us)
    assert len(shapes) >= 18
    for (B, H, L, d), times in shapes.items():
        assert len(times) >= 2
        pick = binding.plan(desc, B, H, L, d).ctas
        assert pick in times, f"{(B, H, L, d)}: the closed form picks {pick} CTAs, which the sweep did not measure"
        assert times[pick] <= 1.05 * min(times.values()), (B, H, L, d, pick, times)
