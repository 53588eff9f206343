"""TEST INFRASTRUCTURE, NOT PRODUCT CODE: restatement of the closed-form tile
derivation and of the HBM-traffic accounting, used to check the C planner.

Nothing here is imported by the product; nothing here imports the product.

* ``derive_tiles_register_machine`` -- the paper's derivation for a machine
  whose accumulators live in vector registers (Section "Tile Derivation" and
  Table 2): the local data share fixes the K/V tile, the register file fixes
  the Q tile at the point between the two GEMMs where the Q fragment, the
  score tile and the output accumulator are all live.  The paper announces the
  register formula but prints only its results (Table 2); the formula below is
  the reading that reproduces all four printed rows:
      V(t_Q) = t_Q * (2 d + t_KV + 8) / wavefront + 16,
      t_KV   = LDS / (2 * d * elem).
  Pinned by Table 2 (tests/golden/paper_table2_tiles.txt).
* ``derive_tiles_tmem_machine`` -- the same fixed-order derivation restated for
  a machine whose accumulators live in tensor memory (B200).  No paper numbers
  exist for it: parity unpinned against the paper.  Its capacity part is pinned
  by capacity invariants; its occupancy part (``grid_candidates`` /
  ``choose_grid``: every way of sharing out the key axis listed with its
  eligibility and cost, the first cheapest taken) is pinned by the properties
  the arithmetic fixes (tests/test_plan_oracle.py) and, for the B200 cost
  constants, by a measured sweep of grid sizes kept under profiles/.
* ``traffic_fused`` / ``traffic_unfused`` -- the paper's HBM accounting
  (savings equation and the "HBM traffic" paragraph of Section "Results").
  Pinned by the printed 34 MB / 1,074 MB / 4,329 MB / 129x / 17 GB figures.
"""
from __future__ import annotations

import math

BIND_NONE, BIND_SMEM, BIND_TMEM, BIND_REG, BIND_ATOM, BIND_SHAPE = range(6)


def _floor_to(x: int, m: int) -> int:
    return (x // m) * m


def _pow2_floor(x: int) -> int:
    return 0 if x < 1 else 1 << (int(x).bit_length() - 1)


def register_file_use(t_q: int, t_kv: int, d: int, wavefront: int) -> int:
    """Registers per thread at the point between the two GEMMs (Table 2)."""
    live = t_q * (2 * d + t_kv + 8)          # Q fragment + O accumulator + S tile + row stats
    return -(-live // wavefront) + 16        # spread over the wavefront, plus fixed overhead


def derive_tiles_register_machine(lds_bytes, regs_per_thread, wavefront, num_units,
                                  atom_m, atom_n, elem_bytes, B, H, L, d):
    t_kv = _floor_to(lds_bytes // (2 * d * elem_bytes), atom_n)   # K_t and V_t both staged
    t_q = _floor_to(((regs_per_thread - 16) * wavefront) // (2 * d + t_kv + 8), atom_m)
    feasible = t_q >= atom_m and t_kv >= atom_n
    tiles = B * H * -(-L // t_q) if feasible else 0
    per_unit = tiles / num_units
    return dict(tile_q=t_q, tile_kv=t_kv, regs=register_file_use(t_q, t_kv, d, wavefront),
                feasible=feasible, binding=BIND_REG, tiles=tiles, ctas_per_unit=per_unit,
                under_occupied=tiles < num_units)


# Role structure of the B200 kernel that the derivation budgets for.
_REGS_CORRECTION = 64      # per thread, correction warpgroup
_REGS_OTHER = 64           # per thread, TMA / MMA-issue warpgroup
_REGS_ROW_OVERHEAD = 32    # softmax thread: addresses, row statistics, loop state
_SMEM_MISC = 3072          # barriers, rescale factors, tensor-memory slot
_OUT_ROW_BYTES = 128       # output staging: per softmax warpgroup 64 bf16 columns of each of its rows
_MAX_STAGES = 8
_MIN_STAGES = 4
_MIN_TILE_KV = 32


def causal_head_units(q_tiles: int, steps: int, ratio: int) -> int:
    """KV steps summed over the Q tiles of one head when tile q needs min(steps, (q+1)*ratio) of them."""
    return sum(min(steps, (q + 1) * ratio) for q in range(q_tiles))


def _cdiv(a: int, b: int) -> int:
    return -(-a // b)


def grid_candidates(desc: dict, heads: int, q_tiles: int, steps: int, ratio: int, causal: bool, n_q: int, d: int,
                    ring_bytes: int, kv_head_bytes: int) -> list:
    """Occupancy step (Section "Tile Derivation": block count against compute units) as a table.

    Every way of sharing the (Q tile, KV step) units out to CTAs is one row: its name, the CTAs per tile k (0 if
    not a per-tile split), the grid size, whether the machine can run it (with the reason if not), the KV steps on
    the longest CTA's path, and that path plus the descriptor's measured start/end cost for this way (`ovh_*`,
    in KV steps).  The derivation takes the first row of least cost among the eligible ones; nothing is searched
    beyond this fixed list.  A part that travels between CTAs of a cluster is 32 rows of d fp32 values plus 256
    bytes of row statistics; what a CTA receives lands in its Q buffer (two parts) or in its K/V ring.
    """
    units = desc["num_units"]
    clusters = list(desc.get("max_clusters", [0] * 8))
    tiles = heads * q_tiles
    part_bytes = 32 * 4 * d + 256
    groups = 4 * n_q                                  # 32-row groups of one Q tile
    rows = []

    def row(mode, k, ctas, path, ovh, reasons):
        rows.append(dict(mode=mode, k=k, ctas=ctas, path=path, cost=path + ovh, eligible=not reasons,
                         why_not=reasons))

    def cluster_reasons(k, min_share):
        why = []
        if tiles * k > units:
            why.append("more CTAs than units")
        if clusters[k - 1] < tiles:
            why.append("clusters not all resident")
        if min_share < 2:
            why.append("fewer than 2 steps per CTA")
        if k > 2 and _cdiv(groups, k) * (k - 1) * part_bytes > ring_bytes:
            why.append("landing areas exceed the ring")
        return why

    if causal:
        total = heads * causal_head_units(q_tiles, steps, ratio)
        g = max(1, min(units, total // 4))
        row("ranges", 0, g, _cdiv(total + 3 * tiles, g), desc["ovh_causal_ranges"], [])
        for k in (2, 3, 4):
            why = cluster_reasons(k, _cdiv(steps, k))
            if ratio < 2:
                why.append("Q tile no longer than the KV tile")
            row("cluster", k, tiles * k, _cdiv(steps, k), desc["ovh_causal_cluster"], why)
        return rows

    total = tiles * steps
    if tiles >= units:
        waves = _cdiv(tiles, units)
        rows.append(dict(mode="whole_tiles", k=1, ctas=tiles, path=waves * steps,
                         cost=waves * (steps + desc["ovh_whole_tile"]), eligible=True, why_not=[]))
        in_flight = min(heads, units)
        cached = desc.get("cache_bytes", 0) > 0 and 3 * in_flight * kv_head_bytes <= 2 * desc["cache_bytes"]
        row("persistent", 0, units, _cdiv(total, units), desc["ovh_persistent"] + waves * desc["ovh_tile_change"],
            [] if cached else ["K/V of the heads in flight exceed two thirds of the cache"])
        return rows

    row("whole_tiles", 1, tiles, steps, desc["ovh_whole_tile"], [])
    for k in range(2, 9):
        row("cluster", k, tiles * k, _cdiv(steps, k), desc["ovh_cluster"], cluster_reasons(k, steps // k))
    k = min(units // tiles, steps // 4)
    row("workspace", k, tiles * max(k, 1), _cdiv(steps, max(k, 1)), desc["ovh_workspace"] + k // 2,
        [] if k >= 2 else ["fewer than two parts of 4 steps"])
    g = min(units, total // 4)
    row("ranges", 0, max(g, 1), _cdiv(total, max(g, 1)), desc["ovh_ranges"],
        [] if g > tiles else ["no more CTAs than tiles"])
    return rows


def choose_grid(rows: list) -> dict:
    """First row of least cost among the eligible ones (ties go to the earlier row)."""
    ok = [r for r in rows if r["eligible"]]
    least = min(r["cost"] for r in ok)
    return next(r for r in ok if r["cost"] == least)


def derive_tiles_tmem_machine(desc: dict, B: int, H: int, L: int, d: int, causal: bool = False, Lk: int = 0) -> dict:
    """L query rows and Lk keys per head (Lk = 0: self-attention, Lk = L)."""
    Lk = Lk or L
    sub = desc["atom_m"]
    out = dict(feasible=False, binding=BIND_SHAPE)
    if d % desc["atom_k"] or d % desc["atom_n"] or d > desc["atom_n_max"] or min(B, H, L, d) <= 0:
        return out
    n_q = 2 if L > sub else 1
    while True:
        threads = 128 * (n_q + 2)
        regs_soft = _floor_to((desc["regs_per_unit"] - 128 * _REGS_CORRECTION - 128 * _REGS_OTHER)
                              // (128 * n_q), 8)
        regs_soft = min(regs_soft, _floor_to(desc["max_regs_per_thread"], 8))
        c_reg = ((regs_soft - _REGS_ROW_OVERHEAD) * 4) // 5       # S row + a quarter row of packed P
        c_tmem = desc["acc_mem_columns"] // n_q - d               # S tile + O accumulator per sub-tile
        c_atom = desc["atom_n_max"]
        c = min(c_reg, c_tmem, c_atom)
        binding = BIND_TMEM if c == c_tmem else (BIND_REG if c == c_reg else BIND_ATOM)
        tile_kv = _pow2_floor(c)
        if tile_kv >= _MIN_TILE_KV or n_q == 1:
            break
        n_q = 1
    if tile_kv < _MIN_TILE_KV:
        out["binding"] = binding
        return out
    q_bytes = n_q * sub * d * desc["elem_bytes"]
    reserve = _SMEM_MISC + n_q * sub * _OUT_ROW_BYTES
    while True:
        stage = tile_kv * d * desc["elem_bytes"]
        stages = min((desc["local_mem_bytes"] - q_bytes - reserve) // stage, _MAX_STAGES)
        if stages >= _MIN_STAGES:
            break
        tile_kv //= 2
        binding = BIND_SMEM
        if tile_kv < _MIN_TILE_KV:
            out["binding"] = BIND_SMEM
            return out
    tile_q = n_q * sub
    q_tiles = _cdiv(L, tile_q)
    tiles = B * H * q_tiles
    steps = _cdiv(Lk, tile_kv)
    under = tiles < desc["num_units"]
    rows = grid_candidates(desc, B * H, q_tiles, steps, tile_q // tile_kv, causal, n_q, d, stages * stage,
                           2 * Lk * d * desc["elem_bytes"])
    pick = choose_grid(rows)
    ctas = pick["ctas"]
    per_unit = ctas / desc["num_units"]
    cols = n_q * (tile_kv + d)
    return dict(feasible=True, binding=binding, tile_q=tile_q, tile_kv=tile_kv, n_q=n_q, n_s=1,
                kv_stages=stages, kv_splits=_cdiv(ctas, tiles),
                smem_bytes=q_bytes + stages * stage + reserve,
                tmem_columns=max(32, 1 << (cols - 1).bit_length()), regs_softmax=regs_soft,
                threads=threads, tiles=tiles, ctas=ctas, ctas_per_unit=per_unit,
                wave_efficiency=per_unit / math.ceil(per_unit), under_occupied=under,
                cost_steps=pick["cost"], mode=pick["mode"], k=pick["k"], candidates=rows, steps=steps,
                ring_bytes=stages * stage)


def traffic_fused(B, H, L, d, elem_bytes):
    """Q, K, V read once and R written once (bytes)."""
    return B * H * 4 * L * d * elem_bytes


def traffic_unfused(B, H, L, d, elem_bytes, score_bytes):
    """Three separate GEMM/softmax passes with the L x L matrix in HBM between
    them: S written, S read, P written, P read, plus Q, K, V, R once (bytes)."""
    return B * H * (4 * L * L * score_bytes + 4 * L * d * elem_bytes)


def savings_ratio(L, d):
    """The paper's savings equation: L^2 elem / (4 L d elem) = L / (4 d)."""
    return L / (4.0 * d)
