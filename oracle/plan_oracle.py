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
  exist for it: parity unpinned against the paper; pinned by capacity
  invariants only.
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
_MIN_STEPS_PER_SPLIT = 4
_SEGMENT_OVERHEAD_STEPS = 3
_CTA_OVERHEAD_STEPS = 2     # start and end of a CTA that handles one whole Q tile
_TRANSITION_STEPS = 1       # a persistent CTA moving on to its next Q tile
# fewer Q tiles than units: cost of the end of a CTA's work, in KV steps
_MIN_STEPS_PER_CLUSTER_SPLIT = 2
_CLUSTER_OVERHEAD_STEPS = 5      # k CTAs per tile as one cluster (partials through distributed shared memory)
_WORKSPACE_OVERHEAD_STEPS = 8    # k CTAs per tile, partials through the workspace (plus k // 2)
_BALANCED_OVERHEAD_STEPS = 12    # equal ranges of the unit line
_LANDING_PART_EXTRA = 256        # m and delta of the 32 rows of one part


def causal_head_units(q_tiles: int, steps: int, ratio: int) -> int:
    """KV steps summed over the Q tiles of one head when tile q needs min(steps, (q+1)*ratio) of them."""
    return sum(min(steps, (q + 1) * ratio) for q in range(q_tiles))


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
    tiles = B * H * -(-L // tile_q)
    steps = -(-Lk // tile_kv)
    under = tiles < desc["num_units"]
    ctas = tiles
    kv_head_bytes = 2 * Lk * d * desc["elem_bytes"]           # K and V of one head
    if causal:
        total = B * H * causal_head_units(-(-L // tile_q), steps, tile_q // tile_kv)
        ctas = max(1, min(total // _MIN_STEPS_PER_SPLIT, desc["num_units"]))
        # equal ranges (3 cost units per tile on the line, 15 steps of overhead) against k = 2..4 CTAs per tile as one
        # cluster, a share of the tile's own key steps each (the longest tile sets the time; 6 steps of overhead)
        cost_ranges = -(-(total + 3 * tiles) // ctas) + 15
        ratio = tile_q // tile_kv
        best = cost_ranges
        clusters = list(desc.get("max_clusters", [0] * 8))
        part = 32 * 4 * d + _LANDING_PART_EXTRA
        for k in (2, 3, 4):
            if ratio < 2 or k * tiles > desc["num_units"] or clusters[k - 1] < tiles or -(-steps // k) < 2:
                continue
            if k > 2 and -(-(4 * n_q) // k) * (k - 1) * part > stages * stage:
                continue
            cost = -(-steps // k) + 6
            if cost < best:
                best, ctas = cost, k * tiles
    elif under:
        # one CTA per tile; k CTAs per tile as one cluster; k CTAs per tile through the workspace; equal ranges.
        # The cheapest wins, ties go to the earlier candidate.
        units = desc["num_units"]
        total = tiles * steps
        best = steps + _CTA_OVERHEAD_STEPS
        clusters = list(desc.get("max_clusters", [0] * 8))
        groups = 4 * n_q
        part = 32 * 4 * d + _LANDING_PART_EXTRA
        for k in range(2, 9):
            if tiles * k > units or steps // k < _MIN_STEPS_PER_CLUSTER_SPLIT or clusters[k - 1] < tiles:
                continue
            if k > 2 and -(-groups // k) * (k - 1) * part > stages * stage:
                continue
            cost = -(-steps // k) + _CLUSTER_OVERHEAD_STEPS
            if cost < best:
                best, ctas = cost, tiles * k
        k = min(units // tiles, steps // _MIN_STEPS_PER_SPLIT)
        if k >= 2:
            cost = -(-steps // k) + _WORKSPACE_OVERHEAD_STEPS + k // 2
            if cost < best:
                best, ctas = cost, tiles * k
        g = min(total // _MIN_STEPS_PER_SPLIT, units)
        if g > tiles:
            cost = -(-total // g) + _BALANCED_OVERHEAD_STEPS
            if cost < best:
                best, ctas = cost, g
    else:
        # enough tiles for every unit: one CTA per tile (whole waves, each CTA its own start and end), or one
        # persistent CTA per unit on an equal range of the (tile, step) line -- only if the K/V of the heads
        # then in flight stay inside two thirds of the last-level cache
        units = desc["num_units"]
        total = tiles * steps
        cost_tiles = -(-tiles // units) * (steps + _CTA_OVERHEAD_STEPS)
        cost_balanced = -(-total // units) + 2 * _SEGMENT_OVERHEAD_STEPS + -(-tiles // units) * _TRANSITION_STEPS
        in_flight = min(B * H, units)
        cached = desc.get("cache_bytes", 0) > 0 and 3 * in_flight * kv_head_bytes <= 2 * desc["cache_bytes"]
        if cached and cost_balanced < cost_tiles:
            ctas = units
    kv_splits = -(-ctas // tiles)
    per_unit = ctas / desc["num_units"]
    cols = n_q * (tile_kv + d)
    return dict(feasible=True, binding=binding, tile_q=tile_q, tile_kv=tile_kv, n_q=n_q, n_s=1,
                kv_stages=stages, kv_splits=kv_splits,
                smem_bytes=q_bytes + stages * stage + reserve,
                tmem_columns=max(32, 1 << (cols - 1).bit_length()), regs_softmax=regs_soft,
                threads=threads, tiles=tiles, ctas=ctas, ctas_per_unit=per_unit,
                wave_efficiency=per_unit / math.ceil(per_unit), under_occupied=under)


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
