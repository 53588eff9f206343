// Closed-form tile derivation for fused attention (host only, no CUDA calls).
//
// The paper derives tiles from a hardware descriptor by applying capacity
// constraints in a fixed order around the compute unit (Section "Tile
// Derivation"): local memory fixes the staged tile, the register file fixes
// the accumulator tile at the point between the two matrix products where
// every intermediate is live, then the block count is checked against the
// number of compute units and the result is aligned to the instruction atom.
// Two machine models are covered:
//   * accumulators in vector registers (the paper's CDNA targets; reproduces
//     its Table 2), selected by acc_mem_columns == 0;
//   * accumulators in tensor memory (B200): S/P and O live in tensor-memory
//     columns, one S row lives in the registers of one softmax thread, K/V
//     tiles live in a shared-memory ring.
// No quantity is searched: each is a floor/ceil of descriptor fields.
#include <cstdint>
#include <cstring>

#include "attn.h"
#include "attn_plan_internal.h"
#include "gemm.h"

namespace {

// Role structure of the B200 kernel the register budget is derived for.
constexpr int kRegsCorrection = 64;   // per thread: O-rescale warpgroup
constexpr int kRegsOther = 64;        // per thread: TMA and MMA-issue warpgroup
constexpr int kRegsRowOverhead = 32;  // softmax thread: row statistics, addresses, loop state
constexpr int kSmemMisc = 3072;       // barriers, rescale factors, tensor-memory slot
constexpr int kOutRowBytes = 128;     // output staging: per softmax warpgroup one chunk of 64 bf16 columns per row
constexpr int kMaxStages = 8;
constexpr int kMinStages = 4;         // K_j, V_j and one of each in flight
constexpr int kMinTileKv = 32;
constexpr int kMinStepsPerSplit = 4;          // least KV steps of a CTA whose partial goes through the workspace
constexpr int kMinStepsPerClusterSplit = 2;
constexpr int kLandingPartExtra = 256;       // m and delta of the 32 rows of one part
constexpr int kCausalTileCostUnits = 3;      // cost units that precede every causal tile on the unit line (kernel constant)

inline int floor_to(int x, int m) { return (x / m) * m; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int pow2_floor(int x) {
  int p = 1;
  if (x < 1) return 0;
  while (p * 2 <= x) p *= 2;
  return p;
}
inline int pow2_ceil(int x) {
  int p = 1;
  while (p < x) p *= 2;
  return p;
}

// Registers per thread at the point between the two products on a register
// machine: Q fragment (d), O accumulator (d), score tile (t_kv) and 8 row
// statistics per Q row, spread over the wavefront, plus 16 of fixed overhead
// (reproduces the four rows of the paper's Table 2).
inline int register_machine_regs(int t_q, int t_kv, int d, int simd) {
  return ceil_div(t_q * (2 * d + t_kv + 8), simd) + 16;
}

}  // namespace

// Work units of one head: every Q tile takes all `steps` KV steps, or -- causal -- only the steps whose
// keys are not after the tile's last row, min(steps, (q+1)*ratio): a triangular number until that saturates.
long long attn_internal::head_units(int q_tiles, int steps, int ratio, int causal) {
  if (!causal) return (long long)q_tiles * steps;
  long long qc = steps / ratio;
  if (qc > q_tiles) qc = q_tiles;
  return (long long)ratio * qc * (qc + 1) / 2 + (long long)(q_tiles - qc) * steps;
}

// Occupancy step of the derivation (shared with the tile-override path of the launcher).  Every candidate's cost is
// KV steps on the longest CTA's path plus the descriptor's measured cost of that candidate's start and end.
attn_internal::Grid attn_internal::grid_size(const attn_hw_desc& h, int heads, int q_tiles, int steps, int ratio, int causal,
                                             long long kv_bytes_per_head, int groups, int part_floats_per_row,
                                             long long ring_bytes) {
  const long long tiles_ll = (long long)heads * q_tiles;
  const long long total = (long long)heads * head_units(q_tiles, steps, ratio, causal);
  const long long part_bytes = 32LL * 4 * part_floats_per_row + kLandingPartExtra;
  if (causal) {
    // Equal ranges of the unit line (every tile preceded by kCausalTileCostUnits cost units, as in the kernel), or -- few
    // and short tiles -- k = 2..4 CTAs per tile as one cluster, each with a share of the tile's own key steps: the
    // longest tile then sets the time, but a CTA has one piece instead of many short ones.
    long long g = total / kMinStepsPerSplit;
    if (g > h.num_units) g = h.num_units;
    if (g < 1) g = 1;
    Grid best = {(int)g, (total + kCausalTileCostUnits * tiles_ll + g - 1) / g + h.ovh_causal_ranges};
    for (int k = 2; k <= 4 && ratio >= 2; ++k) {
      if (k * tiles_ll > h.num_units || h.max_clusters[k - 1] < tiles_ll || ceil_div(steps, k) < 2) continue;
      if (k > 2 && (long long)ceil_div(groups, k) * (k - 1) * part_bytes > ring_bytes) continue;
      const long long cost = ceil_div(steps, k) + h.ovh_causal_cluster;
      if (cost < best.cost) best = {(int)(k * tiles_ll), cost};
    }
    return best;
  }
  const int tiles = (int)tiles_ll;
  if (tiles_ll >= h.num_units) {
    // Enough tiles for every unit.  One CTA per tile runs ceil(tiles/units) waves, the last one partly
    // empty, and every CTA pays its own start and end.  One persistent CTA per unit with an equal range
    // of the unit line has neither cost but works on `units` different places at once: it is taken only
    // when the K and V of the heads then in flight stay in two thirds of the cache.
    const long long g = h.num_units;
    const long long waves = (tiles_ll + g - 1) / g;
    const long long cost_tiles = waves * (steps + h.ovh_whole_tile);
    const long long cost_balanced = (total + g - 1) / g + h.ovh_persistent + waves * h.ovh_tile_change;
    const long long heads_in_flight = heads < g ? heads : g;
    const bool cached = h.cache_bytes > 0 && 3 * heads_in_flight * kv_bytes_per_head <= 2 * (long long)h.cache_bytes;
    if (cached && cost_balanced < cost_tiles) return {(int)g, cost_balanced};
    return {tiles, cost_tiles};
  }
  // Fewer tiles than units: k CTAs per tile along the key axis, or equal ranges of the unit line.  The cheapest wins,
  // ties go to the earlier candidate.
  Grid best = {tiles, steps + h.ovh_whole_tile};             // one CTA per tile, nothing to merge
  // (1) k CTAs per tile as one cluster: the tile's clusters must all be resident, every CTA needs a few steps, and
  // what a CTA receives must fit its landing area -- for two parts the Q buffer, else the K/V ring: the 32-row
  // groups one CTA merges, times the k-1 parts of each.
  for (int k = 2; k <= 8; ++k) {
    if ((long long)tiles * k > h.num_units || steps / k < kMinStepsPerClusterSplit || h.max_clusters[k - 1] < tiles) continue;
    if (k > 2 && (long long)ceil_div(groups, k) * (k - 1) * part_bytes > ring_bytes) continue;
    const long long cost = ceil_div(steps, k) + h.ovh_cluster;
    if (cost < best.cost) best = {tiles * k, cost};
  }
  // (2) k CTAs per tile, partials through the workspace
  {
    int k = h.num_units / tiles;
    const int k_max = steps / kMinStepsPerSplit;
    if (k > k_max) k = k_max;
    if (k >= 2) {
      const long long cost = ceil_div(steps, k) + h.ovh_workspace + k / 2;
      if (cost < best.cost) best = {tiles * k, cost};
    }
  }
  // (3) equal ranges
  {
    long long g = total / kMinStepsPerSplit;
    if (g > h.num_units) g = h.num_units;
    if (g > tiles) {
      const long long cost = (total + g - 1) / g + h.ovh_ranges;
      if (cost < best.cost) best = {(int)g, cost};
    }
  }
  return best;
}

namespace {

void plan_register_machine(const attn_hw_desc& h, int B, int H, int L, int d, attn_tiles* t) {
  // Local memory holds K_t and V_t together.
  const int t_kv = floor_to(h.local_mem_bytes / (2 * d * h.elem_bytes), h.atom_n);
  const int t_q = (t_kv > 0)
      ? floor_to(((h.max_regs_per_thread - 16) * h.simd_width) / (2 * d + t_kv + 8), h.atom_m)
      : 0;
  t->binding_constraint = ATTN_BIND_REG;
  if (t_kv < h.atom_n) { t->binding_constraint = ATTN_BIND_SMEM; return; }
  if (t_q < h.atom_m) return;
  t->feasible = 1;
  t->tile_q = t_q;
  t->tile_kv = t_kv;
  t->n_q = 1;
  t->n_s = 1;
  t->kv_stages = 1;
  t->kv_splits = 1;
  t->smem_bytes = 2 * t_kv * d * h.elem_bytes;
  t->tmem_columns = 0;
  t->regs_softmax = register_machine_regs(t_q, t_kv, d, h.simd_width);
  t->threads = h.simd_width;
  t->tiles = B * H * ceil_div(L, t_q);
  t->ctas = t->tiles;
  t->ctas_per_unit = (float)t->ctas / (float)h.num_units;
  const int waves = ceil_div(t->ctas, h.num_units);
  t->wave_efficiency = (float)((double)t->ctas / ((double)waves * h.num_units));
  t->under_occupied = t->tiles < h.num_units;
}

// L query rows and Lk keys per head (Lk == L for self-attention)
void plan_tmem_machine(const attn_hw_desc& h, int B, int H, int L, int Lk, int d, int causal, attn_tiles* t) {
  const int sub = h.atom_m;  // one tensor-memory lane per Q row
  t->binding_constraint = ATTN_BIND_SHAPE;
  if (d % h.atom_k || d % h.atom_n || d > h.atom_n_max) return;

  // 1. Sub-tiles per CTA, registers and tensor memory => tile_KV.
  int n_q = (L > sub) ? 2 : 1;
  int tile_kv = 0, regs_soft = 0, binding = ATTN_BIND_NONE;
  for (;;) {
    regs_soft = floor_to((h.regs_per_unit - 128 * kRegsCorrection - 128 * kRegsOther) / (128 * n_q), 8);
    const int cap = floor_to(h.max_regs_per_thread, 8);
    if (regs_soft > cap) regs_soft = cap;
    const int c_reg = ((regs_soft - kRegsRowOverhead) * 4) / 5;  // S row + a quarter row of packed P
    const int c_tmem = h.acc_mem_columns / n_q - d;              // S tile + O accumulator per sub-tile
    const int c_atom = h.atom_n_max;
    int c = c_reg < c_tmem ? c_reg : c_tmem;
    if (c_atom < c) c = c_atom;
    binding = (c == c_tmem) ? ATTN_BIND_TMEM : (c == c_reg ? ATTN_BIND_REG : ATTN_BIND_ATOM);
    tile_kv = pow2_floor(c);
    if (tile_kv >= kMinTileKv || n_q == 1) break;
    n_q = 1;
  }
  t->binding_constraint = binding;
  if (tile_kv < kMinTileKv) return;

  // 2. Shared memory => depth of the K/V ring.  Resident beside it: the Q tile, and per softmax warpgroup
  //    one 64-column chunk of its output rows, through which finished Q tiles leave while the next one loads.
  const int q_bytes = n_q * sub * d * h.elem_bytes;
  const int kSmemReserve = kSmemMisc + n_q * sub * kOutRowBytes;
  int stage = 0, stages = 0;
  for (;;) {
    stage = tile_kv * d * h.elem_bytes;
    stages = (h.local_mem_bytes - q_bytes - kSmemReserve) / stage;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages >= kMinStages) break;
    tile_kv /= 2;
    binding = ATTN_BIND_SMEM;
    if (tile_kv < kMinTileKv) { t->binding_constraint = ATTN_BIND_SMEM; return; }
  }

  // 3. Occupancy: blocks against compute units.  With fewer Q tiles than units the key axis is shared
  //    out in whichever way has the shortest critical path, counted in KV steps plus the descriptor's
  //    measured cost of the start and end of a CTA's work under that way (see grid_size).
  //    Q tiles shared by several CTAs are merged with the merge operator of the online softmax.
  const int tile_q = n_q * sub;
  const int tiles = B * H * ceil_div(L, tile_q);
  const int steps = ceil_div(Lk, tile_kv);
  const int under = tiles < h.num_units;
  // (4 n_q groups of 32 rows per tile; a part of one group is 32 rows of d fp32 values plus statistics)
  const attn_internal::Grid grid = attn_internal::grid_size(h, B * H, ceil_div(L, tile_q), steps, tile_q / tile_kv, causal,
                                                            2LL * Lk * d * h.elem_bytes, 4 * n_q, d, (long long)stages * stage);
  const int ctas = grid.ctas;
  const int kv_splits = ceil_div(ctas, tiles);

  t->feasible = 1;
  t->binding_constraint = binding;
  t->tile_q = tile_q;
  t->tile_kv = tile_kv;
  t->n_q = n_q;
  t->n_s = 1;
  t->kv_stages = stages;
  t->kv_splits = kv_splits;
  t->smem_bytes = q_bytes + stages * stage + kSmemReserve;
  t->tmem_columns = pow2_ceil(n_q * (tile_kv + d));
  if (t->tmem_columns < 32) t->tmem_columns = 32;
  t->regs_softmax = regs_soft;
  t->threads = 128 * (n_q + 2);
  t->tiles = tiles;
  t->ctas = ctas;
  t->ctas_per_unit = (float)t->ctas / (float)h.num_units;
  const int waves = ceil_div(t->ctas, h.num_units);
  t->wave_efficiency = (float)((double)t->ctas / ((double)waves * h.num_units));
  t->under_occupied = under;
  t->causal = causal ? 1 : 0;
  t->cost_steps = (int32_t)(grid.cost > 0x7FFFFFFFLL ? 0x7FFFFFFFLL : grid.cost);
  // Predicted time: the longest CTA's path at the per-unit share of the tensor peak against the compulsory HBM
  // traffic (Q, K, V read once, O written once) at the HBM bandwidth.
  if (h.peak_tflops > 0.0 && h.hbm_gbps > 0.0) {
    const double step_flops = 4.0 * tile_q * tile_kv * d;     // both products of one KV step
    const double t_tensor_us = (double)grid.cost * step_flops / (h.peak_tflops / h.num_units * 1e6);
    const double bytes = 2.0 * B * H * ((double)L + Lk) * d * h.elem_bytes;
    const double t_hbm_us = bytes / (h.hbm_gbps * 1e3);
    t->bound = t_hbm_us > t_tensor_us ? 1 : 0;
    t->predicted_us = (float)(t_hbm_us > t_tensor_us ? t_hbm_us : t_tensor_us);
  }
}

}  // namespace

extern "C" int attn_hw_desc_b200(attn_hw_desc* out) {
  if (!out) return ATTN_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  out->struct_bytes = (int32_t)sizeof(attn_hw_desc);
  out->num_units = 148;
  out->local_mem_bytes = 232448;  // 227 KB opt-in dynamic shared memory per block
  out->regs_per_unit = 65536;
  out->max_regs_per_thread = 255;
  out->simd_width = 32;
  out->acc_mem_lanes = 128;
  out->acc_mem_columns = 512;
  out->atom_m = 128;  // tcgen05.mma kind::f16, cta_group::1
  out->atom_n = 16;
  out->atom_k = 16;
  out->atom_n_max = 256;
  {
    // resident clusters of k CTAs with one CTA per SM (the occupancy query on a B200: 8 GPCs of unequal size)
    static const int kClusters[8] = {148, 74, 45, 33, 26, 22, 15, 15};
    for (int k = 0; k < 8; ++k) out->max_clusters[k] = kClusters[k];
  }
  out->elem_bytes = 2;
  out->cache_bytes = 126 << 20;   // L2
  // start and end of a CTA's work under each way of sharing out the key axis, in KV steps (measured on B200;
  // a KV step of 256 query rows x 128 keys x 128 takes about 1.7 us)
  out->ovh_whole_tile = 2;
  out->ovh_cluster = 5;
  out->ovh_workspace = 8;
  out->ovh_ranges = 12;
  out->ovh_persistent = 6;
  out->ovh_tile_change = 1;
  out->ovh_causal_ranges = 15;
  out->ovh_causal_cluster = 6;
  out->hbm_gbps = 7700.0;      // nominal (HGX B200)
  out->peak_tflops = 2250.0;   // nominal dense bf16: 8192 FLOP per clock per SM at 1.86 GHz
  return ATTN_OK;
}

extern "C" int attn_plan(const attn_hw_desc* desc, int B, int H, int L, int d, attn_tiles* out) {
  return attn_plan_ex(desc, B, H, L, d, 0, out);
}

extern "C" int attn_plan_ex(const attn_hw_desc* desc, int B, int H, int L, int d, int causal, attn_tiles* out) {
  return attn_internal::plan_qk(desc, B, H, L, L, d, causal, out);
}

extern "C" int attn_plan_qk(const attn_hw_desc* desc, int B, int H, int Lq, int Lk, int d, attn_tiles* out) {
  if (Lk <= 0) return ATTN_ERR_INVALID_ARG;
  return attn_internal::plan_qk(desc, B, H, Lq, Lk, d, 0, out);
}

int attn_internal::plan_qk(const attn_hw_desc* desc, int B, int H, int L, int Lk, int d, int causal, attn_tiles* out) {
  if (!desc || !out) return ATTN_ERR_INVALID_ARG;
  if (desc->struct_bytes != (int32_t)sizeof(attn_hw_desc)) return ATTN_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  out->binding_constraint = ATTN_BIND_SHAPE;
  if (B <= 0 || H <= 0 || L <= 0 || Lk <= 0 || d <= 0) return ATTN_OK;
  if (desc->num_units <= 0 || desc->local_mem_bytes <= 0 || desc->atom_m <= 0 || desc->atom_n <= 0 ||
      desc->atom_k <= 0 || desc->elem_bytes <= 0 || desc->simd_width <= 0 || desc->max_regs_per_thread <= 16)
    return ATTN_ERR_INVALID_ARG;
  if (desc->acc_mem_columns > 0)
    plan_tmem_machine(*desc, B, H, L, Lk, d, causal, out);
  else
    plan_register_machine(*desc, B, H, L, d, out);
  return ATTN_OK;
}

extern "C" size_t attn_workspace_bytes(const attn_tiles* t, int B, int H, int L, int d) {
  (void)B; (void)H; (void)L;
  if (!t || !t->feasible || t->n_q <= 0 || (t->ctas == t->tiles && !t->causal)) return 0;
  // 64 KB of arrival counters, then two slots per CTA (its first and its last piece of a Q tile) and
  // sub-tile: 128 x d fp32 un-normalised output + 128 (m, delta) pairs.
  const size_t per_sub = (size_t)128 * (size_t)d * 4 + (size_t)128 * 2 * 4;
  return (size_t)65536 + (size_t)2 * (size_t)t->ctas * (size_t)t->n_q * per_sub;
}

// Matrix product: the same derivation for the GEMM kernel's tile structure (Eq. 2: the local memory
// bounds the block tile through the ring depth; Eq. 3: the accumulator storage -- here tensor memory --
// bounds the rows one CTA can accumulate).
extern "C" int gemm_plan(const attn_hw_desc* desc, int batch, int M, int N, int K, gemm_tiles* out) {
  if (!desc || !out) return ATTN_ERR_INVALID_ARG;
  if (desc->struct_bytes != (int32_t)sizeof(attn_hw_desc)) return ATTN_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  if (batch <= 0 || M <= 0 || N <= 0 || K <= 0) return ATTN_ERR_INVALID_ARG;
  const attn_hw_desc& h = *desc;
  out->binding_constraint = ATTN_BIND_TMEM;
  if (h.acc_mem_columns <= 0 || h.atom_n_max <= 0 || h.elem_bytes <= 0) return ATTN_OK;   // not a tensor-memory machine
  // N of one instruction: the largest the atom allows, or half of it when the output is no wider than that
  const int tile_n = (N <= h.atom_n_max / 2) ? h.atom_n_max / 2 : h.atom_n_max;
  int n_sub = h.acc_mem_columns / h.atom_n_max;   // fp32 accumulator columns: one per output column and sub-tile
  if (n_sub > 2) n_sub = 2;
  if (n_sub < 1) return ATTN_OK;
  // Occupancy: if two-sub-tile blocks would leave compute units without a tile, one sub-tile per block
  // (twice as many blocks) is used instead -- the paper's "reduce tiles until occupancy is acceptable".
  if (n_sub == 2 && (long long)batch * ceil_div(M, 2 * h.atom_m) * ceil_div(N, tile_n) < h.num_units) n_sub = 1;
  const int tile_m = n_sub * h.atom_m;
  const int tile_k = 128 / h.elem_bytes;       // one swizzle row
  const int a_rows = (h.acc_mem_columns / h.atom_n_max >= 2 ? 2 : 1) * h.atom_m;   // the stage layout keeps room for two sub-tiles
  const int stage = (a_rows + tile_n) * tile_k * h.elem_bytes;
  const int staging = (a_rows / h.atom_m) * h.atom_m * 128;  // per sub-tile one 64-column chunk of the output rows
  int stages = (h.local_mem_bytes - staging - 1024) / stage;
  if (stages > 8) stages = 8;
  if (stages < 2) { out->binding_constraint = ATTN_BIND_SMEM; return ATTN_OK; }
  // CTA pairs: two CTAs as one 2 atom_m-row matrix unit, each staging its own rows of A and half of B's columns, with
  // as many accumulators as tensor memory holds so that a tile's epilogue runs under the next tile's products.
  // Taken when the machine can run pairs, tensor memory holds two accumulators, the output is wider than half the
  // atom's N, and the pairs occupy at least as many CTAs as the lone-CTA tiling would (the occupancy step).
  {
    const int pairs_max = h.max_clusters[1] < h.num_units / 2 ? h.max_clusters[1] : h.num_units / 2;
    const int pn = h.atom_n_max;
    const long long pt = (long long)batch * ceil_div(M, 2 * h.atom_m) * ceil_div(N, pn);
    const long long lone = (long long)batch * ceil_div(M, tile_m) * ceil_div(N, tile_n);
    const long long lone_ctas = lone < h.num_units ? lone : h.num_units;
    const long long pairs = pt < pairs_max ? pt : pairs_max;
    if (pairs_max > 0 && M > h.atom_m && N > pn / 2 && h.acc_mem_columns >= 2 * pn && 2 * pairs >= lone_ctas &&
        pt <= 0x3FFFFFFFLL) {
      const int pstage = (h.atom_m + pn / 2) * tile_k * h.elem_bytes;
      const int pstaging = 4 * h.atom_m * 128;    // per epilogue warp (4 lane quarters x 2 column halves) two 32-row chunks
      int pstages = (h.local_mem_bytes - pstaging - 1024) / pstage;
      if (pstages > 8) pstages = 8;
      if (pstages >= 2) {
        out->tile_m = 2 * h.atom_m;
        out->tile_n = pn;
        out->tile_k = tile_k;
        out->n_sub = 2;
        out->stages = pstages;
        out->smem_bytes = pstages * pstage + pstaging + 1024;
        out->tmem_columns = pow2_ceil((h.acc_mem_columns / pn) * pn);
        out->tiles = (int)pt;
        out->ctas = (int)(2 * pairs);
        const long long pwaves = (pt + pairs - 1) / pairs;
        // Last wave: the r tiles left after the whole waves run as 2 r half-width items if those fit one wave of pairs.
        const long long r = pt % pairs;
        const bool split = r > 0 && 2 * r <= pairs;
        out->tail_split = split ? (int32_t)r : 0;
        const double waves_eff = split ? (double)(pwaves - 1) + 0.64 : (double)pwaves;   // a half-width item: 0.64 of a tile
        out->wave_efficiency = (float)((double)pt / (waves_eff * pairs));
        out->cta_pair = 2;
        out->acc_buffers = h.acc_mem_columns / pn;
        out->feasible = 1;
        return ATTN_OK;
      }
    }
  }
  const long long tiles = (long long)batch * ceil_div(M, tile_m) * ceil_div(N, tile_n);
  if (tiles > 0x3FFFFFFFLL) return ATTN_OK;
  out->tile_m = tile_m;
  out->tile_n = tile_n;
  out->tile_k = tile_k;
  out->n_sub = n_sub;
  out->stages = stages;
  out->smem_bytes = stages * stage + staging + 1024;
  out->tmem_columns = pow2_ceil(n_sub * tile_n);
  out->tiles = (int)tiles;
  out->ctas = tiles < h.num_units ? (int)tiles : h.num_units;
  const long long waves = (tiles + out->ctas - 1) / out->ctas;
  out->wave_efficiency = (float)((double)tiles / ((double)waves * out->ctas));
  out->cta_pair = 1;
  out->acc_buffers = 1;
  out->feasible = 1;
  return ATTN_OK;
}
