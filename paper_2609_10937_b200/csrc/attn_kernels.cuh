// sm_100a kernels for the fused attention forward pass (Algorithm 1 of the
// paper: K/V tiles streamed through an online softmax; the score tile never
// leaves the chip).
//
//   attn_fwd_kernel        warp-specialised, pipelined: TMA producer warp ->
//                          shared-memory K/V ring -> one MMA-issuing thread
//                          (tcgen05.mma, S = Q K^T into tensor memory) ->
//                          two softmax warpgroups (one Q sub-tile each, one
//                          thread per row) -> P as bf16 back into tensor
//                          memory -> second tcgen05.mma (O += P V, A operand
//                          read from tensor memory) ; a correction warpgroup
//                          rescales O when the running maximum moved.
//                          d = 64: P has tensor-memory columns of its own, so the
//                          next step's Q K^T is issued as soon as the softmax
//                          warpgroup holds the scores in registers.
//                          CTAs walk equal ranges of the (Q tile, KV step) line.  Where
//                          several CTAs share a Q tile, all but the last to finish publish
//                          their partial (O, m, delta) and the last one merges them, per
//                          warp, with the merge operator of the online softmax.  Under a
//                          uniform key split the CTAs of a tile can run as one thread-block
//                          cluster: the partials then go from tensor memory straight into the
//                          merging CTA's shared memory (st.async), not through L2.
//   attn_fwd_simple_kernel the same algorithm with nothing overlapped; used to
//                          cross-check the pipelined kernel and the layouts.
//
// Every device-side wait is bounded: on expiry the CTA records an error word
// in g_attn_dev_status, raises a CTA-wide abort flag and all roles drain.
#pragma once

#include <cuda_bf16.h>

#include "ptx_sm100.cuh"

namespace attn {

using namespace sm100;

constexpr int kSub = 128;                 // rows of one Q sub-tile = tensor-memory lanes
constexpr long long kWaitLimitCycles = 1000000000LL;  // ~0.5 s at 1.9 GHz

// [0] error code (0 = none), [1] role<<24 | barrier<<16 | step, [2] CTA index, [3] spare
__device__ unsigned int g_attn_dev_status[4];

enum Role : uint32_t { kRoleLoad = 1, kRoleMma = 2, kRoleSoftmax = 3, kRoleCorrection = 4, kRoleSimple = 5 };
enum BarId : uint32_t { kBarQ = 1, kBarKvFull = 2, kBarKvEmpty = 3, kBarSFull = 4, kBarPFull = 5, kBarOFull = 6,
                        kBarAlpha = 7, kBarLoad = 8, kBarMma = 9, kBarSync = 10 };

// A CTA's abort flag (shared memory) and, beside it, where this launch reports an expired wait: four words of the
// caller's (attn_forward_ws) or g_attn_dev_status.  Every `abort_flag` pointer in the kernels points at `flag` of
// such a cell.
struct AbortCell {
  int flag;
  int pad;
  unsigned int* status;
};
__device__ __forceinline__ void abort_cell_init(AbortCell* c, unsigned int* status) {
  c->flag = 0;
  c->status = status ? status : g_attn_dev_status;
}
__device__ __noinline__ void report_timeout(uint32_t info, volatile int* abort_flag) {
  unsigned int* st = reinterpret_cast<const AbortCell*>(const_cast<const int*>(abort_flag))->status;
  if (atomicCAS(&st[0], 0u, 1u) == 0u) {
    st[1] = info;
    st[2] = blockIdx.x + gridDim.x * blockIdx.y;
    __threadfence();
  }
}

// Bounded mbarrier wait.  Returns false if the CTA aborted or the limit expired.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t info) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t it = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++it & 127u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        report_timeout(info, abort_flag);
        *abort_flag = 1;
        return false;
      }
    }
  }
}
// Same, for roles whose warps run warp-collective instructions afterwards: the outcome is made warp-uniform.
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t info) {
  return __all_sync(0xffffffffu, wait_bar(bar, parity, abort_flag, info) ? 1 : 0) != 0;
}
__device__ __forceinline__ uint32_t wait_info(uint32_t role, uint32_t bar, uint32_t step) {
  return (role << 24) | (bar << 16) | (step & 0xFFFFu);
}

// ---------------------------------------------------------------------------
// Matrix-product issue helpers (one thread).
// Q and K tiles: K-major, [rows][64] bf16 chunks with 128-byte swizzle, chunk c
// holds head-dimension columns [64c, 64c+64).  V tile: same storage, used as
// the MN-major B operand of the second product (N = head dimension).
// ---------------------------------------------------------------------------
// Descriptor words are split so that the issuing thread only adds a constant to the low
// word per k-step: low = (address >> 4) | (LBO >> 4) << 16, high = (SBO >> 4) | version | swizzle.
__device__ __forceinline__ uint64_t desc_from_words(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
__host__ __device__ constexpr uint32_t desc_hi_sw128(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
  return ((smem_addr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}

template <int D, int TKV>
__device__ __forceinline__ void issue_qk(uint32_t s_tmem, uint32_t q_smem, uint32_t k_smem) {
  constexpr uint32_t idesc = make_idesc_bf16(kSub, TKV, false);
  constexpr uint32_t hi = desc_hi_sw128(1024);
  const uint32_t a_lo = desc_lo(q_smem, 16), b_lo = desc_lo(k_smem, 16);
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const uint32_t chunk = ks >> 2, kin = ks & 3;
    const uint64_t a = desc_from_words(a_lo + ((chunk * (kSub * 128) + kin * 32) >> 4), hi);
    const uint64_t b = desc_from_words(b_lo + ((chunk * (TKV * 128) + kin * 32) >> 4), hi);
    if (ks == 0) umma_ss_c<0>(s_tmem, a, b, idesc);
    else umma_ss_c<1>(s_tmem, a, b, idesc);
  }
}
template <int D, int TKV>
__device__ __forceinline__ void issue_pv(uint32_t o_tmem, uint32_t p_tmem, uint32_t v_smem, bool accumulate,
                                         uint32_t lbo, uint32_t sbo, int ks_begin = 0, int ks_end = TKV / 16) {
  constexpr uint32_t idesc = make_idesc_bf16(kSub, D, true);
  const uint32_t hi = ((sbo >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
  const uint32_t b_lo = desc_lo(v_smem, lbo);
#pragma unroll
  for (int ks = 0; ks < TKV / 16; ++ks) {
    if (ks < ks_begin || ks >= ks_end) continue;
    // 16 key rows per step: two 8-row groups of 1024 bytes
    const uint64_t b = desc_from_words(b_lo + ((ks * 2048) >> 4), hi);
    if (ks == 0) umma_ts(o_tmem, p_tmem + ks * 8, b, idesc, accumulate ? 1u : 0u);
    else umma_ts_c<1>(o_tmem, p_tmem + ks * 8, b, idesc);
  }
}

struct FwdParams {
  int L;                   // sequence length
  int q_tiles;             // Q tiles per head = ceil(L / (NQ*128))
  int n_steps;             // KV steps of the whole key axis = ceil(L / TKV)
  int tiles;               // Q tiles in the whole problem = B * H * q_tiles
  int stages;              // ring depth
  int causal;              // 1: row i attends to keys 0..i only
  int ratio;               // Q-tile rows / TKV (1, 2 or 4)
  long long head_units;    // work units of one head (see tile_prefix)
  float scale_log2;        // log2(e) / sqrt(d)
  __nv_bfloat16* o;        // output, written directly when a result cannot go through the Q buffer
  float* ws;               // partial results of Q tiles shared by several CTAs
  unsigned int* counters;  // arrival counters of shared Q tiles; zero between launches
  unsigned int* status;    // four words that receive the record of an expired wait (nullptr: g_attn_dev_status)
  int cluster_k;           // > 1: the k CTAs of a Q tile are one thread-block cluster (uniform key split only)
  long long seg_skip;      // > 0: (gridDim.x - 1) * n_steps -- CTA c walks the whole tiles c, c + gridDim.x, ...
                           // < 0 (causal, clusters of k = -seg_skip): CTA c takes a share of the key steps of tile c / k
};

// Work decomposition.  A work unit is one KV step of one Q tile.  Q tile q of a head needs
// tile_steps(q) steps: all n_steps of them, or -- causal -- only those whose keys are not after the
// tile's last row, min(n_steps, (q+1)*ratio).  The units of the whole problem form one line (head
// major, Q tile, KV step); CTA c of G owns units [c*T/G, (c+1)*T/G) and walks them as segments, one per
// Q tile it touches.  A Q tile covered by several CTAs is merged by the last of them to finish.
__host__ __device__ __forceinline__ int tile_steps(int n_steps, int ratio, int causal, int q) {
  if (!causal) return n_steps;
  const long long s = (long long)(q + 1) * ratio;
  return s < n_steps ? (int)s : n_steps;
}
// Causal tiles are short at the start of a head, and starting and finishing a piece of a tile costs a CTA
// about as much as a few KV steps.  So that equal ranges of the line mean equal time, every causal tile is
// preceded on the line by kCausalTileCost units that stand for that cost: a CTA whose range covers them
// simply has fewer real steps.  (Non-causal tiles all have the same length: nothing to even out.)
constexpr int kCausalTileCost = 3;
// Units of Q tiles 0..q-1 of one head (closed form: a triangular number until the step count saturates;
// causal: plus the cost units of those tiles).
__host__ __device__ __forceinline__ long long tile_prefix(int n_steps, int ratio, int causal, int q) {
  if (!causal) return (long long)q * n_steps;
  long long qc = n_steps / ratio;
  if (qc > q) qc = q;
  return (long long)ratio * qc * (qc + 1) / 2 + (long long)(q - qc) * n_steps + (long long)kCausalTileCost * q;
}
__device__ __forceinline__ long long range_begin(long long c, long long T, long long G) { return (c * T) / G; }
__device__ __forceinline__ int cta_of_unit(long long u, long long T, long long G) {
  return (int)(((u + 1) * G - 1) / T);
}
template <bool V>
struct MaskTag { static constexpr bool value = V; };
struct Segment { int tile, q, j0, j1, n, bh, q_row0, seg, steps_t; bool full; long long unit0; };   // unit0: the tile's first real unit
// Q tile (head, index) that owns unit u, and the unit at which that tile starts.
// Next piece of the unit range [u, u_hi) that lies inside one Q tile; advances u and the segment counter.
// (Scalar arguments and straight-line code on purpose: the non-causal instantiation must stay as lean as
// it was before causal support existed -- measured, helper structs here cost several per cent.)
template <bool CAUSAL>
__device__ __forceinline__ bool next_segment(long long& u, long long u_hi, int& seg_ctr, int n_steps, int q_tiles,
                                             int ratio, long long head_units, int tile_rows, Segment& sg,
                                             long long skip) {
  if (u >= u_hi) return false;
  if constexpr (!CAUSAL) {
    sg.tile = (int)(u / n_steps);
    sg.j0 = (int)(u % n_steps);
    sg.bh = sg.tile / q_tiles;
    sg.q = sg.tile % q_tiles;
    sg.steps_t = n_steps;
    sg.unit0 = (long long)sg.tile * n_steps;
    const long long left = u_hi - u;
    sg.j1 = (left < (long long)(sg.steps_t - sg.j0)) ? sg.j0 + (int)left : sg.steps_t;
    sg.n = sg.j1 - sg.j0;
    u += sg.n + skip;                                   // skip > 0: whole tiles, every gridDim.x-th one
  } else if (skip < 0) {
    // causal, k = -skip CTAs per tile as one cluster (u = the CTA's index): the tile's own key steps are dealt out
    // in equal shares to its first min(k, steps) CTAs; the others have nothing to do (a tile's first rows have
    // fewer key steps than the cluster has CTAs)
    const int k = (int)-skip;
    const int t_lin = (int)(u / k), part = (int)(u % k);
    sg.bh = t_lin / q_tiles;
    sg.q = t_lin % q_tiles;
    sg.tile = t_lin;
    sg.steps_t = tile_steps(n_steps, ratio, 1, sg.q);
    const int parts = sg.steps_t < k ? sg.steps_t : k;
    if (part >= parts) return false;
    sg.unit0 = 0;
    sg.j0 = (int)((long long)part * sg.steps_t / parts);
    sg.j1 = (int)((long long)(part + 1) * sg.steps_t / parts);
    sg.n = sg.j1 - sg.j0;
    u = u_hi;
  } else {
    for (;;) {
      sg.bh = (int)(u / head_units);
      const long long r = u - (long long)sg.bh * head_units;
      int lo = 0, hi = q_tiles - 1;                     // largest q with tile_prefix(q) <= r
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tile_prefix(n_steps, ratio, 1, mid) <= r) lo = mid; else hi = mid - 1;
      }
      sg.q = lo;
      sg.tile = sg.bh * q_tiles + lo;
      const long long start = (long long)sg.bh * head_units + tile_prefix(n_steps, ratio, 1, lo);   // cost units first
      sg.unit0 = start + kCausalTileCost;
      sg.steps_t = tile_steps(n_steps, ratio, 1, lo);
      long long end = sg.unit0 + sg.steps_t;
      if (end > u_hi) end = u_hi;
      const long long x0 = u - sg.unit0, x1 = end - sg.unit0;   // negative inside the cost units
      sg.j0 = x0 > 0 ? (int)x0 : 0;
      sg.j1 = x1 > 0 ? (int)x1 : 0;
      sg.n = sg.j1 - sg.j0;
      u = end;
      if (sg.n > 0) break;
      if (u >= u_hi) return false;                      // the range ended inside a tile's cost units
    }
  }
  sg.full = (sg.j0 == 0 && sg.j1 == sg.steps_t);
  sg.q_row0 = sg.q * tile_rows;
  sg.seg = seg_ctr++;
  return true;
}

// Shared-memory footprint helpers (host and device agree through these).
template <int D, int TKV, int NQ>
struct FwdSmem {
  static constexpr int kQBytes = NQ * kSub * D * 2;
  static constexpr int kStageBytes = TKV * D * 2;
  static constexpr int kOutBytes = NQ * kSub * 128;    // per softmax warpgroup one [128 rows][64 columns] bf16 output chunk
  static constexpr int kMiscBytes = 3072;
  __host__ __device__ static constexpr int total(int stages) {
    return kQBytes + stages * kStageBytes + kOutBytes + kMiscBytes;
  }
};

constexpr int kMaxStages = 8;
constexpr float kRescaleThreshold = 8.0f;   // log2 units: P stays below 2^8
constexpr float kDominanceFactor = 16.0f;   // a new maximum heavier than delta/16 moves the reference
constexpr int kCounterBytes = 65536;   // head of the workspace: 16384 arrival counters

struct FwdMisc {               // lives in the last 3072 bytes of dynamic shared memory
  float alpha[2][2][kSub];     // [sub-tile][step parity][row] rescale factor
  uint64_t q_full[2];          // one per Q sub-tile: the first product starts when sub-tile 0 and K_0 are in
  uint64_t kv_full[kMaxStages];
  uint64_t kv_empty[kMaxStages];
  uint64_t s_full[2];
  uint64_t p_full[2];          // first half of P written and O rescaled
  uint64_t p_half[2];          // second half of P written
  uint64_t o_full[2];
  uint64_t alpha_full[2];
  uint64_t q_empty;            // every product that reads the Q tile of a segment has finished
  uint64_t o_free[2];          // the epilogue of a segment has read its O accumulator
  uint64_t s_free[2];          // d = 64: the softmax warpgroup holds the step's scores in registers
  uint64_t peers_ready;        // cluster: every other CTA of the tile has finished with its K/V ring
  uint64_t data_ready[8][2];   // cluster: the other CTAs' parts of softmax warp w's rows have landed ([1]: columns 64..)
  AbortCell abort;
  uint32_t tmem_slot;
};
static_assert(sizeof(FwdMisc) <= 3072, "misc region too large");

// Workspace layout for split keys: per (CTA, sub-tile): O[D/4][128][4] fp32, m[128], delta[128].
__host__ __device__ constexpr size_t ws_floats_per_sub(int d) { return (size_t)kSub * d + 2 * kSub; }

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// max of s[B..E) as one dependency chain of 3-input maxima
template <int B, int E>
__device__ __forceinline__ float chain_max(const uint32_t* s) {
  float m = __uint_as_float(s[B]);
#pragma unroll
  for (int k = B + 1; k + 1 < E; k += 2) m = max3(m, __uint_as_float(s[k]), __uint_as_float(s[k + 1]));
  if (((E - B - 1) & 1) != 0) m = fmaxf(m, __uint_as_float(s[E - 1]));
  return m;
}
// Constants of the exponential evaluation, packed once per thread.
struct ExpConsts {
  uint64_t scale2, magic2, c3, c2, c1, c0;
};
__device__ __forceinline__ ExpConsts make_exp_consts(float scale) {
  ExpConsts k;
  k.scale2 = pack_f32x2(scale, scale);
  k.magic2 = pack_f32x2(12582912.0f, 12582912.0f);          // 1.5 * 2^23: adding it rounds to an integer
  // minimax cubic for 2^f on [-0.5, 0.5], relative error 7.6e-5 (bf16 rounding of P is 2e-3)
  k.c3 = pack_f32x2(0.055168043822050095f, 0.055168043822050095f);
  k.c2 = pack_f32x2(0.24260213971138f, 0.24260213971138f);
  k.c1 = pack_f32x2(0.6932607889175415f, 0.6932607889175415f);
  k.c0 = pack_f32x2(0.9999286532402039f, 0.9999286532402039f);
  return k;
}
// exp2 of a packed pair on the FMA/ALU pipes (no MUFU): x = n + f with n integer, f in [-0.5, 0.5];
// 2^f by the cubic, 2^n by adding n to the exponent field.  x is clamped at -126 (result ~1e-38).
__device__ __forceinline__ void exp2_poly_pair(uint64_t x2, const ExpConsts& k, float& e0, float& e1) {
  float x0, x1;
  unpack_f32x2(x2, x0, x1);
  x0 = fmaxf(x0, -126.0f);
  x1 = fmaxf(x1, -126.0f);
  const uint64_t xc = pack_f32x2(x0, x1);
  const uint64_t r2 = add_f32x2(xc, k.magic2);
  const uint64_t n2 = sub_f32x2(r2, k.magic2);
  const uint64_t f2 = sub_f32x2(xc, n2);
  uint64_t p2 = fma_f32x2(f2, k.c3, k.c2);
  p2 = fma_f32x2(p2, f2, k.c1);
  p2 = fma_f32x2(p2, f2, k.c0);
  float p0, p1, r0, r1;
  unpack_f32x2(p2, p0, p1);
  unpack_f32x2(r2, r0, r1);
  e0 = __int_as_float(__float_as_int(p0) + (__float_as_int(r0) << 23));
  e1 = __int_as_float(__float_as_int(p1) + (__float_as_int(r1) << 23));
}
// P = exp2(s * scale - m) for 32 consecutive scores, packed to bf16 pairs; adds them to the packed
// partial sums.  Of every eight pairs, kPolyPairsPer8 are evaluated by the polynomial and the rest
// by MUFU ex2, which balances the two pipes (MUFU alone would take as long as the matrix products).
// Two of eight measured best on B200: more polynomial work costs issue slots that the other warps
// of the scheduler partition (and the MMA-issuing warp) need.
constexpr int kPolyPairsPer8 = 2;
template <int kPolyPairs>
__device__ __forceinline__ void exp_chunk(const uint32_t* s, const ExpConsts& k, uint64_t neg_m2, uint64_t& sum2,
                                          uint32_t (&pk)[16]) {
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[2 * j]), __uint_as_float(s[2 * j + 1])), k.scale2, neg_m2);
    float e0, e1;
    if ((j & 7) < kPolyPairs) {
      exp2_poly_pair(x2, k, e0, e1);
    } else {
      float x0, x1;
      unpack_f32x2(x2, x0, x1);
      e0 = ex2_approx(x0);
      e1 = ex2_approx(x1);
    }
    sum2 = add_f32x2(sum2, pack_f32x2(e0, e1));
    pk[j] = pack_bf16x2(e0, e1);
  }
}
// 32 fp32 values of one output row -> bf16, written into a 128-byte-swizzled [128][64] staging chunk.
__device__ __forceinline__ void stage_row_chunk(uint32_t stage_out, int c, int row, const float (&val)[32]) {
  const uint32_t chunk_base = stage_out + (c >> 1) * (kSub * 128) + row * 128;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) w[e] = pack_bf16x2(val[u * 8 + 2 * e], val[u * 8 + 2 * e + 1]);
    const uint32_t unit = (uint32_t)((c & 1) * 4 + u) ^ (uint32_t)(row & 7);   // 128-byte swizzle
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(chunk_base + unit * 16), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
  }
}

template <int D, int TKV, int NQ, bool CAUSAL, bool EAGER, bool CLUSTER = false>
__global__ void __launch_bounds__(512, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                const FwdParams p) {
  static_assert(D == 64 || D == 128, "head dimension");
  static_assert(TKV == 64 || TKV == 128, "KV tile");
  constexpr int KCH = D / 64;                         // 64-column chunks per row
  constexpr int S_COLS = TKV;                         // fp32 score columns per sub-tile
  constexpr int O_COL0 = NQ * S_COLS;                 // O accumulators follow the score buffers
  constexpr int NCH = TKV / 32;                       // 32-column chunks of one score row
  constexpr int kPoly = kPolyPairsPer8;             // polynomial pairs per 8
  // d = 64 leaves tensor memory for P next to S and O.  The score buffer is then free as soon as the softmax
  // warpgroup has read it into registers, and the next step's Q K^T runs during this step's exponentials instead
  // of after this step's P V.  (d = 128 fills tensor memory: P overwrites the front of the score buffer.)
  constexpr bool kSplitP = (D == 64) && NQ == 2 && (NQ * (S_COLS + D) + NQ * (TKV / 2) <= 512);
  constexpr int P_COL0 = NQ * (S_COLS + D);           // kSplitP: bf16 P, TKV / 2 columns per sub-tile
  constexpr uint32_t kPartBytes = 32 * D * 4 + 256;   // cluster: one warp's part -- O of 32 rows, then m and delta
  constexpr int kTmemUsed = NQ * (S_COLS + D) + (kSplitP ? NQ * (TKV / 2) : 0);
  constexpr int TMEM_COLS = (kTmemUsed <= 32) ? 32 : (kTmemUsed <= 64) ? 64 : (kTmemUsed <= 128) ? 128
                          : (kTmemUsed <= 256) ? 256 : 512;
  using SM = FwdSmem<D, TKV, NQ>;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t q_smem = smem_base;
  const uint32_t ring_smem = smem_base + SM::kQBytes;
  const uint32_t out_smem = ring_smem + p.stages * SM::kStageBytes;   // output staging of segments that are not the CTA's last
  FwdMisc* misc = reinterpret_cast<FwdMisc*>(smem_raw + SM::kQBytes + p.stages * SM::kStageBytes + SM::kOutBytes);
  volatile int* abort_flag = &misc->abort.flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // Work assignment (see range_begin): consecutive CTAs work on neighbouring key ranges of the same
  // head, so K/V are shared through L2.
  const int cta = blockIdx.x;
  const long long G = gridDim.x;
  const long long T = p.head_units * (p.tiles / p.q_tiles);
  // (seg_skip > 0: one CTA per tile executed by a persistent grid -- CTA c takes the whole tiles c, c + G, c + 2G, ...,
  // the order in which the hardware would have started one CTA per tile, without a CTA's start and end per tile)
  // (seg_skip < 0, causal: two CTAs per tile -- the "range" is the CTA's index)
  const long long u_lo = p.seg_skip > 0 ? (long long)cta * p.n_steps : p.seg_skip < 0 ? (long long)cta : range_begin(cta, T, G);
  const long long u_hi = p.seg_skip > 0 ? T : p.seg_skip < 0 ? (long long)cta + 1 : range_begin(cta + 1, T, G);

  // CLUSTER: number of CTAs of this CTA's cluster that have key steps (all of them, except for short causal tiles)
  int cl_parts = p.cluster_k;
  if constexpr (CLUSTER && CAUSAL) {
    const int st = tile_steps(p.n_steps, p.ratio, 1, (cta / p.cluster_k) % p.q_tiles);
    if (st < cl_parts) cl_parts = st;
  }
  (void)cl_parts;
  if (threadIdx.x == 0) {
    abort_cell_init(&misc->abort, p.status);
    if (smem_base & 1023u) {                 // swizzled tiles need 1024-byte alignment
      report_timeout(wait_info(kRoleLoad, 0, 0xFFFF), abort_flag);
      misc->abort.flag = 1;
    }
    mbar_init(smem_u32(&misc->q_full[0]), 1);
    mbar_init(smem_u32(&misc->q_full[1]), 1);
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(smem_u32(&misc->kv_full[s]), 1);
      mbar_init(smem_u32(&misc->kv_empty[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&misc->s_full[i]), 1);
      mbar_init(smem_u32(&misc->p_full[i]), 2 * kSub);   // softmax rows + correction rows
      mbar_init(smem_u32(&misc->p_half[i]), kSub);
      mbar_init(smem_u32(&misc->o_full[i]), 1);
      mbar_init(smem_u32(&misc->alpha_full[i]), kSub);
      mbar_init(smem_u32(&misc->o_free[i]), kSub);
      mbar_init(smem_u32(&misc->s_free[i]), kSub);
    }
    mbar_init(smem_u32(&misc->q_empty), 1);
    if constexpr (CLUSTER) {
      {
        // Partials travel through distributed shared memory (see the end of a segment).  The merging warps of
        // this CTA -- warp w merges if w mod k is this CTA's rank -- expect the parts of the k-1 other CTAs.
        mbar_init(smem_u32(&misc->peers_ready), cl_parts - 1);
        for (int w = 0; w < 4 * NQ; ++w) {
          mbar_init(smem_u32(&misc->data_ready[w][0]), 1);
          mbar_init(smem_u32(&misc->data_ready[w][1]), 1);
          if (w % cl_parts == cta % p.cluster_k) {
            // first the statistics and columns 0..63 of every part, then (d = 128) columns 64..127
            mbar_arrive_expect_tx(smem_u32(&misc->data_ready[w][0]), (uint32_t)(cl_parts - 1) * (32 * 64 * 4 + 256));
            if (KCH == 2) mbar_arrive_expect_tx(smem_u32(&misc->data_ready[w][1]), (uint32_t)(cl_parts - 1) * (32 * 64 * 4));
          }
        }
      }
    }
    fence_mbar_init();
    prefetch_tmap(&tm_q);
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
    prefetch_tmap(&tm_o);
  }
  if (warp == 15) {
    tmem_alloc(smem_u32(&misc->tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // every CTA's barriers must exist before a peer touches them: arrive here, wait where the first peer access is
  bool cluster_waited = false;                           // this thread has completed the wait of that barrier
  (void)cluster_waited;
  if constexpr (CLUSTER) cluster_arrive();
  const uint32_t tmem_base = misc->tmem_slot;
  const bool run = (*abort_flag == 0) && u_hi > u_lo;

  // Every role walks the same list of segments (see next_segment); `g` counts KV steps over all
  // segments of this CTA and gives the parity of the per-step barriers.
  if (warp < 4 * NQ) {
    // ===================================================== softmax warpgroup
    setmaxnreg_inc<(NQ == 2) ? 192 : 232>();
    const int i = warp >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t s_tmem = lane_base + i * S_COLS;
    const uint32_t p_tmem = kSplitP ? lane_base + P_COL0 + i * (TKV / 2) : s_tmem;   // else P aliases the front of S
    const uint32_t o_tmem = lane_base + O_COL0 + i * D;
    const uint32_t bar_s = smem_u32(&misc->s_full[i]);
    const uint32_t bar_p = smem_u32(&misc->p_full[i]);
    const uint32_t bar_h = smem_u32(&misc->p_half[i]);
    const uint32_t bar_a = smem_u32(&misc->alpha_full[i]);
    const float scale = p.scale_log2;
    const ExpConsts ek = make_exp_consts(scale);
    const size_t per_sub = ws_floats_per_sub(D);
    const int kv_tail = p.L % TKV;                     // valid keys in a ragged last KV tile (0: none ragged)
    bool ok = run;
    uint32_t g = 0;
    if (ok) {
      long long u = u_lo;
      int seg_ctr = 0;
      Segment sg;
      while (ok && next_segment<CAUSAL>(u, u_hi, seg_ctr, p.n_steps, p.q_tiles, p.ratio, p.head_units, NQ * kSub, sg, p.seg_skip)) {
        const int tile = sg.tile, j0 = sg.j0, j1 = sg.j1, n = sg.n, bh = sg.bh, q_row0 = sg.q_row0, seg = sg.seg;
        (void)tile; (void)j0; (void)j1; (void)bh; (void)q_row0; (void)seg;
      float m_run = -INFINITY, delta = 0.f;
      const uint32_t g_seg0 = g;                         // first step of this segment
      (void)g_seg0;
      // One KV step of this sub-tile.  The masked variant (a ragged last KV tile, or a causal step that
      // reaches past the sub-tile's first row) is compiled separately so that the common step pays
      // nothing for it; `lim` is the last key column of this step the thread's row may attend to.
      auto softmax_step = [&](auto mask_tag, int lim) __attribute__((always_inline)) -> bool {
        constexpr bool kMasked = decltype(mask_tag)::value;
        if (!wait_bar_warp(bar_s, g & 1, abort_flag, wait_info(kRoleSoftmax, kBarSFull, g))) return false;
        tc_fence_after();
        uint32_t s[TKV];
        // load the row in two halves: the maximum of the first half is taken while the second is in flight
#pragma unroll
        for (int c = 0; c < NCH / 2; ++c) tmem_ld32_nowait(s_tmem + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
#pragma unroll
        for (int c = 0; c < NCH / 2; ++c) tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
#pragma unroll
        for (int c = NCH / 2; c < NCH; ++c) tmem_ld32_nowait(s_tmem + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        // Masked keys -- past the end of the sequence (zero-filled by TMA, which would give them score 0
        // and weight exp(0 - m) > 0) or after the query's position (causal) -- get score -inf, never zero.
        if constexpr (kMasked) {
#pragma unroll
          for (int k = 0; k < TKV / 2; ++k)
            if (k > lim) s[k] = 0xFF800000u;
        }
        const float mx_a = fmaxf(fmaxf(chain_max<0, TKV / 8>(s), chain_max<TKV / 8, TKV / 4>(s)),
                                 fmaxf(chain_max<TKV / 4, 3 * TKV / 8>(s), chain_max<3 * TKV / 8, TKV / 2>(s)));
#pragma unroll
        for (int c = NCH / 2; c < NCH; ++c) tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        if constexpr (kSplitP) {
          tc_fence_before();
          mbar_arrive(smem_u32(&misc->s_free[i]));         // the scores are in registers: the buffer may be overwritten
        }
        if constexpr (kMasked) {
#pragma unroll
          for (int k = TKV / 2; k < TKV; ++k)
            if (k > lim) s[k] = 0xFF800000u;
        }
        const float mx_b = fmaxf(fmaxf(chain_max<TKV / 2, 5 * TKV / 8>(s), chain_max<5 * TKV / 8, 3 * TKV / 4>(s)),
                                 fmaxf(chain_max<3 * TKV / 4, 7 * TKV / 8>(s), chain_max<7 * TKV / 8, TKV>(s)));
        const float mx = fmaxf(mx_a, mx_b);
        // Lazy rescale.  The reference maximum m_run moves (and O, delta are rescaled by alpha) only
        //  (a) when the row maximum grew by more than kRescaleThreshold (log2 units), which bounds
        //      P = exp2(s - m_run) by 2^threshold, or
        //  (b) when the new maximum is a dominant key: its weight 2^gap is more than 1/16 of the
        //      running denominator.  Then P of that key is exactly 1 and carries no bf16 rounding
        //      error; a stale reference would put the rounding error of the heaviest weight on the
        //      whole row.  For flat score distributions (b) stops firing after the first few tiles.
        // Otherwise the reference stays stale, which changes nothing in exact arithmetic because
        // delta and O carry the same factor.  First step: m_run = -inf, gap = +inf, alpha = 0.
        // (masked steps can leave a row with no admissible key yet: keep the reference finite)
        const float m_cand = kMasked ? fmaxf(fmaxf(m_run, mx * scale), -1e30f) : fmaxf(m_run, mx * scale);
        const float gap = m_cand - m_run;
        const float shrink = ex2_approx(-gap);             // 2^-gap: the rescale factor if the reference moves
        const bool move = (gap > kRescaleThreshold) || (gap > 0.f && kDominanceFactor > delta * shrink);
        const float m_new = move ? m_cand : m_run;
        const float alpha = move ? shrink : 1.0f;
        if constexpr (kSplitP) {
          // P has its own columns: the previous step's P V must have read them before they are overwritten (it
          // finished long ago as a rule).  The wait stands BEFORE this step's arrivals on purpose.  With P in its
          // own columns the next scores are produced before this step's P V is issued, so without it a fast warp
          // (softmax or, through alpha_full, correction) could make its arrival of step g+1 on alpha_full / p_full
          // while a slow warp has not made that of step g; arrivals are anonymous, so the barrier's phase g would
          // complete on the wrong 128 / 256 arrivals.  Here every arrival of step g comes after P V(g-1) has
          // finished, hence after every thread's arrivals of step g-1.  (The segment's first step is covered by
          // the wait for the last P V at the end of the previous segment.)
          misc->alpha[i][g & 1][row] = alpha;
          if (g != g_seg0) {
            if (!wait_bar_warp(smem_u32(&misc->o_full[i]), (g - 1) & 1, abort_flag, wait_info(kRoleSoftmax, kBarOFull, 0x4000 | g))) return false;
            tc_fence_after();
          }
        } else {
          misc->alpha[i][g & 1][row] = alpha;
        }
        mbar_arrive(bar_a);
        const uint64_t neg_m2 = pack_f32x2(-m_new, -m_new);
        uint64_t sum_a = 0ull, sum_b = 0ull;               // packed (0.f, 0.f)
        uint32_t pk[16];
        // first half of the row: the second product may start on it while the rest is computed
#pragma unroll
        for (int c = 0; c < NCH / 2; ++c) {
          exp_chunk<kPoly>(&s[c * 32], ek, neg_m2, sum_a, pk);
          tmem_st16(p_tmem + c * 16, pk);
        }
        uint32_t pk2[16];
        exp_chunk<kPoly>(&s[(NCH / 2) * 32], ek, neg_m2, sum_b, pk2);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p);
        tmem_st16(p_tmem + (NCH / 2) * 16, pk2);
#pragma unroll
        for (int c = NCH / 2 + 1; c < NCH; ++c) {
          exp_chunk<kPoly>(&s[c * 32], ek, neg_m2, sum_b, pk);
          tmem_st16(p_tmem + c * 16, pk);
        }
        float sa0, sa1, sb0, sb1;
        unpack_f32x2(sum_a, sa0, sa1);
        unpack_f32x2(sum_b, sb0, sb1);
        delta = delta * alpha + ((sa0 + sa1) + (sb0 + sb1));
        m_run = m_new;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_h);
              return true;
      };
      // Causal: the steps before the sub-tile's diagonal (and before a ragged last key tile) need no mask and run in
      // a loop of their own that holds nothing but the common step; the few masked steps of the segment follow.
      int jj = 0;
      if constexpr (CAUSAL && !CLUSTER) {
        int first_masked = (q_row0 + i * kSub) / TKV;          // first step that reaches past the sub-tile's first row
        if (kv_tail != 0 && p.n_steps - 1 < first_masked) first_masked = p.n_steps - 1;
        int n_plain = first_masked - j0;
        n_plain = n_plain < 0 ? 0 : (n_plain > n ? n : n_plain);
        for (; ok && jj < n_plain; ++jj, ++g) ok = softmax_step(MaskTag<false>{}, TKV - 1);
      }
      for (; ok && jj < n; ++jj, ++g) {
        const int j = j0 + jj;
        const bool ragged = (kv_tail != 0) && (j == p.n_steps - 1);
        const bool diagonal = CAUSAL && ((j + 1) * TKV - 1 > q_row0 + i * kSub);   // warp-uniform
        if (ragged || diagonal) {
          int lim = ragged ? kv_tail - 1 : TKV - 1;
          if (CAUSAL) {
            const int cl = q_row0 + i * kSub + row - j * TKV;     // may be negative: nothing admissible
            if (cl < lim) lim = cl;
          }
          ok = softmax_step(MaskTag<true>{}, lim);
        } else {
          ok = softmax_step(MaskTag<false>{}, TKV - 1);
        }
      }
      // ----------------------------------------------------- end of segment
      // Each warp finishes its own 32 rows without meeting the other warps of its warpgroup.
      if constexpr (CLUSTER) {
        // The peers' barriers exist (arrival at kernel start).  Two parts: what a CTA receives lands in its Q
        // buffer, which is dead one step before the end -- its peers may be told so right away.
        if (ok) {
          cluster_wait();
          cluster_waited = true;
          if (cl_parts == 2 && warp == 0) {
            ok = wait_bar_warp(smem_u32(&misc->q_empty), 0, abort_flag, wait_info(kRoleSoftmax, kBarQ, 0x2000));
            if (ok && lane < 2 && lane != cta % p.cluster_k) mbar_arrive_peer(map_to_cta(smem_u32(&misc->peers_ready), lane));
          }
        }
      }
      if (ok) ok = wait_bar_warp(smem_u32(&misc->o_full[i]), (g - 1) & 1, abort_flag, wait_info(kRoleSoftmax, kBarOFull, g));
      if (!ok) break;
      tc_fence_after();
      const int wq = warp & 3;                               // which 32 rows of the sub-tile
      // This warp's staging: [32 rows][64 columns] bf16 chunks.  Before the CTA's last segment there is one
      // (the next Q tile may already be arriving in the Q buffer) and the two halves of a 128-wide row take
      // turns; for a whole tile on the last segment the warp's slice of its sub-tile's dead Q buffer holds all
      // halves at once (when the last segment ends in a merge, that slice receives the other parts instead).
      const bool last_seg = (u >= u_hi);                     // u was advanced past this segment already
      const bool q_stage = last_seg && sg.full;
      const uint32_t stage_w = q_stage ? q_smem + warp * (KCH * 4096) : out_smem + warp * 4096;
      // 64 normalised columns of this warp's rows -> memory through the staging chunk and a TMA store
      // (coalesced; rows past the end of the sequence are clipped by the tensor map).
      auto store_half = [&](int h, const float (&v0)[32], const float (&v1)[32]) {
        const uint32_t dst = q_stage ? stage_w + h * 4096 : stage_w;
        stage_row_chunk(dst, 0, lane, v0);
        stage_row_chunk(dst, 1, lane, v1);
        if (q_stage && h < KCH - 1) return;
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (q_stage) {
#pragma unroll
            for (int hh = 0; hh < KCH; ++hh)
              tma_store_3d(&tm_o, stage_w + hh * 4096, hh * 64, q_row0 + i * kSub + wq * 32, bh);
          } else {
            tma_store_3d(&tm_o, stage_w, h * 64, q_row0 + i * kSub + wq * 32, bh);
          }
          tma_store_commit();
          tma_store_wait_read();
        }
        __syncwarp();                                        // the staging chunk may be written again
      };
      if (sg.full) {
        // The whole Q tile was processed here: normalise and store.
        const float inv = 1.0f / delta;
#pragma unroll 1
        for (int h = 0; h < KCH; ++h) {
          uint32_t r0[32], r1[32];
          float v0[32], v1[32];
          tmem_ld32_nowait(o_tmem + h * 64, r0);
          tmem_ld32_nowait(o_tmem + h * 64 + 32, r1);
          tmem_ld_fence(r0);
          tmem_ld_fence(r1);
          if (h == KCH - 1) {
            tc_fence_before();
            mbar_arrive(smem_u32(&misc->o_free[i]));         // O may be overwritten by the next segment
          }
#pragma unroll
          for (int k = 0; k < 32; ++k) { v0[k] = __uint_as_float(r0[k]) * inv; v1[k] = __uint_as_float(r1[k]) * inv; }
          store_half(h, v0, v1);
        }
      } else {
        // Part of a Q tile shared with other CTAs (those whose ranges meet the tile's units; the first of
        // them owns the tile's counters).  Per warp: one of the tile's CTAs merges (see "Who merges" below:
        // counter A orders the CTAs by when they finished their key range); all but that one publish their un-normalised partial (O, m, delta) -- slots 2*cta and
        // 2*cta+1: a CTA has at most two partial pieces, its first and its last segment -- and signal that on
        // counter B without waiting; the merging one keeps its part in tensor memory, waits for B and merges
        // all parts in ascending key order (the merge operator of the online softmax), so the result does
        // not depend on who merges.
        if constexpr (CLUSTER) {
          {
            const int mine = cta % p.cluster_k;
            // Uniform key split with the tile's k CTAs as one thread-block cluster (rank = `mine`): the parts go
            // from tensor memory straight into the merging CTA's shared memory -- no trip through L2, no flag
            // in global memory.  Roles as below ("Who merges"): softmax warp w belongs to rank w mod k.  The
            // landing areas lie in the K/V ring, which is dead in a CTA once the last product of both its
            // sub-tiles has finished; every CTA tells its peers when that is so.
            const int k = cl_parts;
            const int owner = warp % k, ms = warp / k;
            // Two parts: what a CTA receives fits its Q buffer (O) and the idle staging chunks of its publishing
            // warps (m, delta), and the Q buffer is dead one step before the end.  More parts: the K/V ring,
            // dead once the last product of the other sub-tile has finished too.
            const bool q_land = (k == 2);
            if (!q_land) {
              if (NQ == 2 &&
                  !wait_bar_warp(smem_u32(&misc->o_full[1 - i]), (g - 1) & 1, abort_flag, wait_info(kRoleSoftmax, kBarOFull, 0x2000 | g))) { ok = false; break; }
              if (warp == 0 && lane < k && lane != mine) mbar_arrive_peer(map_to_cta(smem_u32(&misc->peers_ready), lane));
            }
            // landing area of part `src` (index among the k-1 other parts) of this warp's rows, as local addresses
            auto o_land = [&](int src) -> uint32_t {
              return q_land ? q_smem + (uint32_t)ms * (32 * D * 4) : ring_smem + (uint32_t)(ms * (k - 1) + src) * kPartBytes;
            };
            auto s_land = [&](int src) -> uint32_t {
              return q_land ? out_smem + (uint32_t)(warp ^ 1) * 4096 : o_land(src) + 32 * D * 4;
            };
            if (owner != mine) {
              if (!wait_bar_warp(smem_u32(&misc->peers_ready), 0, abort_flag, wait_info(kRoleSoftmax, kBarSync, 0x6000 | (uint32_t)warp))) { ok = false; break; }
              const int src = mine < owner ? mine : mine - 1;
              const uint32_t land = map_to_cta(o_land(src), owner), sland = map_to_cta(s_land(src), owner);
              const uint32_t rbar0 = map_to_cta(smem_u32(&misc->data_ready[warp][0]), owner);
              st_peer_f1(sland + lane * 4, m_run, rbar0);
              st_peer_f1(sland + 128 + lane * 4, delta, rbar0);
#pragma unroll 1
              for (int hcol = 0; hcol < D / 64; ++hcol) {
                const uint32_t rbar = rbar0 + hcol * 8;
                uint32_t r[64];
                tmem_ld32_nowait(o_tmem + hcol * 64, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld32_nowait(o_tmem + hcol * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
                tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[32]));
#pragma unroll
                for (int gq = 0; gq < 16; ++gq)
                  st_peer_f4(land + (uint32_t)((hcol * 16 + gq) * 32 + lane) * 16, __uint_as_float(r[gq * 4]),
                             __uint_as_float(r[gq * 4 + 1]), __uint_as_float(r[gq * 4 + 2]), __uint_as_float(r[gq * 4 + 3]), rbar);
              }
              tc_fence_before();
              mbar_arrive(smem_u32(&misc->o_free[i]));
            } else {
              if (!wait_bar_warp(smem_u32(&misc->data_ready[warp][0]), 0, abort_flag, wait_info(kRoleSoftmax, kBarSync, 0x5000 | (uint32_t)warp))) { ok = false; break; }
              // part q (ascending key order) of this warp's rows: own part in tensor memory, the others landed
              auto part = [&](int q) -> const float* {           // O of part q: [column / 4][lane] float4
                return reinterpret_cast<const float*>(smem_raw + (o_land(q < mine ? q : q - 1) - smem_base));
              };
              auto stat = [&](int q) -> const float* {           // m[32], delta[32] of part q
                return reinterpret_cast<const float*>(smem_raw + (s_land(q < mine ? q : q - 1) - smem_base));
              };
              float m_all = m_run;
              for (int q = 0; q < k; ++q)
                if (q != mine) m_all = fmaxf(m_all, stat(q)[lane]);
              float d_all = 0.f;
              for (int q = 0; q < k; ++q) {
                const float m_q = (q == mine) ? m_run : stat(q)[lane];
                const float d_q = (q == mine) ? delta : stat(q)[32 + lane];
                d_all += d_q * exp2f(m_q - m_all);
              }
              const float inv = 1.0f / d_all;
#pragma unroll 1
              for (int h = 0; h < KCH; ++h) {
                if (h == 1 &&
                    !wait_bar_warp(smem_u32(&misc->data_ready[warp][1]), 0, abort_flag, wait_info(kRoleSoftmax, kBarSync, 0x5800 | (uint32_t)warp))) { ok = false; break; }
                float val[64];
#pragma unroll
                for (int e = 0; e < 64; ++e) val[e] = 0.f;
                for (int q = 0; q < k; ++q) {
                  if (q == mine) {
                    const float w = exp2f(m_run - m_all);
                    uint32_t r[64];
                    tmem_ld32_nowait(o_tmem + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                    tmem_ld32_nowait(o_tmem + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
                    tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                    tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[32]));
#pragma unroll
                    for (int e = 0; e < 64; ++e) val[e] += w * __uint_as_float(r[e]);
                  } else {
                    const float* b = part(q);
                    const float w = exp2f(stat(q)[lane] - m_all);
#pragma unroll
                    for (int gq = 0; gq < 16; ++gq) {
                      const float4 v4 = reinterpret_cast<const float4*>(b)[(h * 16 + gq) * 32 + lane];
                      val[gq * 4 + 0] += w * v4.x;
                      val[gq * 4 + 1] += w * v4.y;
                      val[gq * 4 + 2] += w * v4.z;
                      val[gq * 4 + 3] += w * v4.w;
                    }
                  }
                }
                if (h == KCH - 1) {
                  tc_fence_before();
                  mbar_arrive(smem_u32(&misc->o_free[i]));
                }
#pragma unroll
                for (int e = 0; e < 64; ++e) val[e] *= inv;
                store_half(h, *reinterpret_cast<float(*)[32]>(&val[0]), *reinterpret_cast<float(*)[32]>(&val[32]));
              }
              if (!ok) break;
            }
          }
        } else {
        const int c_first = cta_of_unit(sg.unit0, T, G);
        const int c_last = cta_of_unit(sg.unit0 + sg.steps_t - 1, T, G);
        const int parts = c_last - c_first + 1, mine = cta - c_first;
        unsigned int* ctr = p.counters + (((size_t)(c_first * NQ + i) * 4 + wq) << 1);
        auto write_partial = [&]() {
          float* ws = p.ws + ((size_t)(2 * cta + (seg == 0 ? 0 : 1)) * NQ + i) * per_sub;
#pragma unroll 1
          for (int hcol = 0; hcol < D / 64; ++hcol) {
            uint32_t r[64];
            tmem_ld32_nowait(o_tmem + hcol * 64, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
            tmem_ld32_nowait(o_tmem + hcol * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
            tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[0]));
            tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[32]));
#pragma unroll
            for (int gq = 0; gq < 16; ++gq) {
              float4 v4 = make_float4(__uint_as_float(r[gq * 4]), __uint_as_float(r[gq * 4 + 1]),
                                      __uint_as_float(r[gq * 4 + 2]), __uint_as_float(r[gq * 4 + 3]));
              reinterpret_cast<float4*>(ws)[(size_t)(hcol * 16 + gq) * kSub + row] = v4;
            }
          }
          ws[(size_t)kSub * D + row] = m_run;
          ws[(size_t)kSub * D + kSub + row] = delta;
        };
        // Who merges.  Balanced ranges: the parts of a tile finish at different times, so the last finisher
        // (by counter A) merges and nobody waits for a part that has not started.  Uniform key split (the EAGER
        // instantiation): all parts finish together, so the roles are fixed in advance -- the tile's 32-row
        // groups are dealt out to the parts in turn; a warp publishes its rows unless its own part owns them.
        // Every CTA then writes and reads only its share, all parts merge in parallel, and nobody waits for
        // the answer of an atomic.
        bool merges;
        if constexpr (EAGER) {
          const int rg = i * 4 + wq;
          merges = (mine == (parts <= NQ * 4 ? rg % parts : rg));
        } else {
          uint32_t order = 0;
          if (lane == 0) order = atomicAdd(&ctr[0], 1u);
          order = __shfl_sync(0xffffffffu, order, 0);
          merges = (order == (uint32_t)(parts - 1));
        }
        if (!merges) {
          write_partial();
          tc_fence_before();
          mbar_arrive(smem_u32(&misc->o_free[i]));           // O may be overwritten by the next segment
          __threadfence();
          __syncwarp();                                      // the lanes' stores are ordered before lane 0's release
          if (lane == 0) red_release_gpu_inc(&ctr[1]);
        } else {
          // wait (bounded) until the other parts are published
          uint32_t seen = 1;
          if (lane == 0) {
            const long long t0 = clock64();
            while (ld_acquire_gpu(&ctr[1]) < (uint32_t)(parts - 1)) {
              if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { seen = 0; break; }
              __nanosleep(100);                              // the publishers update this cache line: poll gently
            }
            if (!seen && !*abort_flag) {
              report_timeout(wait_info(kRoleSoftmax, kBarSync, 0x7000 | (uint32_t)wq), abort_flag);
              *abort_flag = 1;
            }
          }
          seen = __shfl_sync(0xffffffffu, seen, 0);
          if (!seen) { ok = false; break; }
          __threadfence();
          if (lane == 0) { ctr[0] = 0u; ctr[1] = 0u; }       // ready for the next launch
          // part sp comes from CTA c_first + sp: its first piece if its range starts inside this tile
          auto part_ptr = [&](int sp) -> const float* {
            const int c = c_first + sp;
            const int slot = (range_begin(c, T, G) >= sg.unit0 - (CAUSAL ? kCausalTileCost : 0)) ? 0 : 1;
            return p.ws + ((size_t)(2 * c + slot) * NQ + i) * per_sub;
          };
          if (last_seg && parts <= 4) {
            // Usual case.  The other CTAs' parts are copied asynchronously, 32 columns of this warp's rows at
            // a time, into the warp's slice of the dead Q buffer while the previous piece is accumulated, so
            // that the round trips to L2 overlap instead of following one another.
            constexpr int NBUF = KCH;                         // 4 KB pieces the slice holds
            const uint32_t inb = q_smem + warp * (KCH * 4096) + lane * 16;
            const float* pp[4];
#pragma unroll
            for (int sp = 0; sp < 4; ++sp) pp[sp] = part_ptr(sp < parts ? sp : 0);
            const int n_other = parts - 1, n_items = (D / 32) * n_other;
            auto issue = [&](int k) {                         // item k: chunk k / n_other of the (k % n_other)-th other part
              const int c = k / n_other, o = k - c * n_other, sp = o < mine ? o : o + 1;
              const float* base = sp == 0 ? pp[0] : sp == 1 ? pp[1] : sp == 2 ? pp[2] : pp[3];
              const float4* src = reinterpret_cast<const float4*>(base) + (size_t)(c * 8) * kSub + row;
              const uint32_t dst = inb + (uint32_t)(k % NBUF) * 4096;
#pragma unroll
              for (int gq = 0; gq < 8; ++gq) cp_async16(dst + gq * 512, src + (size_t)gq * kSub);
              cp_async_commit();
            };
            for (int k = 0; k < NBUF && k < n_items; ++k) issue(k);
            float mm[4], dd[4], ww[4];
#pragma unroll
            for (int sp = 0; sp < 4; ++sp) {
              mm[sp] = -INFINITY;
              dd[sp] = 0.f;
              if (sp < parts) {
                mm[sp] = (sp == mine) ? m_run : __ldcg(pp[sp] + (size_t)kSub * D + row);
                dd[sp] = (sp == mine) ? delta : __ldcg(pp[sp] + (size_t)kSub * D + kSub + row);
              }
            }
            const float m_all = fmaxf(fmaxf(mm[0], mm[1]), fmaxf(mm[2], mm[3]));
            float d_all = 0.f;
#pragma unroll
            for (int sp = 0; sp < 4; ++sp) {                   // ascending key order
              ww[sp] = (sp < parts) ? exp2f(mm[sp] - m_all) : 0.f;
              if (sp < parts) d_all += dd[sp] * ww[sp];
            }
            const float inv = 1.0f / d_all;
            int k = 0;
#pragma unroll 1
            for (int h = 0; h < KCH; ++h) {
              float val[64];
#pragma unroll
              for (int cc = 0; cc < 2; ++cc) {
                float* v = &val[cc * 32];
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0.f;
#pragma unroll
                for (int sp = 0; sp < 4; ++sp) {
                  if (sp >= parts) continue;
                  if (sp == mine) {
                    uint32_t r[32];
                    tmem_ld32(o_tmem + h * 64 + cc * 32, r);
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] += ww[sp] * __uint_as_float(r[e]);
                  } else {
                    if (NBUF == 2 && k + 1 < n_items) cp_async_wait<1>(); else cp_async_wait<0>();
                    const uint32_t src = inb + (uint32_t)(k % NBUF) * 4096;
#pragma unroll
                    for (int gq = 0; gq < 8; ++gq) {
                      const float4 v4 = ld_shared_f4(src + gq * 512);
                      v[gq * 4 + 0] += ww[sp] * v4.x;
                      v[gq * 4 + 1] += ww[sp] * v4.y;
                      v[gq * 4 + 2] += ww[sp] * v4.z;
                      v[gq * 4 + 3] += ww[sp] * v4.w;
                    }
                    if (k + NBUF < n_items) issue(k + NBUF);
                    ++k;
                  }
                }
              }
              if (h == KCH - 1) {
                tc_fence_before();
                mbar_arrive(smem_u32(&misc->o_free[i]));     // O may be overwritten by the next segment
              }
#pragma unroll
              for (int e = 0; e < 64; ++e) val[e] *= inv;
              store_half(h, *reinterpret_cast<float(*)[32]>(&val[0]), *reinterpret_cast<float(*)[32]>(&val[32]));
            }
          } else {
          // General case (a merge before the CTA's last segment, or more than four parts): from registers.
          float m_all = m_run;
#pragma unroll 4
          for (int sp = 0; sp < parts; ++sp)
            if (sp != mine) m_all = fmaxf(m_all, __ldcg(part_ptr(sp) + (size_t)kSub * D + row));
          float d_all = 0.f;
          for (int sp = 0; sp < parts; ++sp) {                // ascending key order, own part in its place
            const float* b = part_ptr(sp);
            const float m_sp = (sp == mine) ? m_run : __ldcg(b + (size_t)kSub * D + row);
            const float d_sp = (sp == mine) ? delta : __ldcg(b + (size_t)kSub * D + kSub + row);
            d_all += d_sp * exp2f(m_sp - m_all);
          }
          const float inv = 1.0f / d_all;
#pragma unroll 1
          for (int h = 0; h < KCH; ++h) {
            float val[64];
#pragma unroll
            for (int k = 0; k < 64; ++k) val[k] = 0.f;
            for (int sp = 0; sp < parts; ++sp) {
              const float* b = part_ptr(sp);
              if (sp == mine) {
                const float w = exp2f(m_run - m_all);
                uint32_t r[64];
                tmem_ld32_nowait(o_tmem + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld32_nowait(o_tmem + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
                tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[0]));
                tmem_ld_fence(*reinterpret_cast<uint32_t(*)[32]>(&r[32]));
#pragma unroll
                for (int k = 0; k < 64; ++k) val[k] += w * __uint_as_float(r[k]);
              } else {
                const float w = exp2f(__ldcg(b + (size_t)kSub * D + row) - m_all);
#pragma unroll
                for (int gq = 0; gq < 16; ++gq) {
                  const float4 v4 = __ldcg(reinterpret_cast<const float4*>(b) + (size_t)(h * 16 + gq) * kSub + row);
                  val[gq * 4 + 0] += w * v4.x;
                  val[gq * 4 + 1] += w * v4.y;
                  val[gq * 4 + 2] += w * v4.z;
                  val[gq * 4 + 3] += w * v4.w;
                }
              }
            }
            if (h == KCH - 1) {
              tc_fence_before();
              mbar_arrive(smem_u32(&misc->o_free[i]));       // O may be overwritten by the next segment
            }
#pragma unroll
            for (int k = 0; k < 64; ++k) val[k] *= inv;
            store_half(h, *reinterpret_cast<float(*)[32]>(&val[0]), *reinterpret_cast<float(*)[32]>(&val[32]));
          }
          }
        }
        }
      }
      }
    }
  } else if (warp >= 8 && warp < 12) {
    // ================================================== correction warpgroup
    setmaxnreg_dec<64>();
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    bool ok = run;
    uint32_t g = 0;
    if (ok) {
      long long u = u_lo;
      int seg_ctr = 0;
      Segment sg;
      while (ok && next_segment<CAUSAL>(u, u_hi, seg_ctr, p.n_steps, p.q_tiles, p.ratio, p.head_units, NQ * kSub, sg, p.seg_skip)) {
        const int tile = sg.tile, j0 = sg.j0, j1 = sg.j1, n = sg.n, bh = sg.bh, q_row0 = sg.q_row0, seg = sg.seg;
        (void)tile; (void)j0; (void)j1; (void)bh; (void)q_row0; (void)seg;
      for (int jj = 0; ok && jj < n; ++jj, ++g) {
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
          if (!wait_bar_warp(smem_u32(&misc->alpha_full[i]), g & 1, abort_flag, wait_info(kRoleCorrection, kBarAlpha, g))) {
            ok = false;
            break;
          }
          const float a = misc->alpha[i][g & 1][row];
          if (jj > 0) {                                   // the first step of a segment starts O afresh
            const bool need = __any_sync(0xffffffffu, a != 1.0f);
            if (need) {
              if (!wait_bar_warp(smem_u32(&misc->o_full[i]), (g - 1) & 1, abort_flag,
                                 wait_info(kRoleCorrection, kBarOFull, g))) {
                ok = false;
                break;
              }
              tc_fence_after();
              const uint32_t o_tmem = lane_base + O_COL0 + i * D;
#pragma unroll
              for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(o_tmem + c * 32, r);
#pragma unroll
                for (int k = 0; k < 32; ++k) r[k] = __float_as_uint(__uint_as_float(r[k]) * a);
                tmem_st32(o_tmem + c * 32, r);
              }
              tmem_wait_st();
            }
            tc_fence_before();
          }
          mbar_arrive(smem_u32(&misc->p_full[i]));
        }
      }
      if (!ok) break;
      }
    }
  } else if (warp == 12) {
    // ============================================================ MMA issuer
    // The whole warp walks the loop and the waits (converged control flow keeps descriptors and
    // counters in the uniform datapath); one elected lane issues the matrix instructions and the
    // commits.  Sub-tiles are served strictly in turn: that order is what keeps the two softmax
    // warpgroups half a step apart, so that one computes exponentials while the tensor pipe works
    // for the other.  (setmaxnreg is warpgroup-aligned: warps 12-15 request the same count.)
    setmaxnreg_dec<64>();
    bool ok = run;
    uint32_t g = 0;
    int stage = 0;
    uint32_t phase = 0;
    auto advance = [&]() { if (++stage == p.stages) { stage = 0; phase ^= 1u; } };
    if (ok) {
      long long u = u_lo;
      int seg_ctr = 0;
      Segment sg;
      while (ok && next_segment<CAUSAL>(u, u_hi, seg_ctr, p.n_steps, p.q_tiles, p.ratio, p.head_units, NQ * kSub, sg, p.seg_skip)) {
        const int tile = sg.tile, j0 = sg.j0, j1 = sg.j1, n = sg.n, bh = sg.bh, q_row0 = sg.q_row0, seg = sg.seg;
        (void)tile; (void)j0; (void)j1; (void)bh; (void)q_row0; (void)seg;
      ok = wait_bar_warp(smem_u32(&misc->q_full[0]), seg & 1, abort_flag, wait_info(kRoleMma, kBarQ, seg));
      if (ok) ok = wait_bar_warp(smem_u32(&misc->kv_full[stage]), phase, abort_flag, wait_info(kRoleMma, kBarKvFull, g));
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
        issue_qk<D, TKV>(tmem_base, q_smem, ring_smem + stage * SM::kStageBytes);
        umma_commit(smem_u32(&misc->s_full[0]));
      }
      __syncwarp();
      if (NQ == 2) {
        ok = wait_bar_warp(smem_u32(&misc->q_full[1]), seg & 1, abort_flag, wait_info(kRoleMma, kBarQ, 0x8000 | seg));
        if (!ok) break;
        tc_fence_after();
      }
      const int k0_stage = stage;
      // kSplitP: nothing ties the two sub-tiles to each other any more, so the half-step offset between their
      // softmax warpgroups (one computes exponentials while the other loads, reduces and stores) is set up here:
      // sub-tile 1's first scores are produced only after the first half of sub-tile 0's first P (short segments
      // start both at once; holding K_0 that long while K_1 is awaited needs a third ring stage).
      const bool defer_q1 = kSplitP && n >= 4 && p.stages >= 3;
      if (!defer_q1 && elect_one()) {
        if (NQ == 2) {
          issue_qk<D, TKV>(tmem_base + S_COLS, q_smem + kSub * D * 2, ring_smem + stage * SM::kStageBytes);
          umma_commit(smem_u32(&misc->s_full[1]));
        }
        umma_commit(smem_u32(&misc->kv_empty[stage]));
        if (n == 1) umma_commit(smem_u32(&misc->q_empty));   // a one-step segment reads Q only here
      }
      __syncwarp();
      advance();
      for (int jj = 0; ok && jj < n; ++jj, ++g) {
        const int v_stage = stage;
        const uint32_t v_phase = phase;
        advance();
        const int k_stage = stage;
        const uint32_t k_phase = phase;
        const bool more = (jj + 1 < n);
        if (more) advance();
        const uint32_t v_smem = ring_smem + v_stage * SM::kStageBytes;
        const uint32_t k_smem = ring_smem + k_stage * SM::kStageBytes;
        if constexpr (kSplitP) {
          // Products are issued in the order in which their operands become ready when sub-tile 1 runs half a
          // step behind sub-tile 0.
          const uint32_t p0 = tmem_base + P_COL0, p1 = p0 + TKV / 2, o0 = tmem_base + O_COL0, o1 = o0 + D;
          const uint32_t q1_smem = q_smem + kSub * D * 2;
          auto W = [&](uint64_t* bar, uint32_t par, uint32_t tag) -> bool {
            if (!wait_bar_warp(smem_u32(bar), par, abort_flag, wait_info(kRoleMma, kBarPFull, tag))) { ok = false; return false; }
            tc_fence_after();
            return true;
          };
          if (more) {                                                        // A0: scores of sub-tile 0, next step
            if (!W(&misc->s_free[0], g & 1, 0x100) || !W(&misc->kv_full[k_stage], k_phase, 0x101)) break;
            if (elect_one()) { issue_qk<D, TKV>(tmem_base, q_smem, k_smem); umma_commit(smem_u32(&misc->s_full[0])); }
            __syncwarp();
          }
          if (!W(&misc->kv_full[v_stage], v_phase, 0x102) || !W(&misc->p_full[0], g & 1, 0x103)) break;
          if (jj == 0 && seg > 0 && !W(&misc->o_free[0], (seg - 1) & 1, 0x104)) break;
          if (elect_one()) issue_pv<D, TKV>(o0, p0, v_smem, jj > 0, TKV * 128, 1024, 0, TKV / 32);   // B0a
          __syncwarp();
          if (jj == 0 && defer_q1) {                                         // first scores of sub-tile 1
            if (elect_one()) {
              issue_qk<D, TKV>(tmem_base + S_COLS, q1_smem, ring_smem + k0_stage * SM::kStageBytes);
              umma_commit(smem_u32(&misc->s_full[1]));
              umma_commit(smem_u32(&misc->kv_empty[k0_stage]));
            }
            __syncwarp();
          }
          if (more) {                                                        // A1
            if (!W(&misc->s_free[1], g & 1, 0x105)) break;
            if (elect_one()) {
              issue_qk<D, TKV>(tmem_base + S_COLS, q1_smem, k_smem);
              umma_commit(smem_u32(&misc->s_full[1]));
              umma_commit(smem_u32(&misc->kv_empty[k_stage]));
              if (jj + 2 == n) umma_commit(smem_u32(&misc->q_empty));
            }
            __syncwarp();
          }
          if (!W(&misc->p_half[0], g & 1, 0x106)) break;                     // B0b
          if (elect_one()) {
            issue_pv<D, TKV>(o0, p0, v_smem, true, TKV * 128, 1024, TKV / 32, TKV / 16);
            umma_commit(smem_u32(&misc->o_full[0]));
          }
          __syncwarp();
          if (!W(&misc->p_full[1], g & 1, 0x107)) break;                     // B1a
          if (jj == 0 && seg > 0 && !W(&misc->o_free[1], (seg - 1) & 1, 0x108)) break;
          if (elect_one()) issue_pv<D, TKV>(o1, p1, v_smem, jj > 0, TKV * 128, 1024, 0, TKV / 32);
          __syncwarp();
          if (!W(&misc->p_half[1], g & 1, 0x109)) break;                     // B1b
          if (elect_one()) {
            issue_pv<D, TKV>(o1, p1, v_smem, true, TKV * 128, 1024, TKV / 32, TKV / 16);
            umma_commit(smem_u32(&misc->o_full[1]));
            umma_commit(smem_u32(&misc->kv_empty[v_stage]));
          }
          __syncwarp();
          continue;
        }
        if (!wait_bar_warp(smem_u32(&misc->kv_full[v_stage]), v_phase, abort_flag, wait_info(kRoleMma, kBarKvFull, g))) { ok = false; break; }
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
          const uint32_t s_acc = tmem_base + i * S_COLS;
          const uint32_t o_acc = tmem_base + O_COL0 + i * D;
          if (!wait_bar_warp(smem_u32(&misc->p_full[i]), g & 1, abort_flag, wait_info(kRoleMma, kBarPFull, g))) { ok = false; break; }
          if (jj == 0 && seg > 0) {
            // the previous segment's epilogue must have read O before the first product overwrites it
            if (!wait_bar_warp(smem_u32(&misc->o_free[i]), (seg - 1) & 1, abort_flag, wait_info(kRoleMma, kBarOFull, 0x8000 | seg))) { ok = false; break; }
          }
          tc_fence_after();
          if (elect_one()) {
            issue_pv<D, TKV>(o_acc, s_acc, v_smem, jj > 0, TKV * 128, 1024, 0, TKV / 32);
          }
          __syncwarp();
          if (!wait_bar_warp(smem_u32(&misc->p_half[i]), g & 1, abort_flag, wait_info(kRoleMma, kBarPFull, 0x8000 | g))) { ok = false; break; }
          tc_fence_after();
          if (more && i == 0) {
            if (!wait_bar_warp(smem_u32(&misc->kv_full[k_stage]), k_phase, abort_flag, wait_info(kRoleMma, kBarKvFull, g))) { ok = false; break; }
            tc_fence_after();
          }
          if (elect_one()) {
            issue_pv<D, TKV>(o_acc, s_acc, v_smem, true, TKV * 128, 1024, TKV / 32, TKV / 16);
            umma_commit(smem_u32(&misc->o_full[i]));
            if (i == NQ - 1) umma_commit(smem_u32(&misc->kv_empty[v_stage]));
            if (more) {
              issue_qk<D, TKV>(s_acc, q_smem + i * (kSub * D * 2), k_smem);
              umma_commit(smem_u32(&misc->s_full[i]));
              if (i == NQ - 1) {
                umma_commit(smem_u32(&misc->kv_empty[k_stage]));
                // The last product that reads this segment's Q tile is issued one step before the segment
                // ends: the next segment's Q tile can be fetched while that last step runs.
                if (jj + 2 == n) umma_commit(smem_u32(&misc->q_empty));
              }
            }
          }
          __syncwarp();
        }
      }
      if (!ok) break;
      }
    }
  } else if (warp == 13) {
    // ========================================================== TMA producer
    setmaxnreg_dec<64>();
    if (run && elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      int q_loads = 0;
      {
      long long u = u_lo;
      int seg_ctr = 0;
      Segment sg;
      while (ok && next_segment<CAUSAL>(u, u_hi, seg_ctr, p.n_steps, p.q_tiles, p.ratio, p.head_units, NQ * kSub, sg, p.seg_skip)) {
        const int tile = sg.tile, j0 = sg.j0, j1 = sg.j1, n = sg.n, bh = sg.bh, q_row0 = sg.q_row0, seg = sg.seg;
        (void)tile; (void)j0; (void)j1; (void)bh; (void)q_row0; (void)seg;
        if (seg > 0 &&
            !wait_bar(smem_u32(&misc->q_empty), (seg - 1) & 1, abort_flag, wait_info(kRoleLoad, kBarQ, seg))) { ok = false; break; }
        // Q sub-tile 0, then the first K tile, then Q sub-tile 1: the first product needs only the first two.
        auto load_q = [&](int i) {
          mbar_arrive_expect_tx(smem_u32(&misc->q_full[i]), kSub * D * 2);
#pragma unroll
          for (int c = 0; c < KCH; ++c)
            tma_load_3d(q_smem + i * (kSub * D * 2) + c * (kSub * 128), &tm_q, c * 64, q_row0 + i * kSub, bh,
                        smem_u32(&misc->q_full[i]));
        };
        load_q(0);
        ++q_loads;
        for (int t = 0; t < 2 * n; ++t) {
          if (!wait_bar(smem_u32(&misc->kv_empty[stage]), phase ^ 1u, abort_flag, wait_info(kRoleLoad, kBarKvEmpty, t))) { ok = false; break; }
          const uint32_t bar = smem_u32(&misc->kv_full[stage]);
          mbar_arrive_expect_tx(bar, SM::kStageBytes);
          const CUtensorMap* tm = (t & 1) ? &tm_v : &tm_k;
          const int kv_row = (j0 + (t >> 1)) * TKV;
          const uint32_t dst = ring_smem + stage * SM::kStageBytes;
#pragma unroll
          for (int c = 0; c < KCH; ++c) tma_load_3d(dst + c * (TKV * 128), tm, c * 64, kv_row, bh, bar);
          ++issued;
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
          if (t == 0 && NQ == 2) load_q(1);
        }
        if (!ok) break;
        }
    }
      if (!ok) {
        // Drain: every copy this thread started must land before the CTA may exit.
        const int first = issued > p.stages ? issued - p.stages : 0;
        for (int t = first; t < issued; ++t) {
          const int sidx = t % p.stages;
          const uint32_t ph = (uint32_t)(t / p.stages) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&misc->kv_full[sidx]), ph) && clock64() - t0 < kWaitLimitCycles) {}
        }
        if (q_loads > 0) {
          // (sub-tile 1 of the last Q load may not have been started; its barrier then completes no phase
          // and the limit below ends the wait -- the CTA is already aborting)
          for (int i = 0; i < NQ; ++i) {
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&misc->q_full[i]), (uint32_t)(q_loads - 1) & 1u) && clock64() - t0 < kWaitLimitCycles) {}
          }
        }
      }
    }
  } else {
    setmaxnreg_dec<64>();
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (CLUSTER) {
    if (!cluster_waited) cluster_wait();                 // (the softmax warps waited at the end of their segment)
    cluster_arrive();                                    // no CTA leaves while a peer may still write to it
    cluster_wait();
  }
  if (warp == 15) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------
// Non-pipelined kernel: one 128-row Q tile per CTA, 128 threads, one K/V stage,
// every phase separated by a barrier.
// ---------------------------------------------------------------------------
struct SimpleMisc {
  uint64_t load_bar;
  uint64_t mma_bar;
  uint64_t sync_bar;   // bounded replacement for a CTA-wide barrier inside the loop
  AbortCell abort;
  uint32_t tmem_slot;
};

template <int D, int TKV>
__global__ void __launch_bounds__(128, 1)
attn_fwd_simple_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, int L,
                       float scale_log2, float* __restrict__ scores_out) {
  constexpr int KCH = D / 64;
  constexpr int TMEM_COLS = (TKV + D <= 128) ? 128 : 256;
  constexpr int Q_BYTES = kSub * D * 2;
  constexpr int KV_BYTES = TKV * D * 2;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t q_smem = smem_base, k_smem = smem_base + Q_BYTES, v_smem = k_smem + KV_BYTES;
  SimpleMisc* misc = reinterpret_cast<SimpleMisc*>(smem_raw + Q_BYTES + 2 * KV_BYTES);
  volatile int* abort_flag = &misc->abort.flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = threadIdx.x;
  const int q_row0 = blockIdx.x * kSub;
  const int bh = blockIdx.y;
  const int n = (L + TKV - 1) / TKV;
  const int kv_tail = L % TKV;
  const uint32_t bar_load = smem_u32(&misc->load_bar), bar_mma = smem_u32(&misc->mma_bar);
  const uint32_t bar_sync = smem_u32(&misc->sync_bar);

  if (threadIdx.x == 0) {
    abort_cell_init(&misc->abort, nullptr);
    if (smem_base & 1023u) {
      report_timeout(wait_info(kRoleSimple, 0, 0xFFFF), abort_flag);
      misc->abort.flag = 1;
    }
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    mbar_init(bar_sync, kSub);
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&misc->tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = misc->tmem_slot;
  const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
  const uint32_t s_tmem = lane_base, o_tmem = lane_base + TKV;
  const uint32_t lbo = (uint32_t)(TKV * 128), sbo = 1024u;   // V as MN-major B: next 64-column chunk, next 8 key rows

  float m_run = -INFINITY, delta = 0.f;
  uint32_t ph_load = 0, ph_mma = 0;
  bool ok = (*abort_flag == 0);
  for (int j = 0; ok && j < n; ++j) {
    if (threadIdx.x == 0) {
      mbar_arrive_expect_tx(bar_load, (j == 0 ? Q_BYTES : 0) + 2 * KV_BYTES);
      if (j == 0)
        for (int c = 0; c < KCH; ++c) tma_load_3d(q_smem + c * (kSub * 128), &tm_q, c * 64, q_row0, bh, bar_load);
      for (int c = 0; c < KCH; ++c) tma_load_3d(k_smem + c * (TKV * 128), &tm_k, c * 64, j * TKV, bh, bar_load);
      for (int c = 0; c < KCH; ++c) tma_load_3d(v_smem + c * (TKV * 128), &tm_v, c * 64, j * TKV, bh, bar_load);
    }
    if (!wait_bar_warp(bar_load, ph_load, abort_flag, wait_info(kRoleSimple, kBarLoad, j))) { ok = false; break; }
    ph_load ^= 1u;
    if (threadIdx.x == 0) {
      tc_fence_after();
      issue_qk<D, TKV>(tmem_base, q_smem, k_smem);
      umma_commit(bar_mma);
    }
    if (!wait_bar_warp(bar_mma, ph_mma, abort_flag, wait_info(kRoleSimple, kBarMma, 2 * j))) { ok = false; break; }
    ph_mma ^= 1u;
    tc_fence_after();

    uint32_t s[TKV];
#pragma unroll
    for (int c = 0; c < TKV / 32; ++c) tmem_ld32(s_tmem + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
    if (scores_out != nullptr && j == 0 && blockIdx.x == 0 && blockIdx.y == 0) {
      for (int k = 0; k < TKV; ++k) scores_out[(size_t)row * TKV + k] = __uint_as_float(s[k]);
    }
    if (kv_tail != 0 && j == n - 1) {              // keys past the end of the sequence: -inf, never zero padding
#pragma unroll
      for (int k = 0; k < TKV; ++k)
        if (k >= kv_tail) s[k] = 0xFF800000u;
    }
    float mx = __uint_as_float(s[0]);
#pragma unroll
    for (int k = 1; k < TKV; ++k) mx = fmaxf(mx, __uint_as_float(s[k]));
    const float m_new = fmaxf(m_run, mx * scale_log2);
    const float alpha = ex2_approx(m_run - m_new);
    if (j > 0) {
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(o_tmem + c * 32, r);
#pragma unroll
        for (int k = 0; k < 32; ++k) r[k] = __float_as_uint(__uint_as_float(r[k]) * alpha);
        tmem_st32(o_tmem + c * 32, r);
      }
    }
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < TKV / 32; ++c) {
      uint32_t pk[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const float e0 = ex2_approx(fmaf(__uint_as_float(s[c * 32 + 2 * k]), scale_log2, -m_new));
        const float e1 = ex2_approx(fmaf(__uint_as_float(s[c * 32 + 2 * k + 1]), scale_log2, -m_new));
        sum += e0 + e1;
        pk[k] = pack_bf16x2(e0, e1);
      }
      tmem_st16(s_tmem + c * 16, pk);
    }
    delta = delta * alpha + sum;
    m_run = m_new;
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive(bar_sync);
    if (!wait_bar_warp(bar_sync, j & 1, abort_flag, wait_info(kRoleSimple, kBarSync, j))) { ok = false; break; }
    if (threadIdx.x == 0) {
      tc_fence_after();
      issue_pv<D, TKV>(tmem_base + TKV, tmem_base, v_smem, j > 0, lbo, sbo);
      umma_commit(bar_mma);
    }
    if (!wait_bar_warp(bar_mma, ph_mma, abort_flag, wait_info(kRoleSimple, kBarMma, 2 * j + 1))) { ok = false; break; }
    ph_mma ^= 1u;
    tc_fence_after();
  }
  if (ok) {
    const float inv = 1.0f / delta;
    const bool in_range = q_row0 + row < L;
    uint4* orow = reinterpret_cast<uint4*>(o + ((size_t)bh * L + q_row0 + (in_range ? row : 0)) * D);
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t r[32];
      tmem_ld32(o_tmem + c * 32, r);          // warp-collective: every lane takes part
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        uint4 w;
        w.x = pack_bf16x2(__uint_as_float(r[u * 8 + 0]) * inv, __uint_as_float(r[u * 8 + 1]) * inv);
        w.y = pack_bf16x2(__uint_as_float(r[u * 8 + 2]) * inv, __uint_as_float(r[u * 8 + 3]) * inv);
        w.z = pack_bf16x2(__uint_as_float(r[u * 8 + 4]) * inv, __uint_as_float(r[u * 8 + 5]) * inv);
        w.w = pack_bf16x2(__uint_as_float(r[u * 8 + 6]) * inv, __uint_as_float(r[u * 8 + 7]) * inv);
        if (in_range) orow[c * 4 + u] = w;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace attn
