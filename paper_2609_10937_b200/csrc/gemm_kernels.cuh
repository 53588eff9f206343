// sm_100a kernels of the unfused path: a dense bf16 matrix product C = A B (the paper's Section
// "GEMM") on tcgen05 tensor cores, and a row softmax (Section "Online Softmax": per-thread running
// (m, d) statistics merged with the associative operator of that section).
//
//   gemm_kernel   persistent, warp-specialised: one TMA producer warp -> shared-memory ring of
//                 (A tile, B tile) stages -> one MMA-issuing thread (tcgen05.mma, two 128-row
//                 sub-tiles x 256 columns accumulated in tensor memory) -> eight epilogue warps
//                 (tensor memory -> bf16 -> shared-memory staging -> TMA store).
//   softmax_rows_kernel  one CTA per row, the row held in registers: one read, one write.
//   softmax_rows_staged_kernel  the same for rows too wide for registers: staged in shared memory.
//
// Every device-side wait is bounded (see attn_kernels.cuh).
#pragma once

#include "attn_kernels.cuh"

namespace gemm {

using namespace sm100;
using attn::kSub;

constexpr int kTileM = 2 * kSub;   // two 128-row sub-tiles share every B tile
constexpr int kTileNMax = 256;     // largest N of one matrix instruction; narrow outputs (N <= 128) use 128
constexpr int kTileK = 64;         // one 128-byte swizzle row of bf16
constexpr int kStageA = kTileM * kTileK * 2;
__host__ __device__ constexpr int stage_bytes(int tile_n) { return kStageA + tile_n * kTileK * 2; }
constexpr int kOutBytes = 2 * kSub * 128;    // per sub-tile one [128 rows][64 columns] bf16 staging chunk
constexpr int kMiscBytes = 1024;
constexpr int kMaxStages = 8;
constexpr int kThreads = 320;      // producer warp, MMA warp, eight epilogue warps
__host__ __device__ constexpr int smem_total(int stages, int tile_n) { return stages * stage_bytes(tile_n) + kOutBytes + kMiscBytes; }

enum Role : uint32_t { kRoleGemmLoad = 6, kRoleGemmMma = 7, kRoleGemmEpi = 8 };

struct GemmParams {
  int M, N, K;
  int batch;
  int n_sub;              // 128-row sub-tiles per CTA (1 or 2)
  int m_tiles, n_tiles;   // ceil(M / (128 n_sub)), ceil(N / tile_n)
  int k_steps;            // ceil(K / 64)
  int stages;
  int group_m;            // pair kernel: tiles are walked in bands of this many tile rows (see tile_coords)
  int tail_tiles;         // pair kernel: the last this-many tiles are executed as two half-width work items each
  int stream_c;           // pair kernel: C is larger than the cache and its stores carry the evict-first priority
};

// Order in which the persistent grid walks the output tiles.  Tiles that run at the same time should share operand
// panels in the cache: with P tiles in flight, a band of `group_m` tile rows walked column by column keeps
// group_m row panels of A and about P / group_m column panels of B live -- (group_m + P / group_m) panels, least for
// group_m ~ sqrt(P) -- where walking whole tile rows would stream all of B for every wave.
__device__ __forceinline__ void tile_coords(long long t, int m_tiles, int n_tiles, int group_m, int& mt, int& nt, int& b) {
  const long long per_batch = (long long)m_tiles * n_tiles;
  b = (int)(t / per_batch);
  const int r = (int)(t - (long long)b * per_batch);
  const int band = r / (group_m * n_tiles);
  const int first = band * group_m;
  const int rows = (m_tiles - first) < group_m ? (m_tiles - first) : group_m;
  const int in = r - band * group_m * n_tiles;
  mt = first + in % rows;
  nt = in / rows;
}

struct GemmMisc {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t acc_full;      // all products of a tile have finished
  uint64_t acc_empty;     // the epilogue has read the accumulators of a tile
  uint64_t epi_sync[2];   // rendezvous of the four epilogue warps of a sub-tile
  attn::AbortCell abort;
  uint32_t tmem_slot;
};
static_assert(sizeof(GemmMisc) <= kMiscBytes, "misc region too large");

// B_KN: B is stored [K][N] row-major (C = A B; the MN-major operand form, as V in P V);
// otherwise B is stored [N][K] row-major (C = A B^T; K-major, as K in Q K^T).
template <bool B_KN, int kTileN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
            const __grid_constant__ CUtensorMap tm_c, const GemmParams p) {
  static_assert(kTileN == 128 || kTileN == 256, "tile N");
  constexpr int kStageBytes = stage_bytes(kTileN);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t out_smem = smem_base + p.stages * kStageBytes;
  GemmMisc* misc = reinterpret_cast<GemmMisc*>(smem_raw + p.stages * kStageBytes + kOutBytes);
  volatile int* abort_flag = &misc->abort.flag;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    attn::abort_cell_init(&misc->abort, nullptr);
    if (smem_base & 1023u) {
      attn::report_timeout(attn::wait_info(kRoleGemmLoad, 0, 0xFFFF), abort_flag);
      misc->abort.flag = 1;
    }
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(smem_u32(&misc->full[s]), 1);
      mbar_init(smem_u32(&misc->empty[s]), 1);
    }
    mbar_init(smem_u32(&misc->acc_full), 1);
    mbar_init(smem_u32(&misc->acc_empty), p.n_sub * kSub);
    mbar_init(smem_u32(&misc->epi_sync[0]), kSub);
    mbar_init(smem_u32(&misc->epi_sync[1]), kSub);
    fence_mbar_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b);
    prefetch_tmap(&tm_c);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&misc->tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = misc->tmem_slot;
  const long long tiles = (long long)p.batch * p.m_tiles * p.n_tiles;
  const int tile_m = p.n_sub * kSub;
  const bool run = (*abort_flag == 0);

  if (warp == 0) {
    // ========================================================== TMA producer
    if (run && elect_one()) {
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long t = blockIdx.x; ok && t < tiles; t += gridDim.x) {
        const int nt = (int)(t % p.n_tiles), mt = (int)((t / p.n_tiles) % p.m_tiles), b = (int)(t / ((long long)p.n_tiles * p.m_tiles));
        for (int ks = 0; ks < p.k_steps; ++ks) {
          if (!attn::wait_bar(smem_u32(&misc->empty[stage]), phase ^ 1u, abort_flag, attn::wait_info(kRoleGemmLoad, 1, ks))) { ok = false; break; }
          const uint32_t bar = smem_u32(&misc->full[stage]);
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kStageA;
          mbar_arrive_expect_tx(bar, kStageBytes - (2 - p.n_sub) * (kSub * kTileK * 2));
          tma_load_3d(a_dst, &tm_a, ks * kTileK, mt * tile_m, b, bar);
          if (p.n_sub == 2) tma_load_3d(a_dst + kSub * 128, &tm_a, ks * kTileK, mt * tile_m + kSub, b, bar);
          if (B_KN) {
#pragma unroll
            for (int c = 0; c < kTileN / 64; ++c)
              tma_load_3d(b_dst + c * (kTileK * 128), &tm_b, nt * kTileN + c * 64, ks * kTileK, b, bar);
          } else {
            tma_load_3d(b_dst, &tm_b, ks * kTileK, nt * kTileN, b, bar);
          }
          ++issued;
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Drain: every copy this thread started must land before the CTA may exit.
        const int first = issued > p.stages ? issued - p.stages : 0;
        for (int t = first; t < issued; ++t) {
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&misc->full[t % p.stages]), (uint32_t)(t / p.stages) & 1u) &&
                 clock64() - t0 < attn::kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // ============================================================ MMA issuer
    bool ok = run;
    int stage = 0;
    uint32_t phase = 0, tile_ctr = 0;
    constexpr uint32_t idesc = make_idesc_bf16(kSub, kTileN, B_KN);
    constexpr uint32_t hi_k = attn::desc_hi_sw128(1024);
    for (long long t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++tile_ctr) {
      if (tile_ctr > 0) {
        ok = attn::wait_bar_warp(smem_u32(&misc->acc_empty), (tile_ctr - 1) & 1, abort_flag, attn::wait_info(kRoleGemmMma, 2, tile_ctr));
        if (!ok) break;
        tc_fence_after();
      }
      for (int ks = 0; ok && ks < p.k_steps; ++ks) {
        if (!attn::wait_bar_warp(smem_u32(&misc->full[stage]), phase, abort_flag, attn::wait_info(kRoleGemmMma, 1, ks))) { ok = false; break; }
        tc_fence_after();
        if (elect_one()) {
          const uint32_t a_smem = smem_base + stage * kStageBytes, b_smem = a_smem + kStageA;
          const uint32_t b_lo = B_KN ? attn::desc_lo(b_smem, kTileK * 128) : attn::desc_lo(b_smem, 16);
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            if (sub >= p.n_sub) break;
            const uint32_t a_lo = attn::desc_lo(a_smem + sub * (kSub * 128), 16);
#pragma unroll
            for (int k16 = 0; k16 < kTileK / 16; ++k16) {
              const uint64_t a = attn::desc_from_words(a_lo + ((k16 * 32) >> 4), hi_k);
              // K-major B: 16 columns further along the swizzle row; MN-major B: 16 key rows = 2048 bytes further
              const uint64_t b = attn::desc_from_words(b_lo + ((B_KN ? k16 * 2048 : k16 * 32) >> 4), hi_k);
              umma_ss(tmem_base + sub * kTileN, a, b, idesc, (ks > 0 || k16 > 0) ? 1u : 0u);
            }
          }
          umma_commit(smem_u32(&misc->empty[stage]));
          if (ks == p.k_steps - 1) umma_commit(smem_u32(&misc->acc_full));
        }
        __syncwarp();
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // ============================================================== epilogue
    const int sub = (warp - 2) >> 2;
    const int row = (warp & 3) * 32 + lane;
    const uint32_t acc = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + sub * kTileN;
    const uint32_t bar_e = smem_u32(&misc->epi_sync[sub]);
    const uint32_t stage_out = out_smem + sub * (kSub * 128);
    const bool leader = ((warp - 2) & 3) == 0 && lane == 0;
    uint32_t ep_phase = 0, tile_ctr = 0;
    bool ok = run && sub < p.n_sub;
    auto group_sync = [&](uint32_t tag) -> bool {
      mbar_arrive(bar_e);
      const bool r = attn::wait_bar_warp(bar_e, ep_phase, abort_flag, attn::wait_info(kRoleGemmEpi, 3, tag));
      ep_phase ^= 1u;
      return r;
    };
    for (long long t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++tile_ctr) {
      const int nt = (int)(t % p.n_tiles), mt = (int)((t / p.n_tiles) % p.m_tiles), b = (int)(t / ((long long)p.n_tiles * p.m_tiles));
      ok = attn::wait_bar_warp(smem_u32(&misc->acc_full), tile_ctr & 1, abort_flag, attn::wait_info(kRoleGemmEpi, 2, tile_ctr));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < kTileN / 32; ++c) {
        uint32_t r[32];
        float val[32];
        tmem_ld32(acc + c * 32, r);
#pragma unroll
        for (int k = 0; k < 32; ++k) val[k] = __uint_as_float(r[k]);
        if (c == kTileN / 32 - 1) {
          tc_fence_before();
          mbar_arrive(smem_u32(&misc->acc_empty));       // the next tile may overwrite the accumulators
        }
        attn::stage_row_chunk(stage_out, c & 1, row, val);
        if ((c & 1) == 0) continue;
        fence_proxy_async_smem();
        if (!(ok = group_sync(c))) break;
        if (leader) {
          tma_store_3d(&tm_c, stage_out, nt * kTileN + (c >> 1) * 64, mt * tile_m + sub * kSub, b);
          tma_store_commit();
          tma_store_wait_read();
        }
        if (!(ok = group_sync(0x100 | c))) break;          // the staging chunk may be written again
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------
// gemm_pair_kernel: the same product with two CTAs per matrix instruction (cta_group::2).
//
// A cluster of two CTAs owns a 256 x kPairN output tile.  CTA r of the pair holds rows [128 r, 128 r + 128) of the A
// tile and columns [r kPairN / 2, (r + 1) kPairN / 2) of the B tile in its shared memory -- every byte of B is
// fetched and stored once per pair, so a CTA's ring stage is half as large as for a lone CTA working on 256 rows --
// and the 128 x kPairN fp32 accumulator of its rows in its tensor memory.  One thread of the even CTA issues
// tcgen05.mma.cta_group::2 for both; its completion releases the ring stage in both CTAs (a commit multicast to
// the two CTAs' barriers).  An accumulator takes kPairN of the 512 tensor-memory columns, so there are 512 / kPairN
// of them and the epilogue of tile i (tensor memory -> bf16 -> staging -> TMA store, per CTA for its own rows) runs
// under the products of tile i + 1.  Barriers: full[s] of the even CTA counts the bytes of both CTAs' loads (the
// odd CTA's copies name that barrier; no load is multicast); empty[s] and acc_full[b] exist in both CTAs;
// acc_empty[b] of the even CTA counts one arrival per epilogue warp of both CTAs.
// ---------------------------------------------------------------------------
constexpr int kPairEpiWarps = 8;           // four lane quarters x two column halves of the accumulator
constexpr int kPairThreads = 64 + 32 * kPairEpiWarps;   // producer warp, MMA warp, epilogue warps
constexpr int kPairStageA = kSub * kTileK * 2;
__host__ __device__ constexpr int pair_stage_bytes(int pair_n) { return kPairStageA + (pair_n / 2) * kTileK * 2; }
constexpr int kPairOutBytes = kPairEpiWarps * 2 * 4096;  // per epilogue warp two [32 rows][64 columns] bf16 staging chunks
__host__ __device__ constexpr int pair_smem_total(int stages, int pair_n) {
  return stages * pair_stage_bytes(pair_n) + kPairOutBytes + kMiscBytes;
}

struct GemmPairMisc {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t acc_full[4];
  uint64_t acc_empty[4];
  attn::AbortCell abort;
  uint32_t tmem_slot;
};
static_assert(sizeof(GemmPairMisc) <= kMiscBytes, "misc region too large");

template <bool B_KN, int kPairN>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                 const __grid_constant__ CUtensorMap tm_c, const GemmParams p) {
  static_assert(kPairN == 128 || kPairN == 256, "pair tile N");
  constexpr int kStageBytes = pair_stage_bytes(kPairN);
  constexpr int kHalfN = kPairN / 2;                 // B columns held by one CTA
  constexpr int kBufs = 512 / kPairN;                // accumulators in tensor memory
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t out_smem = smem_base + p.stages * kStageBytes;
  GemmPairMisc* misc = reinterpret_cast<GemmPairMisc*>(smem_raw + p.stages * kStageBytes + kPairOutBytes);
  volatile int* abort_flag = &misc->abort.flag;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();           // 0: issues the matrix instructions of the pair
  const long long pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    attn::abort_cell_init(&misc->abort, nullptr);
    if (smem_base & 1023u) {
      attn::report_timeout(attn::wait_info(kRoleGemmLoad, 0, 0xFFFF), abort_flag);
      misc->abort.flag = 1;
    }
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(smem_u32(&misc->full[s]), 1);
      mbar_init(smem_u32(&misc->empty[s]), 1);
    }
    for (int b = 0; b < 4; ++b) {
      mbar_init(smem_u32(&misc->acc_full[b]), 1);
      mbar_init(smem_u32(&misc->acc_empty[b]), 2 * kPairEpiWarps);   // the epilogue warps of both CTAs of the pair
    }
    fence_mbar_init();
    prefetch_tmap(&tm_a);
    prefetch_tmap(&tm_b);
    prefetch_tmap(&tm_c);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&misc->tmem_slot), 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  // the peer's barriers must exist before this CTA's copies or commits touch them
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = misc->tmem_slot;
  const long long tiles = (long long)p.batch * p.m_tiles * p.n_tiles;
  const bool run = (*abort_flag == 0);
  // Work items.  The tiles that would make up a last, partly empty wave (p.tail_tiles of them, fewer than half the
  // pairs) are executed as two items of half the width each, so that the last wave keeps twice as many pairs busy for
  // about 0.6 of a tile's time (a 128-wide instruction of a pair runs at about 0.8 of the rate of a 256-wide one).
  const long long full_tiles = tiles - (kPairN == 256 ? p.tail_tiles : 0);
  const long long items = full_tiles + 2 * (tiles - full_tiles);
  auto item_of = [&](long long t, int& mt, int& nt, int& b, int& narrow, int& hcol) {
    narrow = t >= full_tiles ? 1 : 0;
    hcol = narrow ? (int)((t - full_tiles) & 1) : 0;
    tile_coords(narrow ? full_tiles + ((t - full_tiles) >> 1) : t, p.m_tiles, p.n_tiles, p.group_m, mt, nt, b);
  };

  if (warp == 0) {
    // ========================================================== TMA producer (both CTAs, each for what it holds)
    if (run && elect_one()) {
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long t = pair; ok && t < items; t += n_pairs) {
        int nt, mt, b, narrow, hcol;
        item_of(t, mt, nt, b, narrow, hcol);
        // a half-width item: this CTA holds 64 of its 128 columns (the [N][K] box still brings 128 rows: the matrix
        // instruction reads the first 64)
        const int row0 = mt * kTileM + (int)rank * kSub;
        const int col0 = nt * kPairN + (narrow ? hcol * (kPairN / 2) + (int)rank * (kHalfN / 2) : (int)rank * kHalfN);
        const int b_chunks = narrow ? kHalfN / 128 : kHalfN / 64;
        const uint32_t tx = (B_KN && narrow) ? 2u * (kPairStageA + (kHalfN / 2) * kTileK * 2) : 2u * kStageBytes;
        for (int ks = 0; ks < p.k_steps; ++ks) {
          if (!attn::wait_bar(smem_u32(&misc->empty[stage]), phase ^ 1u, abort_flag, attn::wait_info(kRoleGemmLoad, 1, ks))) { ok = false; break; }
          // the even CTA's barrier counts the bytes of both CTAs' copies of this stage
          const uint32_t bar = map_to_cta(smem_u32(&misc->full[stage]), 0);
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kPairStageA;
          if (rank == 0) mbar_arrive_expect_tx(smem_u32(&misc->full[stage]), tx);
          tma_load_3d_pair(a_dst, &tm_a, ks * kTileK, row0, b, bar);
          if (B_KN) {
            for (int c = 0; c < b_chunks; ++c)
              tma_load_3d_pair(b_dst + c * (kTileK * 128), &tm_b, col0 + c * 64, ks * kTileK, b, bar);
          } else {
            tma_load_3d_pair(b_dst, &tm_b, ks * kTileK, col0, b, bar);
          }
          ++issued;
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Drain: a copy this thread started must land before the CTA may exit.  The bytes are counted on the even
        // CTA's barrier; the odd CTA cannot poll it, so it waits out the time a copy can take instead.
        if (rank == 0) {
          const int first = issued > p.stages ? issued - p.stages : 0;
          for (int t = first; t < issued; ++t) {
            const long long t0 = clock64();
            while (!mbar_try_wait(smem_u32(&misc->full[t % p.stages]), (uint32_t)(t / p.stages) & 1u) &&
                   clock64() - t0 < attn::kWaitLimitCycles) {}
          }
        } else {
          const long long t0 = clock64();
          while (clock64() - t0 < 2000000LL) {}
        }
      }
    }
  } else if (warp == 1) {
    // ============================================================ MMA issuer (even CTA only)
    bool ok = run && rank == 0;
    int stage = 0;
    uint32_t phase = 0, tile_ctr = 0;
    constexpr uint32_t idesc_full = make_idesc_bf16(2 * kSub, kPairN, B_KN);
    constexpr uint32_t idesc_narrow = make_idesc_bf16(2 * kSub, kPairN / 2, B_KN);
    constexpr uint32_t hi_k = attn::desc_hi_sw128(1024);
    for (long long t = pair; ok && t < items; t += n_pairs, ++tile_ctr) {
      const uint32_t buf = tile_ctr % kBufs, use = tile_ctr / kBufs;
      const uint32_t idesc = t >= full_tiles ? idesc_narrow : idesc_full;
      if (use > 0) {
        ok = attn::wait_bar_warp(smem_u32(&misc->acc_empty[buf]), (use - 1) & 1, abort_flag, attn::wait_info(kRoleGemmMma, 2, tile_ctr));
        if (!ok) break;
        tc_fence_after();
      }
      for (int ks = 0; ok && ks < p.k_steps; ++ks) {
        if (!attn::wait_bar_warp(smem_u32(&misc->full[stage]), phase, abort_flag, attn::wait_info(kRoleGemmMma, 1, ks))) { ok = false; break; }
        tc_fence_after();
        if (elect_one()) {
          const uint32_t a_smem = smem_base + stage * kStageBytes, b_smem = a_smem + kPairStageA;
          const uint32_t a_lo = attn::desc_lo(a_smem, 16);
          const uint32_t b_lo = B_KN ? attn::desc_lo(b_smem, kTileK * 128) : attn::desc_lo(b_smem, 16);
#pragma unroll
          for (int k16 = 0; k16 < kTileK / 16; ++k16) {
            const uint64_t a = attn::desc_from_words(a_lo + ((k16 * 32) >> 4), hi_k);
            const uint64_t b = attn::desc_from_words(b_lo + ((B_KN ? k16 * 2048 : k16 * 32) >> 4), hi_k);
            umma_ss_pair(tmem_base + buf * kPairN, a, b, idesc, (ks > 0 || k16 > 0) ? 1u : 0u);
          }
          umma_commit_pair(smem_u32(&misc->empty[stage]), 3);
          if (ks == p.k_steps - 1) umma_commit_pair(smem_u32(&misc->acc_full[buf]), 3);
        }
        __syncwarp();
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // ============================================================== epilogue (both CTAs, each its own 128 rows)
    // Eight warps, none of which meets another: warp w reads lanes 32 (w mod 4) .. + 31 (its rows) of one column
    // half of the accumulator, 64 columns at a time, and sends them off through two staging chunks of its own
    // (tensor memory -> bf16 -> swizzled [32 rows][64 columns] chunk -> TMA store of a 32-row box), the store of
    // one chunk running under the conversion of the next.
    const int ew = warp - 2;
    const int half = ew >> 2;                                 // column half of the accumulator
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t stage_w = out_smem + ew * 8192;
    uint32_t tile_ctr = 0, chunk_ctr = 0;
    bool ok = run;
    for (long long t = pair; ok && t < items; t += n_pairs, ++tile_ctr) {
      int nt, mt, b, narrow, hcol;
      item_of(t, mt, nt, b, narrow, hcol);
      const int width = narrow ? kPairN / 2 : kPairN;           // columns of this item's accumulator
      const int kChunks = width / 128;                          // 64-column chunks per warp and item
      const uint32_t buf = tile_ctr % kBufs, use = tile_ctr / kBufs;
      ok = attn::wait_bar_warp(smem_u32(&misc->acc_full[buf]), use & 1, abort_flag, attn::wait_info(kRoleGemmEpi, 2, tile_ctr));
      if (!ok) break;
      tc_fence_after();
      const uint32_t acc = lane_base + buf * kPairN + half * (width / 2);
      const int row0 = mt * kTileM + (int)rank * kSub + (warp & 3) * 32;
      const int col_w = nt * kPairN + hcol * (kPairN / 2) + half * (width / 2);   // first column of this warp's part
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c, ++chunk_ctr) {
        uint32_t r0[32], r1[32];
        tmem_ld32_nowait(acc + c * 64, r0);
        tmem_ld32_nowait(acc + c * 64 + 32, r1);
        tmem_ld_fence(r0);
        tmem_ld_fence(r1);
        if (c == kChunks - 1) {
          // this warp has read its part of the accumulator: one arrival per warp on the even CTA's barrier (the
          // tensor-memory loads have completed and are fenced; no memory of this thread has to reach the peer)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_peer(map_to_cta(smem_u32(&misc->acc_empty[buf]), 0));
        }
        const uint32_t dst = stage_w + (chunk_ctr & 1) * 4096;
        // the store that last read this chunk (two chunks ago) must have finished reading it
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        __syncwarp();
        float v0[32], v1[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) { v0[k] = __uint_as_float(r0[k]); v1[k] = __uint_as_float(r1[k]); }
        attn::stage_row_chunk(dst, 0, lane, v0);
        attn::stage_row_chunk(dst, 1, lane, v1);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (p.stream_c) tma_store_3d_hint(&tm_c, dst, col_w + c * 64, row0, b, l2_policy_evict_first());
          else tma_store_3d(&tm_c, dst, col_w + c * 64, row0, b);
          tma_store_commit();
        }
      }
    }
    if (lane == 0) tma_store_wait_read();                    // shared memory is read by the stores until here
    __syncwarp();
  }
  tc_fence_before();
  __syncthreads();
  // no CTA leaves while its peer may still read its shared memory, signal its barriers or use its tensor memory
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------
// Row softmax of scale * S, bf16 in and out (in place allowed).  One CTA of THREADS threads per row; thread t
// holds VPT vectors of 8 consecutive columns (vector v covers columns (v * THREADS + t) * 8 ...).  Each thread keeps
// the running statistics (m, d) of its columns; partials are merged with
//   (m1, d1) (+) (m2, d2) = (max(m1, m2), d1 2^(m1 - m) + d2 2^(m2 - m))
// first across the warp by shuffles, then across warps through shared memory.
// ---------------------------------------------------------------------------

__device__ __forceinline__ void merge_md(float& m, float& d, float m2, float d2) {
  const float mn = fmaxf(m, m2);
  // a side with no element yet has m = -inf and d = 0: its term is 0, not NaN
  const float t1 = (m == -INFINITY) ? 0.f : d * exp2f(m - mn);
  const float t2 = (m2 == -INFINITY) ? 0.f : d2 * exp2f(m2 - mn);
  m = mn;
  d = t1 + t2;
}

template <int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS)
softmax_rows_kernel(const __nv_bfloat16* s, __nv_bfloat16* pout, int cols, float scale_log2) {
  __shared__ float sm_m[THREADS / 32], sm_d[THREADS / 32];
  const size_t row = blockIdx.x;
  const uint4* src = reinterpret_cast<const uint4*>(s + row * (size_t)cols);
  uint4* dst = reinterpret_cast<uint4*>(pout + row * (size_t)cols);
  const int nvec = cols / 8;
  // Pass 1 on the packed bf16 words: load, running maximum per lane pair (scale > 0 keeps the order).
  uint32_t w[VPT][4];
  uint32_t mx2 = 0xFF80FF80u;                               // (-inf, -inf) in bf16
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
    const int idx = v * THREADS + threadIdx.x;
    if (idx < nvec) {
      const uint4 q = src[idx];
      w[v][0] = q.x; w[v][1] = q.y; w[v][2] = q.z; w[v][3] = q.w;
#pragma unroll
      for (int e = 0; e < 4; ++e) mx2 = max_bf16x2(mx2, w[v][e]);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) w[v][e] = 0xFF80FF80u;    // -inf: weight 0
    }
  }
  float m = fmaxf(__uint_as_float(mx2 << 16), __uint_as_float(mx2 & 0xFFFF0000u)) * scale_log2;
  // this thread's statistics; the exponentials are kept (relative to the thread's own maximum) and only
  // rescaled once the row's maximum is known: one exponential per element
  const float m_own = m;
  const float neg_m = (m_own == -INFINITY) ? 0.f : -m_own;
  const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2), negm2 = pack_f32x2(neg_m, neg_m);
  uint64_t x[VPT][4];
  uint64_t d2 = 0ull;
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint64_t t = fma_f32x2(pack_f32x2(__uint_as_float(w[v][e] << 16), __uint_as_float(w[v][e] & 0xFFFF0000u)), scale2, negm2);
      float t0, t1;
      unpack_f32x2(t, t0, t1);
      x[v][e] = pack_f32x2(ex2_approx(t0), ex2_approx(t1));
      d2 = add_f32x2(d2, x[v][e]);
    }
  }
  float d0, d1;
  unpack_f32x2(d2, d0, d1);
  float d = d0 + d1;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, off), dd = __shfl_xor_sync(0xffffffffu, d, off);
    merge_md(m, d, m2, dd);
  }
  if ((threadIdx.x & 31) == 0) { sm_m[threadIdx.x >> 5] = m; sm_d[threadIdx.x >> 5] = d; }
  __syncthreads();
  float mr = sm_m[0], dr = sm_d[0];
#pragma unroll
  for (int k = 1; k < THREADS / 32; ++k) merge_md(mr, dr, sm_m[k], sm_d[k]);
  const float f = (m_own == -INFINITY) ? 0.f : exp2f(m_own - mr) / dr;
  const uint64_t f2 = pack_f32x2(f, f);
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
    const int idx = v * THREADS + threadIdx.x;
    if (idx < nvec) {
      uint32_t o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float a0, a1;
        unpack_f32x2(mul_f32x2(x[v][e], f2), a0, a1);
        o[e] = pack_bf16x2(a0, a1);
      }
      dst[idx] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// Rows too wide for registers (more than 2048 vectors of 8 columns): the row is staged in shared memory (2 bytes per
// column) -- still one read and one write of the matrix.  Pass 1: global -> shared, running maximum on the packed
// words; pass 2: sum of exp2(scale x - m) from shared memory; pass 3: the exponentials again, normalised, to global
// (two exponentials per element cost less than a second trip to HBM or than fp32 staging, which would halve the rows
// in flight per SM).
template <int THREADS>
__global__ void __launch_bounds__(THREADS)
softmax_rows_staged_kernel(const __nv_bfloat16* s, __nv_bfloat16* pout, int cols, float scale_log2) {
  extern __shared__ __align__(16) uint8_t smem_row[];
  __shared__ float sm_m[THREADS / 32], sm_d[THREADS / 32];
  const size_t row = blockIdx.x;
  const uint4* src = reinterpret_cast<const uint4*>(s + row * (size_t)cols);
  uint4* dst = reinterpret_cast<uint4*>(pout + row * (size_t)cols);
  uint4* stage = reinterpret_cast<uint4*>(smem_row);
  const int nvec = cols / 8;
  uint32_t mx2 = 0xFF80FF80u;                               // (-inf, -inf) in bf16
#pragma unroll 4
  for (int idx = threadIdx.x; idx < nvec; idx += THREADS) {
    const uint4 q = src[idx];
    stage[idx] = q;                                         // (each thread re-reads only what it wrote: no barrier)
    mx2 = max_bf16x2(max_bf16x2(mx2, q.x), max_bf16x2(max_bf16x2(q.y, q.z), q.w));
  }
  float m = fmaxf(__uint_as_float(mx2 << 16), __uint_as_float(mx2 & 0xFFFF0000u)) * scale_log2;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if ((threadIdx.x & 31) == 0) sm_m[threadIdx.x >> 5] = m;
  __syncthreads();
  float mr = sm_m[0];
#pragma unroll
  for (int k = 1; k < THREADS / 32; ++k) mr = fmaxf(mr, sm_m[k]);
  const float neg_m = (mr == -INFINITY) ? 0.f : -mr;
  const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2), negm2 = pack_f32x2(neg_m, neg_m);
  auto exp_pair = [&](uint32_t w) -> uint64_t {
    const uint64_t t = fma_f32x2(pack_f32x2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)), scale2, negm2);
    float t0, t1;
    unpack_f32x2(t, t0, t1);
    return pack_f32x2(ex2_approx(t0), ex2_approx(t1));
  };
  uint64_t d2 = 0ull;
#pragma unroll 2
  for (int idx = threadIdx.x; idx < nvec; idx += THREADS) {
    const uint4 q = stage[idx];
    d2 = add_f32x2(d2, add_f32x2(add_f32x2(exp_pair(q.x), exp_pair(q.y)), add_f32x2(exp_pair(q.z), exp_pair(q.w))));
  }
  float d0, d1;
  unpack_f32x2(d2, d0, d1);
  float d = d0 + d1;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
  if ((threadIdx.x & 31) == 0) sm_d[threadIdx.x >> 5] = d;
  __syncthreads();
  float dr = sm_d[0];
#pragma unroll
  for (int k = 1; k < THREADS / 32; ++k) dr += sm_d[k];
  const float inv = 1.0f / dr;
  const uint64_t inv2 = pack_f32x2(inv, inv);
  auto out_pair = [&](uint32_t w) -> uint32_t {
    float a0, a1;
    unpack_f32x2(mul_f32x2(exp_pair(w), inv2), a0, a1);
    return pack_bf16x2(a0, a1);
  };
#pragma unroll 2
  for (int idx = threadIdx.x; idx < nvec; idx += THREADS) {
    const uint4 q = stage[idx];
    dst[idx] = make_uint4(out_pair(q.x), out_pair(q.y), out_pair(q.z), out_pair(q.w));
  }
}

}  // namespace gemm
