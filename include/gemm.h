/*
 * C ABI of the unfused path: dense bf16 matrix product with closed-form tiles,
 * row softmax, and the three-kernel attention built from them.  Same library
 * (libattn_b200.so), same conventions and status codes as attn.h.
 *
 * What the paper defines:
 *   - Section "GEMM": C = A B with tiles derived from the hardware descriptor
 *     (Section "Tile Derivation", Eq. 2 and Eq. 3: the local memory fixes the
 *     block tile, the accumulator storage fixes the per-instruction tile);
 *   - Section "Online Softmax": row softmax with running (m, d) statistics and
 *     the associative merge of partial statistics;
 *   - Section "Results", the unfused baseline: S = Q K^T written to memory, a
 *     separate softmax pass, then P V.
 *
 * All data pointers are DEVICE pointers to contiguous bf16 arrays, 16-byte
 * aligned; the caller owns every buffer; nothing is allocated here; calls are
 * asynchronous on `cuda_stream` (a cudaStream_t, NULL = default stream).
 */
#ifndef PAPER_2609_10937_GEMM_H_
#define PAPER_2609_10937_GEMM_H_

#include "attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Result of the closed-form tile derivation for the matrix product. */
typedef struct gemm_tiles {
  int32_t tile_m;       /* rows of C per CTA = n_sub * atom_m                                   */
  int32_t tile_n;       /* columns of C per CTA = N of one matrix instruction                    */
  int32_t tile_k;       /* K extent of one ring stage (one 128-byte swizzle row of elements)     */
  int32_t n_sub;        /* atom_m-row sub-tiles per CTA that share every B tile                  */
  int32_t stages;       /* depth of the shared-memory ring of (A tile, B tile) pairs             */
  int32_t smem_bytes;   /* dynamic shared memory per CTA                                         */
  int32_t tmem_columns; /* tensor-memory columns of the accumulators                             */
  int32_t tiles;        /* batch * ceil(M / tile_m) * ceil(N / tile_n)                           */
  int32_t ctas;         /* persistent grid: min(num_units, tiles)                                */
  int32_t feasible;     /* 1 if the kernel's tile shape fits this descriptor                     */
  float wave_efficiency;/* tiles / (ceil(tiles / ctas) * ctas); per pair of CTAs if cta_pair == 2 */
  int32_t binding_constraint; /* attn_binding: what fixed the tile (tensor memory or ring depth) */
  int32_t cta_pair;     /* CTAs that share one matrix instruction: 1, or 2 (a cluster of two CTAs owns a
                           tile_m x tile_n tile, each holding half of its rows and half of B's columns)  */
  int32_t acc_buffers;  /* accumulators that fit tensor memory: with more than one the epilogue of a tile
                           runs under the products of the next                                        */
  int32_t tail_split;   /* CTA pairs: the last this-many tiles -- those that would form a partly empty last wave,
                           if they are no more than half the pairs -- run as two half-width work items each      */
} gemm_tiles;

/*
 * Tiles for C[batch][M][N] = A[batch][M][K] B (Eq. 2 and Eq. 3 re-derived for
 * tensor memory): tile_n = atom_n_max (atom_n_max / 2 if N <= atom_n_max / 2);
 * n_sub = min(2, acc_mem_columns / atom_n_max), reduced to 1 if two-sub-tile blocks
 * would be fewer than the compute units (occupancy);
 * tile_k = 128 bytes / elem_bytes; stages = min(8, (local_mem - staging - 1024)
 * / ((tile_m + tile_n) * tile_k * elem_bytes)), at least 2.
 * CTA pairs: taken when the descriptor says pairs can run (max_clusters[1] > 0), tensor memory holds two
 * accumulators (acc_mem_columns >= 2 atom_n_max), M > atom_m, N > atom_n_max / 2 (any K: measured, 16384 x 16384 x K,
 * pairs 100 / 98 / 131 / 198 us against 121 / 147 / 195 / 263 us for lone CTAs at K = 64 / 128 / 256 / 512) and
 * the pairs, P = min(max_clusters[1], num_units / 2, tiles), occupy at least as many CTAs as the lone-CTA tiling
 * above would (the paper's occupancy step).  A pair owns a 2 atom_m x atom_n_max tile; every CTA stages its own
 * atom_m rows of A and atom_n_max / 2 columns of B, so stages = min(8, (local_mem - 4 atom_m 128 - 1024) /
 * ((atom_m + atom_n_max / 2) * tile_k * elem_bytes)); acc_buffers = acc_mem_columns / atom_n_max; ctas = 2 P.
 * Last wave: r = tiles mod P tiles remain after the whole waves; if 0 < 2 r <= P they are executed as 2 r work items
 * of half the width (tail_split = r), which keeps twice as many pairs busy for the shorter last wave; wave_efficiency
 * then counts a half-width item as 0.64 of a tile (measured on B200: the narrow instruction runs at 0.78 of the rate).
 * Pure host arithmetic.  Returns ATTN_OK (then check out->feasible) or ATTN_ERR_INVALID_ARG.
 */
int gemm_plan(const attn_hw_desc *desc, int batch, int M, int N, int K, gemm_tiles *out);

/*
 * C = A B per batch entry, bf16 in, fp32 accumulation, bf16 out (round to
 * nearest even).  a: [batch][M][K].  b_layout 0: b is [batch][K][N] (C = A B);
 * b_layout 1: b is [batch][N][K] (C = A B^T).  c: [batch][M][N].  Any M, N >= 1;
 * K, N (and for b_layout 0 also N as the row length of b) must be multiples of 8
 * so that every row starts 16-byte aligned.  c must not overlap a or b.
 * Errors: ATTN_ERR_INVALID_ARG, ATTN_ERR_UNSUPPORTED_SHAPE, ATTN_ERR_MISALIGNED,
 * ATTN_ERR_ALIASING, ATTN_ERR_WRONG_ARCH, ATTN_ERR_INFEASIBLE_PLAN, ATTN_ERR_CUDA.
 */
int gemm_forward(const void *a, const void *b, void *c, int batch, int M, int N, int K, int b_layout,
                 void *cuda_stream);

/* Same with tile fields overridden (tile sweep only; 0 keeps the closed-form value): cta_pair = 1 runs the
 * lone-CTA tiling where the closed form takes pairs, cta_pair = 2 insists on pairs; tile_n (128 | 256) narrows a
 * pair's tile; tail_split < 0 keeps whole tiles in the last wave.  ATTN_ERR_BAD_TILES if the combination was not compiled or does not fit. */
int gemm_forward_tiles(const void *a, const void *b, void *c, int batch, int M, int N, int K, int b_layout,
                       const gemm_tiles *override_tiles, void *cuda_stream);

/*
 * p[r][:] = softmax(scale * s[r][:]) for `rows` rows of `cols` bf16 values
 * (cols a multiple of 8, at most 32768); p may be s (in place).  One read and
 * one write of the matrix: the row is held in registers, or staged in shared
 * memory when it has more than 16384 columns.  scale must be positive and finite
 * (the row maximum is taken on the unscaled scores, which a positive scale keeps
 * in order): ATTN_ERR_INVALID_ARG otherwise.
 * Errors: ATTN_ERR_INVALID_ARG, ATTN_ERR_UNSUPPORTED_SHAPE, ATTN_ERR_MISALIGNED, ATTN_ERR_CUDA.
 */
int softmax_rows_forward(const void *s, void *p, long long rows, int cols, float scale, void *cuda_stream);

/*
 * Unfused attention, for comparison with attn_forward: S = Q K^T into
 * `scores` (caller-owned, B*H*L*L bf16), softmax(S / sqrt(d)) in place, then
 * O = P V.  q, k, v, o as in attn_forward; L a multiple of 8, at most 32768;
 * d a multiple of 8.  Three kernel launches.
 * Errors: as gemm_forward and softmax_rows_forward, ATTN_ERR_INVALID_ARG if
 * scores_bytes < B*H*L*L*2.
 */
int attn_forward_unfused(const void *q, const void *k, const void *v, void *o, void *scores, size_t scores_bytes,
                         int B, int H, int L, int d, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif  /* PAPER_2609_10937_GEMM_H_ */
