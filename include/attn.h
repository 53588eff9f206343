/*
 * attn.h -- C ABI of the B200 fused-attention library (libattn_b200.so).
 *
 * One operation: the fused attention forward pass of the paper's Section
 * "Fused Attention",  O = softmax(Q K^T / sqrt(d)) V,  evaluated with
 * Algorithm 1 (K/V tiles streamed through an online softmax, the L x L score
 * matrix never written to memory), with tile sizes derived in closed form from
 * a hardware descriptor (Sections "Hardware Model" and "Tile Derivation")
 * instead of being searched.
 *
 * Conventions
 *   - Plain C types only; no exceptions cross the boundary; every function
 *     returns an attn_status (0 = success, negative = error) unless noted.
 *   - q, k, v, o are DEVICE pointers to contiguous [B][H][L][d] bf16 arrays
 *     (d fastest), 16-byte aligned.  Scale 1/sqrt(d), fp32 accumulation, bf16
 *     (round-to-nearest-even) output.  attn_forward is non-causal (the paper's
 *     operator); attn_forward_causal applies a triangular -inf mask.
 *   - The caller owns every buffer, including the workspace.  The library
 *     allocates no device memory and keeps no reference to q/k/v/o after a
 *     call returns.  attn_forward* are asynchronous on `cuda_stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream) and never
 *     synchronise.
 *   - Supported shapes: d in {64, 128}; any L >= 1 (a ragged last key tile is
 *     masked with -inf, never zero-padded; the paper's boundary note in Section
 *     "Online Softmax"), B, H >= 1.
 *   - Results are bitwise reproducible run to run (fixed merge order, no
 *     atomics on the output).
 */
#ifndef ATTN_B200_H_
#define ATTN_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum attn_status {
  ATTN_OK = 0,
  ATTN_ERR_INVALID_ARG = -1,       /* null pointer, non-positive size, bad struct_bytes   */
  ATTN_ERR_UNSUPPORTED_SHAPE = -2, /* d not in {64,128}, or B*H*L beyond the index range  */
  ATTN_ERR_MISALIGNED = -3,        /* a device pointer is not 16-byte aligned             */
  ATTN_ERR_ALIASING = -4,          /* o overlaps q, k or v                                */
  ATTN_ERR_INFEASIBLE_PLAN = -5,   /* no tile choice fits; see binding_constraint         */
  ATTN_ERR_WRONG_ARCH = -6,        /* current device is not compute capability 10.x       */
  ATTN_ERR_NEED_WORKSPACE = -7,    /* CTAs share Q tiles but no (large enough) workspace  */
  ATTN_ERR_CUDA = -8,              /* a CUDA runtime/driver call failed                   */
  ATTN_ERR_DEVICE_TIMEOUT = -9,    /* a bounded device-side wait expired                  */
  ATTN_ERR_BAD_TILES = -10,        /* tile override not among the compiled variants       */
  ATTN_ERR_SCRATCH_LIMIT = -11     /* problem needs more than the built-in scratch array  */
} attn_status;

/* Which capacity fixed the tile (the "binding constraint" returned by the
 * paper's derive_tiles / FeasibilityVisitor, Section "Tile Derivation"). */
typedef enum attn_binding {
  ATTN_BIND_NONE = 0,
  ATTN_BIND_SMEM = 1,  /* shared memory / local data share                       */
  ATTN_BIND_TMEM = 2,  /* tensor-memory columns                                  */
  ATTN_BIND_REG = 3,   /* register file                                          */
  ATTN_BIND_ATOM = 4,  /* largest N of one matrix instruction                    */
  ATTN_BIND_SHAPE = 5  /* problem shape not aligned to the atom                  */
} attn_binding;

/*
 * Hardware descriptor: only the quantities the derivation uses (the paper's
 * HardwareDescriptor / MFMAAtom listing, Section "Hardware Model").
 * acc_mem_columns == 0 describes a machine whose accumulators live in vector
 * registers (the paper's CDNA targets); > 0 describes tensor memory (B200).
 * Caller-owned plain data; set struct_bytes = sizeof(attn_hw_desc).
 *
 * The ovh_* fields are hardware facts in the same sense as the capacities: what
 * the start and the end of a CTA's work cost on this machine under each way of
 * sharing out the key axis, measured once per target, in units of one KV step of
 * the kernel (the occupancy step of the derivation compares critical paths in
 * KV steps).  Changing them re-runs the occupancy step like changing a capacity
 * re-runs the tile step.  hbm_gbps and peak_tflops feed the predicted time and
 * bound that attn_plan reports (attn_tiles.predicted_us, .bound).
 */
typedef struct attn_hw_desc {
  int32_t struct_bytes;
  int32_t num_units;           /* SMs / CUs                                           */
  int32_t local_mem_bytes;     /* on-chip scratch one CTA may use (SMEM opt-in / LDS) */
  int32_t regs_per_unit;       /* 32-bit registers per SM (0 if not modelled)         */
  int32_t max_regs_per_thread; /* architectural per-thread limit                      */
  int32_t simd_width;          /* warp / wavefront width                              */
  int32_t acc_mem_lanes;       /* tensor-memory lanes (128), 0 if none                */
  int32_t acc_mem_columns;     /* tensor-memory 32-bit columns (512), 0 if none       */
  int32_t atom_m;              /* rows of one matrix instruction (128 | 16)           */
  int32_t atom_n;              /* N granularity (16)                                  */
  int32_t atom_k;              /* K of one instruction (16 | 4)                       */
  int32_t atom_n_max;          /* largest N of one instruction (256 | 16)             */
  int32_t elem_bytes;          /* operand element size (2 = bf16, 4 = fp32)           */
  int32_t cache_bytes;         /* last-level cache shared by all units (L2); 0 if not modelled */
  int32_t max_clusters[8];     /* [k-1]: clusters of k CTAs (one CTA per unit, distributed shared    */
                               /* memory between them) that can be resident at once; 0: none        */
  /* cost of a CTA's start and end, in KV steps (B200 values in attn_hw_desc_b200) */
  int32_t ovh_whole_tile;      /* one CTA per whole Q tile, nothing to merge                         */
  int32_t ovh_cluster;         /* k CTAs per tile as one cluster, partials through distributed SMEM  */
  int32_t ovh_workspace;       /* k CTAs per tile, partials through the workspace (plus k / 2)       */
  int32_t ovh_ranges;          /* equal ranges of the (tile, step) line, fewer tiles than units      */
  int32_t ovh_persistent;      /* one persistent CTA per unit on an equal range, more tiles than units */
  int32_t ovh_tile_change;     /* a persistent CTA moving on to its next Q tile                      */
  int32_t ovh_causal_ranges;   /* causal, equal ranges: many short pieces per CTA                    */
  int32_t ovh_causal_cluster;  /* causal, k CTAs per tile as one cluster                             */
  double hbm_gbps;             /* HBM bandwidth, GB/s (nominal, or measured by the caller)           */
  double peak_tflops;          /* dense tensor peak for the operand type, TFLOP/s                    */
} attn_hw_desc;

/* Result of the closed-form derivation.  Caller-owned plain data. */
typedef struct attn_tiles {
  int32_t tile_q;         /* Q rows per CTA = n_q * atom_m                              */
  int32_t tile_kv;        /* K/V rows per streamed tile                                 */
  int32_t n_q;            /* Q sub-tiles per CTA (ping-pong partners), 1 or 2           */
  int32_t n_s;            /* score buffers per sub-tile (1)                             */
  int32_t kv_stages;      /* depth of the shared-memory K/V ring (one K or V tile each) */
  int32_t kv_splits;      /* ceil(ctas / tiles): CTAs sharing one Q tile along the key axis (1 for a persistent
                             grid of fewer CTAs than tiles; a tile at a range boundary is then still shared by two) */
  int32_t smem_bytes;     /* dynamic shared memory per CTA                              */
  int32_t tmem_columns;   /* tensor-memory columns allocated per CTA                    */
  int32_t regs_softmax;   /* register allowance of a softmax thread                     */
  int32_t threads;        /* threads per CTA                                            */
  int32_t tiles;          /* B * H * ceil(L / tile_q)                                   */
  int32_t ctas;           /* grid size: tiles, or fewer/more CTAs walking equal ranges of the (tile, step) line */
  float ctas_per_unit;    /* ctas / num_units                                           */
  float wave_efficiency;  /* ctas_per_unit / ceil(ctas_per_unit)                        */
  int32_t feasible;       /* 1 if a tile choice fits                                    */
  int32_t binding_constraint; /* attn_binding                                           */
  int32_t under_occupied; /* 1 if tiles < num_units (occupancy check of the derivation) */
  int32_t causal;         /* 1 if planned for causal attention (row i sees keys 0..i)   */
  int32_t cost_steps;     /* what the occupancy step minimised: KV steps on the longest CTA's path plus the
                             ovh_* cost of the chosen way of sharing out the key axis                      */
  int32_t bound;          /* 0: tensor time exceeds HBM time (predicted), 1: the reverse                   */
  float predicted_us;     /* max(cost_steps * FLOPs of one KV step / (peak_tflops / num_units),
                             compulsory bytes / hbm_gbps); 0 if the descriptor gives no peaks            */
} attn_tiles;

/* Built-in descriptor of one B200 (148 SMs, 227 KB SMEM opt-in, 64 K registers,
 * 128 x 512 tensor memory, tcgen05 kind::f16 atom 128 x N x 16; ovh_* = 2, 5, 8, 12,
 * 6, 1, 15, 6 KV steps as measured on B200; 7.7 TB/s and 2250 TFLOP/s nominal).  Host only. */
int attn_hw_desc_b200(attn_hw_desc *out);

/* Descriptor of CUDA device `device`, from cudaDeviceGetAttribute plus the
 * per-architecture constants above.  ATTN_ERR_WRONG_ARCH unless cc 10.x. */
int attn_hw_desc_query(int device, attn_hw_desc *out);

/*
 * Closed-form tile derivation (the paper's derive_tiles(desc, L, d); Section
 * "Tile Derivation": capacity constraints in a fixed order, then the occupancy
 * check, then atom alignment; Table 2 for the attention case).  Host only, no
 * CUDA calls, no search.  Fills *out and returns ATTN_OK even when the result
 * is infeasible (out->feasible == 0 and out->binding_constraint says why);
 * returns ATTN_ERR_INVALID_ARG for null pointers or a bad struct_bytes.
 * Occupancy step with fewer Q tiles than units (costs in KV steps per CTA, the
 * cheapest wins, ties to the earlier; the result is attn_tiles.cost_steps): one CTA
 * per tile, steps + ovh_whole_tile; k CTAs per tile along the keys as one
 * thread-block cluster, ceil(steps / k) + ovh_cluster (2 <= k <= 8, tiles * k <=
 * num_units, steps / k >= 2, max_clusters[k-1] >= tiles, landing areas fit); k CTAs
 * per tile through the workspace, ceil(steps / k) + ovh_workspace + k / 2 with
 * k = min(num_units / tiles, steps / 4); equal ranges of the (tile, step) line for
 * G = min(num_units, tiles * steps / 4) CTAs, ceil(tiles * steps / G) + ovh_ranges.
 * With at least as many tiles as units: one CTA per tile in whole waves,
 * ceil(tiles / units) * (steps + ovh_whole_tile), or -- only if the K and V of the
 * heads then in flight fit two thirds of cache_bytes -- one persistent CTA per unit
 * on an equal range, ceil(tiles * steps / units) + ovh_persistent +
 * ceil(tiles / units) * ovh_tile_change.
 */
int attn_plan(const attn_hw_desc *desc, int B, int H, int L, int d, attn_tiles *out);

/* Same derivation for causal attention (causal != 0): Q tile q needs only the key
 * steps up to its own last row, so the work per tile is unequal and the occupancy
 * step always deals the (Q tile, KV step) units out in equal ranges, one per unit.
 * Exception: k = 2..4 CTAs per tile as one cluster, each with a share of the tile's own key
 * steps, if tiles * k <= num_units, max_clusters[k-1] >= tiles, ceil(steps / k) >= 2, the
 * landing areas fit and ceil(steps / k) + ovh_causal_cluster < ceil((units + 3 * tiles) / G) +
 * ovh_causal_ranges (few short tiles: a CTA then has one piece instead of many short ones;
 * ctas == k * tiles).
 * (The paper treats non-causal attention only; this applies its -inf masking rule,
 * Section "Online Softmax", to a triangular mask.) */
int attn_plan_ex(const attn_hw_desc *desc, int B, int H, int L, int d, int causal, attn_tiles *out);

/* Bytes of workspace attn_forward* needs for this plan: 0 if every CTA owns exactly
 * one whole Q tile (ctas == tiles, not causal); otherwise 64 KB of arrival counters,
 * then two slots per CTA of partial outputs and row statistics for the merge
 * operator, Section "Online Softmax". */
size_t attn_workspace_bytes(const attn_tiles *tiles, int B, int H, int L, int d);

/* Registers a caller-owned device buffer as the workspace of `device` (pass
 * NULL, 0 to clear) and zeroes its first 64 KB (the arrival counters) with a
 * synchronous cudaMemset on the current device, which must be `device`.  The
 * buffer must stay valid until replaced; concurrent attn_forward calls on
 * different streams of one device must not share it (use attn_forward_ws with a
 * workspace per stream for that).  After ATTN_ERR_DEVICE_TIMEOUT the counters may
 * be non-zero: attn_last_device_status clears them when it reports the timeout, so
 * poll it before the workspace is used again. */
int attn_set_workspace(int device, void *dev_ptr, size_t bytes);

/*
 * Fused attention forward (Algorithm 1) with the closed-form default tiles for
 * the current device.  Asynchronous on cuda_stream.  Errors: INVALID_ARG,
 * UNSUPPORTED_SHAPE, MISALIGNED, ALIASING, WRONG_ARCH, INFEASIBLE_PLAN,
 * NEED_WORKSPACE (the plan's CTAs share Q tiles -- ctas != tiles, e.g. a key split
 * or equal ranges of the (tile, step) line; kv_splits may still be 1 -- and the
 * registered workspace is smaller than attn_workspace_bytes), CUDA.
 */
int attn_forward(const void *q, const void *k, const void *v, void *o,
                 int B, int H, int L, int d, void *cuda_stream);

/*
 * attn_forward (causal == 0) or attn_forward_causal (causal != 0) with the workspace and the status words of
 * THIS call instead of the device-wide ones: what two streams of one device need to run plans that share Q
 * tiles at the same time, and what attributes an expired device-side wait to the launch it happened in.
 *   workspace        DEVICE buffer, 16-byte aligned, at least attn_workspace_bytes for the plan (may be NULL
 *                    with workspace_bytes 0 when that is 0); caller-owned; must not be used by another call
 *                    that may run at the same time.  Its first 64 KB (arrival counters) must be zero before
 *                    the first launch that uses it -- attn_workspace_init queues that clearing on a stream --
 *                    and every launch that ends normally leaves them zero.
 *   status_dev       four DEVICE words, 16-byte aligned, zero before first use (attn_workspace_init clears
 *                    them too), or NULL: then an expired wait is recorded in the device-wide record that
 *                    attn_last_device_status reads.  attn_status_read(status_dev, workspace, stream, detail)
 *                    synchronises the stream, returns ATTN_ERR_DEVICE_TIMEOUT with the four words in detail
 *                    (as attn_last_device_status) if a wait expired, clears the words and -- an aborted
 *                    launch may leave counters non-zero -- the workspace's counters; ATTN_OK otherwise.
 * A uniform key split that cannot run as thread-block clusters is merged here by the last CTA of a tile to finish
 * (never by fixed roles, whose merging warps wait for CTAs that a second kernel on the device could keep from
 * starting); the output bits are the same.
 * The paper's operator and merge (Sections "Fused Attention", "Online Softmax") are unchanged; this is the
 * ownership rule of the boundary made explicit per call.  Errors as attn_forward; NEED_WORKSPACE if the
 * buffer is too small.
 */
int attn_workspace_init(void *workspace, size_t workspace_bytes, uint32_t *status_dev, void *cuda_stream);
int attn_forward_ws(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int d, int causal,
                    void *workspace, size_t workspace_bytes, uint32_t *status_dev, void *cuda_stream);
int attn_status_read(uint32_t *status_dev, void *workspace, void *cuda_stream, uint32_t *detail);

/*
 * The same with Lq query rows and Lk keys per head (q, o: [B][H][Lq][d]; k, v: [B][H][Lk][d]):
 * O = softmax(Q K^T / sqrt(d)) V with every query row attending to all Lk keys.  The paper's
 * operator is the case Lq == Lk; a block of query rows of a longer sequence is the case
 * q = Q + r0 * d, Lq = rows in the block (what attn_forward_host uses to overlap copies with
 * compute).  attn_plan_qk is the derivation for it (tiles from Lq, key steps from Lk).
 * Errors as attn_forward.
 */
int attn_plan_qk(const attn_hw_desc *desc, int B, int H, int Lq, int Lk, int d, attn_tiles *out);
int attn_forward_qk(const void *q, const void *k, const void *v, void *o,
                    int B, int H, int Lq, int Lk, int d, void *cuda_stream);

/*
 * Causal fused attention forward: as attn_forward, but row i attends to keys 0..i
 * only -- the scores of later keys are -inf before the softmax (the paper's rule
 * that masked elements are -inf, never zero, Section "Online Softmax", applied to
 * a triangular mask; the paper itself evaluates non-causal attention only).
 * Key steps wholly after a Q tile's last row are skipped, not computed and masked.
 * Always needs a registered workspace (attn_workspace_bytes of attn_plan_ex(...,1,...)).
 */
int attn_forward_causal(const void *q, const void *k, const void *v, void *o,
                        int B, int H, int L, int d, void *cuda_stream);

/* Same, with tile fields overridden (tile sweep only).  Honoured fields (0 keeps
 * the closed-form value): n_q (1|2), tile_kv (64|128), kv_stages (2..plan maximum),
 * kv_splits (that many CTAs per Q tile) or ctas (the grid size itself, from 1 up
 * to the number of (Q tile, KV step) units; a uniform split whose grid exceeds the SM count
 * is merged by the last CTA of a tile to finish, since fixed merge roles need every CTA resident), causal (non-zero selects causal
 * attention; a grid of 2, 3 or 4 CTAs per tile then runs as clusters that share out
 * each tile's own key steps, any other grid as equal ranges of the unit line).  ATTN_ERR_BAD_TILES if the combination was not compiled or does not
 * fit. */
int attn_forward_tiles(const void *q, const void *k, const void *v, void *o,
                       int B, int H, int L, int d, const attn_tiles *override_tiles,
                       void *cuda_stream);

/*
 * Non-pipelined variant of the same algorithm: one 128-row Q tile per CTA, a
 * single K/V stage, the two matrix products and the softmax strictly in
 * sequence, plain global stores.  Slow; exists so that two independently
 * scheduled kernels can be compared (the paper validates its two attention
 * kernels against each other, Section "MFMA Kernel").  tile_kv in {64, 128}.
 * If scores_out is non-NULL it receives the raw fp32 score tile Q_0 K_0^T of
 * (batch 0, head 0): [128][tile_kv] floats (unscaled), for layout tests.
 */
int attn_forward_simple(const void *q, const void *k, const void *v, void *o,
                        int B, int H, int L, int d, int tile_kv, float *scores_out,
                        void *cuda_stream);

/*
 * attn_forward (causal == 0) or attn_forward_causal (causal != 0) with the tiles
 * derived from a caller-supplied descriptor instead of the device's own: the
 * paper's portability claim -- changing the hardware descriptor re-runs the same
 * derivation, no code changes -- carried through to the launch.  `desc` must
 * describe the current device or a smaller machine of the same architecture
 * (no more compute units, local memory, registers or tensor-memory columns than
 * the device has; same instruction atom), else ATTN_ERR_INVALID_ARG; a plan that
 * no compiled kernel variant covers gives ATTN_ERR_BAD_TILES, one that does not
 * fit gives ATTN_ERR_INFEASIBLE_PLAN.  Workspace as for attn_forward, sized with
 * attn_workspace_bytes for the plan of that descriptor.  Other errors as
 * attn_forward.
 */
int attn_forward_desc(const attn_hw_desc *desc, const void *q, const void *k, const void *v, void *o,
                      int B, int H, int L, int d, int causal, void *cuda_stream);

/*
 * Host-buffer form of attn_forward (the end-to-end path of Figure 2: Q, K, V
 * come from host memory, R goes back to it).  q_host, k_host, v_host, o_host
 * are HOST pointers (pinned memory for the copies to be asynchronous) in the
 * same [B][H][L][d] bf16 layout; dev_scratch is a caller-owned DEVICE buffer of
 * at least 4 * B*H*L*d*2 bytes, 256-byte aligned, that receives the device
 * copies of q, k, v and o.  Queues three host-to-device copies, the forward
 * pass and one device-to-host copy on cuda_stream; does not synchronise.
 *
 * One long head (B * H == 1 and L >= 8192) is pipelined: the query rows go as two
 * blocks, ceil(L / 2) rows rounded up to 256 and the rest, each an independent
 * attn_forward_qk problem against all L keys, so that the second block's copy in
 * runs under the first block's kernel and the first block's result leaves under
 * the second block's kernel.  Those copies are queued on two streams the library
 * creates on the device's first such call; cuda_stream waits for them before the
 * call's work counts as done on it, so to the caller the call is still one unit
 * of work on cuda_stream.  Calls of this form are serialised by a lock while
 * they queue their work.
 *
 * Workspace: attn_forward_host_workspace_bytes (it covers the blocks' plans
 * as well as the unsplit one; 0 if the shape has no feasible plan).
 * Errors: as attn_forward, plus ATTN_ERR_INVALID_ARG if the scratch is small.
 */
size_t attn_forward_host_workspace_bytes(const attn_hw_desc *desc, int B, int H, int L, int d);
int attn_forward_host(const void *q_host, const void *k_host, const void *v_host, void *o_host,
                      int B, int H, int L, int d, void *dev_scratch, size_t dev_scratch_bytes,
                      void *cuda_stream);

/*
 * Allocation-free form of attn_forward.  (The paper has no counterpart: this is a
 * packaging variant of the same kernel, not another algorithm.)
 *
 * Who it is for: callers that are not allowed to obtain device memory at the
 * point where they run attention -- a serving loop whose memory budget was
 * fixed at start-up, code running under an allocator that must not be
 * re-entered, a plug-in that only ever receives its input and output buffers.
 * attn_forward needs a caller-supplied workspace whenever the plan splits the
 * key axis; such callers have nowhere to get one from.  Here the partial
 * results and arrival counters live in an array that is part of the library
 * image itself: ATTN_STATIC_SCRATCH_BYTES (about 37.6 MiB) of device memory,
 * held by every GPU that loads the library until the process exits.
 *
 * q, k, v, o, shapes, stream and results are exactly those of attn_forward (same
 * kernel, same closed-form plan, bitwise the same output).  The call makes no
 * cudaMalloc / cudaFree and calls no allocating library routine.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and remembers it; make that first call outside any
 *     stream capture.
 *   - Every call on a device shares the one array, and the array keeps whatever
 *     the previous call left in it: the counters that must start at zero are
 *     cleared on `cuda_stream` before each launch.  Two calls that overlap in
 *     time on one GPU (different streams, or another thread) race on it and give
 *     wrong results; serialise them.
 *   - ATTN_ERR_SCRATCH_LIMIT if the plan for this shape needs more scratch than
 *     ATTN_STATIC_SCRATCH_BYTES (never the case for the built-in B200 descriptor
 *     with d <= 128); other errors as attn_forward.
 */
#define ATTN_STATIC_SCRATCH_BYTES 39469056
int attn_forward_static_scratch(const void *q, const void *k, const void *v, void *o,
                                int B, int H, int L, int d, void *cuda_stream);

/* Synchronises cuda_stream and reports whether any bounded device-side wait
 * expired since the last query (ATTN_ERR_DEVICE_TIMEOUT) -- then detail[0..3]
 * (optional, may be NULL) receive code, role/barrier/step word, CTA index and
 * a spare word -- or ATTN_OK.  Clears the record. */
int attn_last_device_status(void *cuda_stream, uint32_t *detail);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper: part of the error
 * behaviour of this boundary).  Every wait inside the kernels -- on a barrier, a flag, a peer CTA --
 * gives up after a fixed cycle count (about half a second), records where, and lets the kernel
 * return, so that a lost signal shows as ATTN_ERR_DEVICE_TIMEOUT from attn_last_device_status
 * instead of a hung GPU.  This call queues, on cuda_stream, one warp that waits with that same
 * routine on a barrier nothing ever arrives at; it ends by itself when the limit runs out.
 * Afterwards attn_last_device_status reports ATTN_ERR_DEVICE_TIMEOUT with detail[1] =
 * role 5 << 24 | barrier 10 << 16 | ATTN_SELFTEST_STEP, and the context stays usable.
 * Errors: WRONG_ARCH, CUDA.
 */
#define ATTN_SELFTEST_STEP 0x7E57
int attn_selftest_wait_expiry(void *cuda_stream);
/* The same with the record going to four caller-owned DEVICE words (as attn_forward_ws's status_dev; NULL: the
 * device-wide record): shows that an expiry is attributed to the launch whose status words were given. */
int attn_selftest_wait_expiry_to(uint32_t *status_dev, void *cuda_stream);

/* Number of kernels the last attn_forward* call on this thread launched. */
int attn_last_launch_count(void);

/* CTAs per thread-block cluster of the last fused launch on this thread: k if the plan was a
 * uniform key split of k CTAs per Q tile and those were launched as one cluster each (their
 * partial results then travel through distributed shared memory), 0 otherwise. */
int attn_last_cluster_size(void);

/* Static description of a status code; never NULL. */
const char *attn_status_string(int status);

/* Last CUDA error text recorded by the library on this thread ("" if none). */
const char *attn_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_B200_H_ */
