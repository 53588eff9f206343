// C ABI of the fused-attention library: argument checks, closed-form plan,
// TMA tensor maps, kernel launches.  No device memory is allocated here.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "attn.h"
#include "attn_kernels.cuh"
#include "attn_plan_internal.h"
#include "gemm.h"
#include "gemm_kernels.cuh"

namespace {

thread_local char t_cuda_error[256] = "";
thread_local int t_launch_count = 0;
thread_local int t_cluster_size = 0;   // CTAs per thread-block cluster of the last fused launch (0: no clusters)

int cuda_fail(cudaError_t e, const char* what) {
  std::snprintf(t_cuda_error, sizeof t_cuda_error, "%s: %s", what, cudaGetErrorString(e));
  return ATTN_ERR_CUDA;
}
#define ATTN_CUDA_TRY(expr)                               \
  do {                                                    \
    cudaError_t e__ = (expr);                             \
    if (e__ != cudaSuccess) return cuda_fail(e__, #expr); \
  } while (0)

// ---- driver entry point for tensor-map encoding (no link-time libcuda dependency)
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// 3-D map over a contiguous [BH][L][d] bf16 tensor; box = (64 columns, box_rows rows, 1 head), 128-byte swizzle.
int make_tmap(CUtensorMap* m, const void* base, int BH, int L, int d, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) {
    std::snprintf(t_cuda_error, sizeof t_cuda_error, "cuTensorMapEncodeTiled entry point not found");
    return ATTN_ERR_CUDA;
  }
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)L, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)L * (cuuint64_t)d * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::snprintf(t_cuda_error, sizeof t_cuda_error, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return ATTN_ERR_CUDA;
  }
  return ATTN_OK;
}

// ---- per-device state: workspace registry and cached descriptor
constexpr int kMaxDevices = 64;
struct DeviceState {
  void* ws = nullptr;
  size_t ws_bytes = 0;
  bool arch_checked = false;
  bool arch_ok = false;
  attn_hw_desc desc;
  int resident[2][9] = {};     // [causal][k]: clusters of k CTAs that fit at once, + 1 (0 = not asked yet); guarded by g_mu
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mu;

int device_state(DeviceState** out) {
  int dev = 0;
  ATTN_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ATTN_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceState& s = g_dev[dev];
  if (!s.arch_checked) {
    int rc = attn_hw_desc_query(dev, &s.desc);
    if (rc == ATTN_ERR_CUDA) return rc;
    s.arch_ok = (rc == ATTN_OK);
    s.arch_checked = true;
  }
  *out = &s;
  return s.arch_ok ? ATTN_OK : ATTN_ERR_WRONG_ARCH;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
  return a0 < b0 + nb && b0 < a0 + na;
}

int check_args(const void* q, const void* k, const void* v, const void* o, int B, int H, int L, int d, int Lk = 0) {
  if (Lk == 0) Lk = L;
  if (!q || !k || !v || !o || B <= 0 || H <= 0 || L <= 0 || Lk <= 0 || d <= 0) return ATTN_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return ATTN_ERR_UNSUPPORTED_SHAPE;
  if ((long long)B * H * ((L + 127) / 128) > 0x3FFFFFFFLL) return ATTN_ERR_UNSUPPORTED_SHAPE;  // grid index range
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15u) return ATTN_ERR_MISALIGNED;
  if ((long long)B * H * ((Lk + 127) / 128) > 0x3FFFFFFFLL) return ATTN_ERR_UNSUPPORTED_SHAPE;
  const size_t bytes = (size_t)B * H * L * d * 2, kv_bytes = (size_t)B * H * Lk * d * 2;
  if (overlaps(o, bytes, q, bytes) || overlaps(o, bytes, k, kv_bytes) || overlaps(o, bytes, v, kv_bytes))
    return ATTN_ERR_ALIASING;
  return ATTN_OK;
}

template <int D, int TKV, int NQ>
int launch_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int Lk, const attn_tiles& t,
               float* ws, unsigned int* status, DeviceState* st, cudaStream_t stream, bool may_overlap) {
  using SM = attn::FwdSmem<D, TKV, NQ>;
  const int BH = B * H;
  CUtensorMap tq, tk, tv, to;
  int rc;
  if ((rc = make_tmap(&tq, q, BH, L, D, attn::kSub)) != ATTN_OK) return rc;
  if ((rc = make_tmap(&tk, k, BH, Lk, D, TKV)) != ATTN_OK) return rc;
  if ((rc = make_tmap(&tv, v, BH, Lk, D, TKV)) != ATTN_OK) return rc;
  if ((rc = make_tmap(&to, o, BH, L, D, 32)) != ATTN_OK) return rc;    // every warp stores its own 32 rows

  attn::FwdParams p;
  p.L = Lk;                                                       // keys per head (L: query rows per head)
  p.q_tiles = (L + NQ * attn::kSub - 1) / (NQ * attn::kSub);
  p.n_steps = (Lk + TKV - 1) / TKV;
  p.tiles = BH * p.q_tiles;
  p.stages = t.kv_stages;
  p.causal = t.causal ? 1 : 0;
  p.ratio = NQ * attn::kSub / TKV;
  p.head_units = attn::tile_prefix(p.n_steps, p.ratio, p.causal, p.q_tiles);
  p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D));
  p.o = reinterpret_cast<__nv_bfloat16*>(o);
  p.status = status;
  p.counters = reinterpret_cast<unsigned int*>(ws);                   // head of the workspace
  p.ws = ws ? ws + attn::kCounterBytes / sizeof(float) : nullptr;    // partial results follow
  int grid = t.ctas;
  p.seg_skip = 0;
  // One CTA per tile with more tiles than SMs: a persistent grid of one CTA per SM runs them in the same order.
  const int sms = st->desc.num_units;                      // of the device itself (the plan may be for a smaller machine)
  if (!p.causal && t.ctas == t.tiles) {
    if (sms > 0 && t.tiles > sms) {
      grid = sms;
      p.seg_skip = (long long)(grid - 1) * p.n_steps;
    }
  }
  const long long total_units = p.head_units * BH;
  // at least one KV step per CTA; when Q tiles are shared, the counters of every (CTA, sub-tile, warp) --
  // two each -- must fit the counter block
  if (grid < 1 || (long long)grid > total_units) return ATTN_ERR_BAD_TILES;
  if (ws && (size_t)grid * NQ * 8 > attn::kCounterBytes / sizeof(unsigned int)) return ATTN_ERR_BAD_TILES;
  const int smem = SM::total(t.kv_stages);
  // uniform key split (k CTAs per tile, all parts of a tile finish together): the instantiation with fixed merge roles.
  // Its merging warps wait for the other CTAs of their tile, so every CTA of the grid must be resident at once (one
  // CTA per SM); a larger grid takes the instantiation in which the last CTA to finish merges and nobody waits for a
  // CTA that has not started.  The same holds for a launch that may run beside another one of its kind on the same
  // device (attn_forward_ws: two such kernels could each hold part of the SMs and wait for CTAs that cannot start);
  // thread-block clusters are scheduled as a whole and stay in use there.
  const bool eager = !p.causal && t.ctas > t.tiles && t.ctas % t.tiles == 0 && grid <= sms;
  const bool wait_roles_ok = !may_overlap;
  auto launch = [&](auto kern) -> int {
    ATTN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    kern<<<grid, 512, smem, stream>>>(tq, tk, tv, to, p);
    return ATTN_OK;
  };
  // Uniform key split with few parts: the k CTAs of a tile are launched as one thread-block cluster and exchange
  // their partial results through distributed shared memory (landing areas in the K/V ring: the groups of rows one
  // CTA merges, times the k-1 parts it receives for each, must fit).  Used only if all clusters can be resident at
  // once, like the CTAs of the plain launch; otherwise, or if the cluster launch is not possible, the partials go
  // through the workspace.
  p.cluster_k = 0;
  t_cluster_size = 0;
  auto launch_eager = [&](auto kern, auto kern_cluster) -> int {
    ATTN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    ATTN_CUDA_TRY(cudaFuncSetAttribute(kern_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int kk = t.ctas / t.tiles;
    const size_t landing = (size_t)((4 * NQ + kk - 1) / kk) * (kk - 1) * (32 * D * 4 + 256);
    if (kk >= 2 && kk <= 8 && landing <= (size_t)t.kv_stages * SM::kStageBytes) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(grid);
      cfg.blockDim = dim3(512);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = kk;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int n_res;
      {
        std::lock_guard<std::mutex> lk(g_mu);
        if (st->resident[0][kk] == 0) {
          int n = 0;
          if (cudaOccupancyMaxActiveClusters(&n, kern_cluster, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
          st->resident[0][kk] = n + 1;
        }
        n_res = st->resident[0][kk] - 1;
      }
      if ((long long)n_res * kk >= grid) {
        attn::FwdParams pc = p;
        pc.cluster_k = kk;
        if (cudaLaunchKernelEx(&cfg, kern_cluster, tq, tk, tv, to, pc) == cudaSuccess) {
          t_cluster_size = kk;
          return ATTN_OK;
        }
        (void)cudaGetLastError();                         // fall through to the plain launch
      }
    }
    if (!wait_roles_ok) return ATTN_ERR_BAD_TILES;        // (marker: the caller launches the last-finisher instantiation)
    kern<<<grid, 512, smem, stream>>>(tq, tk, tv, to, p);
    return ATTN_OK;
  };
  const int ck = (t.tiles > 0 && t.ctas % t.tiles == 0) ? t.ctas / t.tiles : 0;
  const size_t c_landing = ck > 2 ? (size_t)((4 * NQ + ck - 1) / ck) * (ck - 1) * (32 * D * 4 + 256) : 0;
  if (p.causal && ck >= 2 && ck <= 4 && p.ratio >= 2 && c_landing <= (size_t)t.kv_stages * SM::kStageBytes) {
    // causal, ck CTAs per tile as one cluster: each a share of the tile's own key steps (the only way to run this grid)
    auto kern = attn::attn_fwd_kernel<D, TKV, NQ, true, true, true>;
    ATTN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(512);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ck;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    attn::FwdParams pc = p;
    pc.cluster_k = ck;
    pc.seg_skip = -ck;
    // all clusters resident at once, else (or if the cluster launch fails) the same grid as equal ranges
    int n_res = 0;
    {
      std::lock_guard<std::mutex> lk(g_mu);
      if (st->resident[1][ck] == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
        st->resident[1][ck] = n + 1;
      }
      n_res = st->resident[1][ck] - 1;
    }
    if ((long long)n_res * ck >= grid && cudaLaunchKernelEx(&cfg, kern, tq, tk, tv, to, pc) == cudaSuccess) {
      t_cluster_size = ck;
      rc = ATTN_OK;
    } else {
      (void)cudaGetLastError();
      rc = launch(attn::attn_fwd_kernel<D, TKV, NQ, true, false>);
    }
  } else if (p.causal) rc = launch(attn::attn_fwd_kernel<D, TKV, NQ, true, false>);
  else if (eager) {
    rc = launch_eager(attn::attn_fwd_kernel<D, TKV, NQ, false, true>, attn::attn_fwd_kernel<D, TKV, NQ, false, true, true>);
    if (rc == ATTN_ERR_BAD_TILES && !wait_roles_ok) rc = launch(attn::attn_fwd_kernel<D, TKV, NQ, false, false>);
  } else rc = launch(attn::attn_fwd_kernel<D, TKV, NQ, false, false>);
  if (rc != ATTN_OK) return rc;
  ATTN_CUDA_TRY(cudaGetLastError());
  t_launch_count = 1;
  return ATTN_OK;
}

int dispatch_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d,
                 const attn_tiles& t, float* ws, unsigned int* status, DeviceState* st, cudaStream_t s, int Lk = 0,
                 bool may_overlap = false) {
  if (Lk == 0) Lk = L;
#define ATTN_CASE(D_, TKV_, NQ_) \
  if (d == D_ && t.tile_kv == TKV_ && t.n_q == NQ_) \
    return launch_fwd<D_, TKV_, NQ_>(q, k, v, o, B, H, L, Lk, t, ws, status, st, s, may_overlap);
  ATTN_CASE(128, 128, 2)
  ATTN_CASE(128, 64, 2)
  ATTN_CASE(128, 128, 1)
  ATTN_CASE(128, 64, 1)
  ATTN_CASE(64, 128, 2)
  ATTN_CASE(64, 64, 2)
  ATTN_CASE(64, 128, 1)
  ATTN_CASE(64, 64, 1)
#undef ATTN_CASE
  return ATTN_ERR_BAD_TILES;
}

// A plan needs the workspace unless every CTA owns exactly one whole Q tile.
bool plan_needs_workspace(const attn_tiles& t) { return t.causal != 0 || t.ctas != t.tiles; }

// A workspace handed to one call (attn_forward_ws) instead of the one registered for the device.
struct CallWorkspace {
  void* ws;
  size_t bytes;
  unsigned int* status;
};

int forward_impl(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d, int causal,
                 const attn_tiles* ovr, void* cuda_stream, const attn_hw_desc* plan_desc = nullptr, int Lk = 0,
                 const CallWorkspace* call_ws = nullptr) {
  t_launch_count = 0;
  if (Lk == 0) Lk = L;                       // keys per head; L is the number of query rows per head
  int rc = check_args(q, k, v, o, B, H, L, d, Lk);
  if (rc != ATTN_OK) return rc;
  if (Lk != L && (causal || (ovr && ovr->causal))) return ATTN_ERR_UNSUPPORTED_SHAPE;
  DeviceState* st = nullptr;
  if ((rc = device_state(&st)) != ATTN_OK) return rc;
  if (ovr && ovr->causal) causal = 1;
  if (plan_desc) {
    // a caller-supplied descriptor must describe this device or a smaller machine of the same architecture
    const attn_hw_desc& a = *plan_desc;
    const attn_hw_desc& dv = st->desc;
    if (a.struct_bytes != (int32_t)sizeof(attn_hw_desc)) return ATTN_ERR_INVALID_ARG;
    if (a.num_units < 1 || a.num_units > dv.num_units || a.local_mem_bytes > dv.local_mem_bytes ||
        a.regs_per_unit > dv.regs_per_unit || a.acc_mem_columns > dv.acc_mem_columns || a.acc_mem_columns <= 0 ||
        a.acc_mem_lanes != dv.acc_mem_lanes || a.atom_m != dv.atom_m || a.atom_n != dv.atom_n || a.atom_k != dv.atom_k ||
        a.atom_n_max > dv.atom_n_max || a.elem_bytes != dv.elem_bytes || a.simd_width != dv.simd_width)
      return ATTN_ERR_INVALID_ARG;
  }
  const attn_hw_desc& desc = plan_desc ? *plan_desc : st->desc;
  attn_tiles t;
  if ((rc = attn_internal::plan_qk(&desc, B, H, L, Lk, d, causal, &t)) != ATTN_OK) return rc;
  if (!t.feasible) return ATTN_ERR_INFEASIBLE_PLAN;
  if (ovr) {
    if (ovr->n_q > 0) t.n_q = ovr->n_q;
    if (ovr->tile_kv > 0) t.tile_kv = ovr->tile_kv;
    if (t.n_q != 1 && t.n_q != 2) return ATTN_ERR_BAD_TILES;
    if (t.tile_kv != 64 && t.tile_kv != 128) return ATTN_ERR_BAD_TILES;
    const int q_bytes = t.n_q * 128 * d * 2, stage = t.tile_kv * d * 2;
    const int reserve = 3072 + t.n_q * 128 * 128;   // barriers etc. + output staging (see FwdSmem)
    int max_stages = (desc.local_mem_bytes - q_bytes - reserve) / stage;
    if (max_stages > attn::kMaxStages) max_stages = attn::kMaxStages;
    t.kv_stages = ovr->kv_stages > 0 ? ovr->kv_stages : max_stages;
    if (t.kv_stages < 2 || t.kv_stages > max_stages) return ATTN_ERR_BAD_TILES;
    t.tile_q = t.n_q * 128;
    t.tiles = B * H * ((L + t.tile_q - 1) / t.tile_q);
    // grid: ctas if given, else kv_splits CTAs per Q tile if given, else the planner's occupancy rule
    // re-applied to the overridden tile shape
    const int steps = (Lk + t.tile_kv - 1) / t.tile_kv;
    if (ovr->ctas > 0) {
      t.ctas = ovr->ctas;
    } else if (ovr->kv_splits > 0) {
      t.ctas = t.tiles * ovr->kv_splits;
    } else {
      t.ctas = attn_internal::grid_size(desc, B * H, (L + t.tile_q - 1) / t.tile_q, steps, t.tile_q / t.tile_kv, causal,
                                        2LL * Lk * d * desc.elem_bytes, 4 * t.n_q, d, (long long)t.kv_stages * stage).ctas;
    }
    t.kv_splits = (t.ctas + t.tiles - 1) / t.tiles;
    if (t.ctas < 1) return ATTN_ERR_BAD_TILES;
    t.smem_bytes = q_bytes + t.kv_stages * stage + reserve;
  }
  float* ws = nullptr;
  if (plan_needs_workspace(t)) {
    const size_t need = attn_workspace_bytes(&t, B, H, L, d);
    if (call_ws) {
      if (!call_ws->ws || call_ws->bytes < need) return ATTN_ERR_NEED_WORKSPACE;
      ws = static_cast<float*>(call_ws->ws);
    } else {
      std::lock_guard<std::mutex> lk(g_mu);
      if (!st->ws || st->ws_bytes < need) return ATTN_ERR_NEED_WORKSPACE;
      ws = static_cast<float*>(st->ws);
    }
  }
  return dispatch_fwd(q, k, v, o, B, H, L, d, t, ws, call_ws ? call_ws->status : nullptr, st,
                      static_cast<cudaStream_t>(cuda_stream), Lk, call_ws != nullptr);
}

template <int D, int TKV>
int launch_simple(const void* q, const void* k, const void* v, void* o, int B, int H, int L, float* scores_out,
                  cudaStream_t stream) {
  const int BH = B * H;
  CUtensorMap tq, tk, tv;
  int rc;
  if ((rc = make_tmap(&tq, q, BH, L, D, attn::kSub)) != ATTN_OK) return rc;
  if ((rc = make_tmap(&tk, k, BH, L, D, TKV)) != ATTN_OK) return rc;
  if ((rc = make_tmap(&tv, v, BH, L, D, TKV)) != ATTN_OK) return rc;
  const int smem = attn::kSub * D * 2 + 2 * TKV * D * 2 + 1024;
  auto kern = attn::attn_fwd_simple_kernel<D, TKV>;
  ATTN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  const float scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)D));
  dim3 grid((L + attn::kSub - 1) / attn::kSub, BH);
  kern<<<grid, 128, smem, stream>>>(tq, tk, tv, reinterpret_cast<__nv_bfloat16*>(o), L, scale_log2, scores_out);
  ATTN_CUDA_TRY(cudaGetLastError());
  t_launch_count = 1;
  return ATTN_OK;
}

}  // namespace

extern "C" int attn_hw_desc_query(int device, attn_hw_desc* out) {
  if (!out) return ATTN_ERR_INVALID_ARG;
  int major = 0, minor = 0, sms = 0, smem_optin = 0, regs = 0, clock_khz = 0;
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, device));
  if (major != 10) return ATTN_ERR_WRONG_ARCH;
  attn_hw_desc_b200(out);  // per-architecture constants (tensor memory, atom shapes)
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&regs, cudaDevAttrMaxRegistersPerMultiprocessor, device));
  int l2 = 0;
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device));
  if (l2 > 0) out->cache_bytes = l2;
  ATTN_CUDA_TRY(cudaDeviceGetAttribute(&clock_khz, cudaDevAttrClockRate, device));
  out->num_units = sms;
  out->local_mem_bytes = smem_optin;
  out->regs_per_unit = regs;
  // dense bf16: 8192 FLOP per clock per SM at the device's maximum SM clock
  out->peak_tflops = 8192.0 * sms * (clock_khz * 1e3) / 1e12;
  // Resident clusters of k CTAs, asked for the kernel that uses them at its largest shared-memory footprint.
  {
    int cur = 0;
    ATTN_CUDA_TRY(cudaGetDevice(&cur));
    if (cur != device) ATTN_CUDA_TRY(cudaSetDevice(device));
    auto kern = attn::attn_fwd_kernel<128, 128, 2, false, true, true>;
    const int smem = attn::FwdSmem<128, 128, 2>::total(4);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    for (int k = 1; k <= 8; ++k) {
      int n = 0;
      if (e == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(sms / k * k));
        cfg.blockDim = dim3(512);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = k;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) n = 0;
      }
      out->max_clusters[k - 1] = n;
    }
    (void)cudaGetLastError();
    if (cur != device) ATTN_CUDA_TRY(cudaSetDevice(cur));
  }
  return ATTN_OK;
}

extern "C" int attn_set_workspace(int device, void* dev_ptr, size_t bytes) {
  if (device < 0 || device >= kMaxDevices) return ATTN_ERR_INVALID_ARG;
  if (dev_ptr && ((uintptr_t)dev_ptr & 15u)) return ATTN_ERR_MISALIGNED;
  if (dev_ptr && bytes >= (size_t)attn::kCounterBytes) {
    // arrival counters at the head of the workspace start at zero; kernels leave them at zero
    ATTN_CUDA_TRY(cudaMemset(dev_ptr, 0, attn::kCounterBytes));
  }
  std::lock_guard<std::mutex> lk(g_mu);
  g_dev[device].ws = dev_ptr;
  g_dev[device].ws_bytes = dev_ptr ? bytes : 0;
  return ATTN_OK;
}

extern "C" int attn_forward(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d,
                            void* cuda_stream) {
  return forward_impl(q, k, v, o, B, H, L, d, 0, nullptr, cuda_stream);
}

extern "C" int attn_workspace_init(void* workspace, size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  if (!workspace && !status_dev) return ATTN_ERR_INVALID_ARG;
  if (workspace && (((uintptr_t)workspace & 15u) || workspace_bytes < (size_t)attn::kCounterBytes)) return ATTN_ERR_INVALID_ARG;
  if (status_dev && ((uintptr_t)status_dev & 15u)) return ATTN_ERR_MISALIGNED;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (workspace) ATTN_CUDA_TRY(cudaMemsetAsync(workspace, 0, attn::kCounterBytes, s));
  if (status_dev) ATTN_CUDA_TRY(cudaMemsetAsync(status_dev, 0, 4 * sizeof(uint32_t), s));
  return ATTN_OK;
}

extern "C" int attn_forward_ws(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d, int causal,
                               void* workspace, size_t workspace_bytes, uint32_t* status_dev, void* cuda_stream) {
  if (workspace && ((uintptr_t)workspace & 15u)) return ATTN_ERR_MISALIGNED;
  if (status_dev && ((uintptr_t)status_dev & 15u)) return ATTN_ERR_MISALIGNED;
  const CallWorkspace cw = {workspace, workspace ? workspace_bytes : 0, status_dev};
  return forward_impl(q, k, v, o, B, H, L, d, causal ? 1 : 0, nullptr, cuda_stream, nullptr, 0, &cw);
}

extern "C" int attn_status_read(uint32_t* status_dev, void* workspace, void* cuda_stream, uint32_t* detail) {
  if (!status_dev) return ATTN_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  ATTN_CUDA_TRY(cudaStreamSynchronize(s));
  unsigned int h[4] = {0, 0, 0, 0};
  ATTN_CUDA_TRY(cudaMemcpy(h, status_dev, sizeof h, cudaMemcpyDeviceToHost));
  if (detail)
    for (int i = 0; i < 4; ++i) detail[i] = h[i];
  if (h[0] == 0) return ATTN_OK;
  // the aborted launch may have left arrival counters non-zero
  ATTN_CUDA_TRY(cudaMemset(status_dev, 0, sizeof h));
  if (workspace) ATTN_CUDA_TRY(cudaMemset(workspace, 0, attn::kCounterBytes));
  return ATTN_ERR_DEVICE_TIMEOUT;
}

extern "C" int attn_forward_qk(const void* q, const void* k, const void* v, void* o, int B, int H, int Lq, int Lk, int d,
                               void* cuda_stream) {
  if (Lk <= 0) return ATTN_ERR_INVALID_ARG;
  return forward_impl(q, k, v, o, B, H, Lq, d, 0, nullptr, cuda_stream, nullptr, Lk);
}

extern "C" int attn_forward_causal(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d,
                                   void* cuda_stream) {
  return forward_impl(q, k, v, o, B, H, L, d, 1, nullptr, cuda_stream);
}

extern "C" int attn_forward_desc(const attn_hw_desc* desc, const void* q, const void* k, const void* v, void* o, int B, int H,
                                 int L, int d, int causal, void* cuda_stream) {
  if (!desc) return ATTN_ERR_INVALID_ARG;
  return forward_impl(q, k, v, o, B, H, L, d, causal ? 1 : 0, nullptr, cuda_stream, desc);
}

extern "C" int attn_forward_tiles(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d,
                                  const attn_tiles* override_tiles, void* cuda_stream) {
  return forward_impl(q, k, v, o, B, H, L, d, 0, override_tiles, cuda_stream);
}

extern "C" int attn_forward_simple(const void* q, const void* k, const void* v, void* o, int B, int H, int L, int d,
                                   int tile_kv, float* scores_out, void* cuda_stream) {
  t_launch_count = 0;
  int rc = check_args(q, k, v, o, B, H, L, d);
  if (rc != ATTN_OK) return rc;
  DeviceState* st = nullptr;
  if ((rc = device_state(&st)) != ATTN_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (d == 128 && tile_kv == 128) return launch_simple<128, 128>(q, k, v, o, B, H, L, scores_out, s);
  if (d == 128 && tile_kv == 64) return launch_simple<128, 64>(q, k, v, o, B, H, L, scores_out, s);
  if (d == 64 && tile_kv == 128) return launch_simple<64, 128>(q, k, v, o, B, H, L, scores_out, s);
  if (d == 64 && tile_kv == 64) return launch_simple<64, 64>(q, k, v, o, B, H, L, scores_out, s);
  return ATTN_ERR_BAD_TILES;
}

namespace {
// Streams and events of the host-buffer entry point's copy/compute pipeline, created on first use per device.
constexpr int kHostBlocksMax = 2;
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, done = nullptr, loaded[kHostBlocksMax] = {}, computed[kHostBlocksMax] = {};
  bool ok = false;
};
HostPipe g_pipe[kMaxDevices];
std::mutex g_pipe_mu;

HostPipe* host_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  HostPipe& hp = g_pipe[dev];
  if (!hp.ok) {
    bool good = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
                cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
                cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
                cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; good && i < kHostBlocksMax; ++i)
      good = cudaEventCreateWithFlags(&hp.loaded[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!good) { (void)cudaGetLastError(); return nullptr; }
    hp.ok = true;
  }
  return &hp;
}

// The blocks of query rows of the pipelined host path (one long head): kHostBlocksMax blocks of at least 4096
// rows, a multiple of 256 each but the last.  Returns the number of blocks, 0 if not pipelined.
// (Measured at L = 16384, d = 128: unsplit 0.450 ms, two blocks 0.398 ms, four blocks 0.475 ms -- a 4096-row
// launch against 16384 keys fills the machine worse than the copies it hides.)
int host_split(int B, int H, int L, int rows[kHostBlocksMax]) {
  if ((long long)B * H != 1 || L < 8192) return 0;
  const int n = std::min(kHostBlocksMax, L / 4096);
  const int per = ((L + n - 1) / n + 255) / 256 * 256;
  int left = L, c = 0;
  for (; c < n && left > 0; ++c) { rows[c] = std::min(per, left); left -= rows[c]; }
  return c;
}
}  // namespace

extern "C" size_t attn_forward_host_workspace_bytes(const attn_hw_desc* desc, int B, int H, int L, int d) {
  attn_tiles t;
  if (!desc || attn_plan(desc, B, H, L, d, &t) != ATTN_OK || !t.feasible) return 0;
  size_t need = attn_workspace_bytes(&t, B, H, L, d);
  int rows[kHostBlocksMax];
  const int blocks = host_split(B, H, L, rows);
  for (int c = 0; c < blocks; ++c)
    if (c == 0 || rows[c] != rows[c - 1])
      if (attn_plan_qk(desc, B, H, rows[c], L, d, &t) == ATTN_OK && t.feasible)
        need = std::max(need, attn_workspace_bytes(&t, B, H, rows[c], d));
  return need;
}

extern "C" int attn_forward_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, int B,
                                 int H, int L, int d, void* dev_scratch, size_t dev_scratch_bytes,
                                 void* cuda_stream) {
  if (!q_host || !k_host || !v_host || !o_host || !dev_scratch || B <= 0 || H <= 0 || L <= 0 || d <= 0)
    return ATTN_ERR_INVALID_ARG;
  const size_t bytes = (size_t)B * H * L * d * 2;
  if (dev_scratch_bytes < 4 * bytes || ((uintptr_t)dev_scratch & 255u)) return ATTN_ERR_INVALID_ARG;
  char* base = static_cast<char*>(dev_scratch);
  char *dq = base, *dk = base + bytes, *dv = base + 2 * bytes, *dout = base + 3 * bytes;
  int rc = check_args(dq, dk, dv, dout, B, H, L, d);
  if (rc != ATTN_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // One long head: the query rows go in blocks (every query row attends to all keys, so the blocks are
  // independent problems of attn_forward_qk).  K, V and the first block are copied, then each later block's copy
  // runs under the kernel before it and each block's result leaves under the kernel after it.
  // The copies use two streams of the library's own; the caller's stream sees the call as one unit of work.
  int rows[kHostBlocksMax];
  const int blocks = host_split(B, H, L, rows);
  if (blocks > 0) {
    std::lock_guard<std::mutex> lk(g_pipe_mu);
    HostPipe* hp = host_pipe();
    if (hp) {
      int first[kHostBlocksMax] = {};
      for (int c = 1; c < blocks; ++c) first[c] = first[c - 1] + rows[c - 1];
      const char *qh = static_cast<const char*>(q_host);
      char* oh = static_cast<char*>(o_host);
      const size_t row_bytes = (size_t)d * 2;
      ATTN_CUDA_TRY(cudaEventRecord(hp->start, s));
      ATTN_CUDA_TRY(cudaStreamWaitEvent(hp->in, hp->start, 0));
      ATTN_CUDA_TRY(cudaMemcpyAsync(dk, k_host, bytes, cudaMemcpyHostToDevice, hp->in));
      ATTN_CUDA_TRY(cudaMemcpyAsync(dv, v_host, bytes, cudaMemcpyHostToDevice, hp->in));
      for (int c = 0; c < blocks; ++c) {
        ATTN_CUDA_TRY(cudaMemcpyAsync(dq + first[c] * row_bytes, qh + first[c] * row_bytes, rows[c] * row_bytes,
                                      cudaMemcpyHostToDevice, hp->in));
        ATTN_CUDA_TRY(cudaEventRecord(hp->loaded[c], hp->in));
      }
      int launches = 0;
      for (int c = 0; c < blocks; ++c) {
        ATTN_CUDA_TRY(cudaStreamWaitEvent(s, hp->loaded[c], 0));
        rc = forward_impl(dq + first[c] * row_bytes, dk, dv, dout + first[c] * row_bytes, 1, 1, rows[c], d, 0, nullptr,
                          cuda_stream, nullptr, L);
        if (rc != ATTN_OK) break;
        launches += t_launch_count;
        ATTN_CUDA_TRY(cudaEventRecord(hp->computed[c], s));
        ATTN_CUDA_TRY(cudaStreamWaitEvent(hp->out, hp->computed[c], 0));
        ATTN_CUDA_TRY(cudaMemcpyAsync(oh + first[c] * row_bytes, dout + first[c] * row_bytes, rows[c] * row_bytes,
                                      cudaMemcpyDeviceToHost, hp->out));
      }
      // the caller's stream continues only after every copy of this call
      ATTN_CUDA_TRY(cudaEventRecord(hp->done, hp->out));
      ATTN_CUDA_TRY(cudaStreamWaitEvent(s, hp->done, 0));
      ATTN_CUDA_TRY(cudaStreamWaitEvent(s, hp->loaded[blocks - 1], 0));
      t_launch_count = launches;
      return rc;
    }
  }
  ATTN_CUDA_TRY(cudaMemcpyAsync(dq, q_host, bytes, cudaMemcpyHostToDevice, s));
  ATTN_CUDA_TRY(cudaMemcpyAsync(dk, k_host, bytes, cudaMemcpyHostToDevice, s));
  ATTN_CUDA_TRY(cudaMemcpyAsync(dv, v_host, bytes, cudaMemcpyHostToDevice, s));
  rc = forward_impl(dq, dk, dv, dout, B, H, L, d, 0, nullptr, cuda_stream);
  if (rc != ATTN_OK) return rc;
  ATTN_CUDA_TRY(cudaMemcpyAsync(o_host, dout, bytes, cudaMemcpyDeviceToHost, s));
  return ATTN_OK;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free entry point.  The scratch that a split plan needs (arrival counters followed by
// the partial outputs) is this file-scope device array instead of a caller-supplied workspace.
// In host code the name below is only a handle: its device address is obtained once per device
// with cudaGetSymbolAddress and that pointer is what the kernel receives.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_attn_static_scratch[ATTN_STATIC_SCRATCH_BYTES];

namespace {
void* g_static_scratch_ptr[kMaxDevices] = {};
std::mutex g_static_mu;

// Device address of the array on the current device, looked up on first use.
int static_scratch_address(void** out) {
  int dev = 0;
  ATTN_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ATTN_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (!g_static_scratch_ptr[dev]) {
    void* ptr = nullptr;
    ATTN_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_attn_static_scratch));
    if (!ptr) return ATTN_ERR_CUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  *out = g_static_scratch_ptr[dev];
  return ATTN_OK;
}
}  // namespace

extern "C" int attn_forward_static_scratch(const void* q, const void* k, const void* v, void* o, int B, int H, int L,
                                           int d, void* cuda_stream) {
  t_launch_count = 0;
  int rc = check_args(q, k, v, o, B, H, L, d);
  if (rc != ATTN_OK) return rc;
  DeviceState* st = nullptr;
  if ((rc = device_state(&st)) != ATTN_OK) return rc;
  attn_tiles t;
  if ((rc = attn_plan(&st->desc, B, H, L, d, &t)) != ATTN_OK) return rc;
  if (!t.feasible) return ATTN_ERR_INFEASIBLE_PLAN;
  void* scratch = nullptr;
  if ((rc = static_scratch_address(&scratch)) != ATTN_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (plan_needs_workspace(t)) {
    if (attn_workspace_bytes(&t, B, H, L, d) > (size_t)ATTN_STATIC_SCRATCH_BYTES) return ATTN_ERR_SCRATCH_LIMIT;
    // the array keeps the previous call's contents: the arrival counters must start at zero
    ATTN_CUDA_TRY(cudaMemsetAsync(scratch, 0, attn::kCounterBytes, stream));
  }
  return dispatch_fwd(q, k, v, o, B, H, L, d, t, static_cast<float*>(scratch), nullptr, st, stream);
}

namespace {
// One warp waits, with the kernels' bounded wait, on a barrier that nothing arrives at: the wait runs out
// after its cycle limit (about half a second), records the expiry and the kernel returns by itself.
__global__ void wait_expiry_selftest_kernel(unsigned int* status) {
  __shared__ uint64_t bar;
  __shared__ attn::AbortCell abort_cell;
  if (threadIdx.x == 0) {
    attn::abort_cell_init(&abort_cell, status);
    sm100::mbar_init(sm100::smem_u32(&bar), 1);
    sm100::fence_mbar_init();
  }
  __syncthreads();
  (void)attn::wait_bar_warp(sm100::smem_u32(&bar), 0, &abort_cell.flag,
                            attn::wait_info(attn::kRoleSimple, attn::kBarSync, ATTN_SELFTEST_STEP));
}
}  // namespace

extern "C" int attn_selftest_wait_expiry_to(uint32_t* status_dev, void* cuda_stream) {
  if (status_dev && ((uintptr_t)status_dev & 15u)) return ATTN_ERR_MISALIGNED;
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != ATTN_OK) return rc;
  wait_expiry_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(status_dev);
  ATTN_CUDA_TRY(cudaGetLastError());
  return ATTN_OK;
}

extern "C" int attn_selftest_wait_expiry(void* cuda_stream) { return attn_selftest_wait_expiry_to(nullptr, cuda_stream); }

extern "C" int attn_last_device_status(void* cuda_stream, uint32_t* detail) {
  ATTN_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
  unsigned int h[4] = {0, 0, 0, 0};
  ATTN_CUDA_TRY(cudaMemcpyFromSymbol(h, attn::g_attn_dev_status, sizeof h));
  if (detail)
    for (int i = 0; i < 4; ++i) detail[i] = h[i];
  if (h[0] == 0) return ATTN_OK;
  unsigned int z[4] = {0, 0, 0, 0};
  ATTN_CUDA_TRY(cudaMemcpyToSymbol(attn::g_attn_dev_status, z, sizeof z));
  {
    // an aborted launch may have left arrival counters non-zero
    int dev = 0;
    ATTN_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(g_mu);
    if (dev >= 0 && dev < kMaxDevices && g_dev[dev].ws && g_dev[dev].ws_bytes >= (size_t)attn::kCounterBytes)
      ATTN_CUDA_TRY(cudaMemset(g_dev[dev].ws, 0, attn::kCounterBytes));
  }
  return ATTN_ERR_DEVICE_TIMEOUT;
}

extern "C" int attn_last_launch_count(void) { return t_launch_count; }
extern "C" int attn_last_cluster_size(void) { return t_cluster_size; }

extern "C" const char* attn_last_cuda_error(void) { return t_cuda_error; }

extern "C" const char* attn_status_string(int status) {
  switch (status) {
    case ATTN_OK: return "ok";
    case ATTN_ERR_INVALID_ARG: return "invalid argument";
    case ATTN_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (need d in {64,128})";
    case ATTN_ERR_MISALIGNED: return "device pointer not 16-byte aligned";
    case ATTN_ERR_ALIASING: return "output overlaps an input";
    case ATTN_ERR_INFEASIBLE_PLAN: return "no feasible tile plan";
    case ATTN_ERR_WRONG_ARCH: return "device is not compute capability 10.x";
    case ATTN_ERR_NEED_WORKSPACE: return "CTAs share Q tiles: register a workspace with attn_set_workspace (or pass one to attn_forward_ws)";
    case ATTN_ERR_CUDA: return "CUDA error (see attn_last_cuda_error)";
    case ATTN_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case ATTN_ERR_BAD_TILES: return "tile override not available";
    case ATTN_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the library's built-in array holds";
    default: return "unknown status";
  }
}

// ===========================================================================
// Unfused path: matrix product, row softmax, three-kernel attention
// ===========================================================================
namespace {

// 3-D map over a contiguous [batch][rows][cols] bf16 tensor with a (64 columns, box_rows rows, 1) box.
int make_tmap_mat(CUtensorMap* m, const void* base, int batch, int rows, int cols, int box_rows) {
  return make_tmap(m, base, batch, rows, cols, box_rows);
}

int gemm_launch(const void* a, const void* b, void* c, int batch, int M, int N, int K, int b_layout, cudaStream_t stream,
                const gemm_tiles* ovr = nullptr) {
  if (!a || !b || !c || batch <= 0 || M <= 0 || N <= 0 || K <= 0) return ATTN_ERR_INVALID_ARG;
  if (b_layout != 0 && b_layout != 1) return ATTN_ERR_INVALID_ARG;
  if ((K & 7) || (N & 7)) return ATTN_ERR_UNSUPPORTED_SHAPE;
  if (((uintptr_t)a | (uintptr_t)b | (uintptr_t)c) & 15u) return ATTN_ERR_MISALIGNED;
  const size_t a_bytes = (size_t)batch * M * K * 2, b_bytes = (size_t)batch * N * K * 2, c_bytes = (size_t)batch * M * N * 2;
  if (overlaps(c, c_bytes, a, a_bytes) || overlaps(c, c_bytes, b, b_bytes)) return ATTN_ERR_ALIASING;
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != ATTN_OK) return rc;
  gemm_tiles t;
  if (ovr) {
    // tile sweep: the derivation re-run with pairs switched off (cta_pair 1) or with the other tile width
    attn_hw_desc d2 = st->desc;
    if (ovr->cta_pair == 1) d2.max_clusters[1] = 0;
    if ((rc = gemm_plan(&d2, batch, M, N, K, &t)) != ATTN_OK) return rc;
    if (ovr->cta_pair == 2 && t.cta_pair != 2) return ATTN_ERR_BAD_TILES;
    if (ovr->tile_n > 0 && ovr->tile_n != t.tile_n) {
      if (t.cta_pair != 2 || (ovr->tile_n != 128 && ovr->tile_n != 256)) return ATTN_ERR_BAD_TILES;
      t.tile_n = ovr->tile_n;
      const int stage = gemm::pair_stage_bytes(t.tile_n);
      t.stages = std::min(gemm::kMaxStages, (st->desc.local_mem_bytes - gemm::kPairOutBytes - gemm::kMiscBytes) / stage);
      t.tiles = batch * ((M + 255) / 256) * ((N + t.tile_n - 1) / t.tile_n);
      t.ctas = 2 * std::min(t.tiles, std::min(st->desc.max_clusters[1], st->desc.num_units / 2));
      t.acc_buffers = 512 / t.tile_n;
      t.tail_split = 0;
    }
    if (ovr->tail_split < 0) t.tail_split = 0;                 // (sweep: whole tiles in the last wave too)
  } else if ((rc = gemm_plan(&st->desc, batch, M, N, K, &t)) != ATTN_OK) {
    return rc;
  }
  // the kernels are compiled for exactly the tile shapes the derivation gives on this architecture
  if (!t.feasible || (t.n_sub != 1 && t.n_sub != 2) || t.tile_m != t.n_sub * attn::kSub || (t.tile_n != 128 && t.tile_n != 256) ||
      t.tile_k != gemm::kTileK || t.stages > gemm::kMaxStages || t.stages < 2)
    return ATTN_ERR_INFEASIBLE_PLAN;
  CUtensorMap ta, tb, tc;
  const bool pair = t.cta_pair == 2;
  // a CTA of a pair stages its own 128 rows of A and tile_n / 2 columns (rows, for [N][K]) of B
  if ((rc = make_tmap_mat(&ta, a, batch, M, K, attn::kSub)) != ATTN_OK) return rc;
  if (b_layout == 0) rc = make_tmap_mat(&tb, b, batch, K, N, gemm::kTileK);    // [K][N]: box 64 columns x 64 k-rows
  else rc = make_tmap_mat(&tb, b, batch, N, K, pair ? t.tile_n / 2 : t.tile_n);   // [N][K]: box 64 k-columns x rows of B
  if (rc != ATTN_OK) return rc;
  // (a pair's epilogue warps each store their own 32 rows)
  if ((rc = make_tmap_mat(&tc, c, batch, M, N, pair ? 32 : attn::kSub)) != ATTN_OK) return rc;
  gemm::GemmParams p;
  p.M = M; p.N = N; p.K = K; p.batch = batch;
  p.n_sub = t.n_sub;
  p.m_tiles = (M + t.tile_m - 1) / t.tile_m;
  p.n_tiles = (N + t.tile_n - 1) / t.tile_n;
  p.k_steps = (K + gemm::kTileK - 1) / gemm::kTileK;
  p.stages = t.stages;
  p.group_m = 1;
  p.tail_tiles = 0;
  p.stream_c = (long long)batch * M * N * 2 > (long long)st->desc.cache_bytes ? 1 : 0;
  if (pair) {
    // Bands of about sqrt(pairs) tile rows: the tiles in flight then share the fewest operand panels.  Only when the
    // operands of a tile outweigh its output eightfold (K >= 1024 for 256 x 256 tiles): below that the output
    // dominates the traffic, and tile rows walked whole write whole rows of C (16384 x 16384 x 64: 141 against 156 us).
    const int pairs = t.ctas / 2;
    int gm = 1;
    if ((long long)(t.tile_m + t.tile_n) * K >= 8LL * t.tile_m * t.tile_n)
      while ((gm + 1) * (gm + 1) <= pairs) ++gm;
    p.group_m = gm;
    p.tail_tiles = t.tail_split;
    const int smem = gemm::pair_smem_total(t.stages, t.tile_n);
    auto launch_pair = [&](auto kernel) -> int {
      ATTN_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)t.ctas);
      cfg.blockDim = dim3(gemm::kPairThreads);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      ATTN_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, ta, tb, tc, p));
      return ATTN_OK;
    };
    if (t.tile_n == 256) rc = (b_layout == 0) ? launch_pair(gemm::gemm_pair_kernel<true, 256>) : launch_pair(gemm::gemm_pair_kernel<false, 256>);
    else rc = (b_layout == 0) ? launch_pair(gemm::gemm_pair_kernel<true, 128>) : launch_pair(gemm::gemm_pair_kernel<false, 128>);
  } else {
    const int smem = gemm::smem_total(t.stages, t.tile_n);
    auto launch = [&](auto kernel) -> int {
      ATTN_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
      kernel<<<t.ctas, gemm::kThreads, smem, stream>>>(ta, tb, tc, p);
      return ATTN_OK;
    };
    if (t.tile_n == 256) rc = (b_layout == 0) ? launch(gemm::gemm_kernel<true, 256>) : launch(gemm::gemm_kernel<false, 256>);
    else rc = (b_layout == 0) ? launch(gemm::gemm_kernel<true, 128>) : launch(gemm::gemm_kernel<false, 128>);
  }
  if (rc != ATTN_OK) return rc;
  ATTN_CUDA_TRY(cudaGetLastError());
  ++t_launch_count;
  return ATTN_OK;
}

int softmax_launch(const void* s, void* pout, long long rows, int cols, float scale, cudaStream_t stream) {
  // the kernels take the row maximum on the raw scores and scale it afterwards: the scale must keep the order
  if (!s || !pout || rows <= 0 || cols <= 0 || !(scale > 0.0f) || !std::isfinite(scale)) return ATTN_ERR_INVALID_ARG;
  if ((cols & 7) || cols > 32768 || rows > 0x7FFFFFFFLL) return ATTN_ERR_UNSUPPORTED_SHAPE;
  if (((uintptr_t)s | (uintptr_t)pout) & 15u) return ATTN_ERR_MISALIGNED;
  const float scale_log2 = scale * 1.4426950408889634f;
  const int nvec = cols / 8;                        // 16-byte vectors per row
  const __nv_bfloat16* sp = static_cast<const __nv_bfloat16*>(s);
  __nv_bfloat16* pp = static_cast<__nv_bfloat16*>(pout);
  const dim3 grid((unsigned)rows);
  // threads x vectors per thread >= nvec.  Small blocks (128 or 256 threads, the row in up to 8 -- for the widest
  // rows 32 -- vectors per thread): several rows are then in flight per SM in different phases (load, reduce, store),
  // which one large block per row does not give (measured: 1024-thread blocks reach half the bandwidth).
  if (nvec <= 128) gemm::softmax_rows_kernel<1, 128><<<grid, 128, 0, stream>>>(sp, pp, cols, scale_log2);
  else if (nvec <= 256) gemm::softmax_rows_kernel<2, 128><<<grid, 128, 0, stream>>>(sp, pp, cols, scale_log2);
  else if (nvec <= 512) gemm::softmax_rows_kernel<4, 128><<<grid, 128, 0, stream>>>(sp, pp, cols, scale_log2);
  else if (nvec <= 1024) gemm::softmax_rows_kernel<4, 256><<<grid, 256, 0, stream>>>(sp, pp, cols, scale_log2);
  else if (nvec <= 2048) gemm::softmax_rows_kernel<8, 256><<<grid, 256, 0, stream>>>(sp, pp, cols, scale_log2);
  else {
    // wider than the registers of one block hold: the row is staged in shared memory (2 bytes per column)
    auto kern = gemm::softmax_rows_staged_kernel<256>;
    ATTN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536));
    kern<<<grid, 256, cols * 2, stream>>>(sp, pp, cols, scale_log2);
  }
  ATTN_CUDA_TRY(cudaGetLastError());
  ++t_launch_count;
  return ATTN_OK;
}

}  // namespace

extern "C" int gemm_forward(const void* a, const void* b, void* c, int batch, int M, int N, int K, int b_layout,
                            void* cuda_stream) {
  t_launch_count = 0;
  return gemm_launch(a, b, c, batch, M, N, K, b_layout, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int gemm_forward_tiles(const void* a, const void* b, void* c, int batch, int M, int N, int K, int b_layout,
                                  const gemm_tiles* override_tiles, void* cuda_stream) {
  t_launch_count = 0;
  return gemm_launch(a, b, c, batch, M, N, K, b_layout, static_cast<cudaStream_t>(cuda_stream), override_tiles);
}

extern "C" int softmax_rows_forward(const void* s, void* p, long long rows, int cols, float scale, void* cuda_stream) {
  t_launch_count = 0;
  return softmax_launch(s, p, rows, cols, scale, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int attn_forward_unfused(const void* q, const void* k, const void* v, void* o, void* scores, size_t scores_bytes,
                                    int B, int H, int L, int d, void* cuda_stream) {
  t_launch_count = 0;
  if (!q || !k || !v || !o || !scores || B <= 0 || H <= 0 || L <= 0 || d <= 0) return ATTN_ERR_INVALID_ARG;
  if ((L & 7) || (d & 7) || L > 32768) return ATTN_ERR_UNSUPPORTED_SHAPE;
  const size_t need = (size_t)B * H * L * L * 2;
  if (scores_bytes < need) return ATTN_ERR_INVALID_ARG;
  const size_t bytes = (size_t)B * H * L * d * 2;
  if (overlaps(o, bytes, q, bytes) || overlaps(o, bytes, k, bytes) || overlaps(o, bytes, v, bytes)) return ATTN_ERR_ALIASING;
  if (overlaps(scores, need, q, bytes) || overlaps(scores, need, k, bytes) || overlaps(scores, need, v, bytes) ||
      overlaps(scores, need, o, bytes))
    return ATTN_ERR_ALIASING;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int rc;
  if ((rc = gemm_launch(q, k, scores, B * H, L, L, d, 1, stream)) != ATTN_OK) return rc;           // S = Q K^T
  if ((rc = softmax_launch(scores, scores, (long long)B * H * L, L, 1.0f / std::sqrt((float)d), stream)) != ATTN_OK)
    return rc;                                                                                      // P = softmax(S / sqrt(d))
  return gemm_launch(scores, v, o, B * H, L, d, L, 0, stream);                                      // O = P V
}
