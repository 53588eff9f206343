"""ctypes binding of libattn_b200.so: argument marshalling only.

Every step of the attention path runs inside the library's CUDA kernels; this
module turns torch tensors into device pointers, keeps the caller-owned
workspace alive and raises on error codes.  There is no CPU fallback: if the
shared library is missing or fails to load, every call raises.
"""
from __future__ import annotations

import ctypes
import math
from pathlib import Path

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libattn_b200.so"

ATTN_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_MISALIGNED, ERR_ALIASING = -1, -2, -3, -4
ERR_INFEASIBLE_PLAN, ERR_WRONG_ARCH, ERR_NEED_WORKSPACE, ERR_CUDA = -5, -6, -7, -8
ERR_DEVICE_TIMEOUT, ERR_BAD_TILES, ERR_SCRATCH_LIMIT = -9, -10, -11
BIND_NAMES = ("none", "smem", "tmem", "reg", "atom", "shape")

EXPORTED_SYMBOLS = (
    "attn_hw_desc_b200", "attn_hw_desc_query", "attn_plan", "attn_plan_ex", "attn_workspace_bytes",
    "attn_set_workspace", "attn_workspace_init", "attn_forward_ws", "attn_status_read", "attn_forward", "attn_forward_causal", "attn_forward_tiles", "attn_forward_simple", "attn_forward_host", "attn_forward_host_workspace_bytes", "attn_forward_static_scratch", "attn_forward_desc", "attn_plan_qk", "attn_forward_qk",
    "attn_last_device_status", "attn_selftest_wait_expiry", "attn_selftest_wait_expiry_to",
    "attn_last_launch_count", "attn_last_cluster_size", "attn_status_string", "attn_last_cuda_error",
    "gemm_plan", "gemm_forward", "gemm_forward_tiles", "softmax_rows_forward", "attn_forward_unfused",
)


class AttnHwDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "struct_bytes", "num_units", "local_mem_bytes", "regs_per_unit", "max_regs_per_thread", "simd_width",
        "acc_mem_lanes", "acc_mem_columns", "atom_m", "atom_n", "atom_k", "atom_n_max", "elem_bytes", "cache_bytes",
    )] + [("max_clusters", ctypes.c_int32 * 8)] + [(n, ctypes.c_int32) for n in (
        "ovh_whole_tile", "ovh_cluster", "ovh_workspace", "ovh_ranges", "ovh_persistent", "ovh_tile_change",
        "ovh_causal_ranges", "ovh_causal_cluster",
    )] + [("hbm_gbps", ctypes.c_double), ("peak_tflops", ctypes.c_double)]


class AttnTiles(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "tile_q", "tile_kv", "n_q", "n_s", "kv_stages", "kv_splits", "smem_bytes", "tmem_columns", "regs_softmax",
        "threads", "tiles", "ctas",
    )] + [("ctas_per_unit", ctypes.c_float), ("wave_efficiency", ctypes.c_float)] + [
        (n, ctypes.c_int32) for n in ("feasible", "binding_constraint", "under_occupied", "causal", "cost_steps",
                                      "bound")] + [("predicted_us", ctypes.c_float)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class GemmTiles(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "tile_m", "tile_n", "tile_k", "n_sub", "stages", "smem_bytes", "tmem_columns", "tiles", "ctas", "feasible",
    )] + [("wave_efficiency", ctypes.c_float), ("binding_constraint", ctypes.c_int32), ("cta_pair", ctypes.c_int32),
          ("acc_buffers", ctypes.c_int32), ("tail_split", ctypes.c_int32)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class AttnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = status_string(code)
        if code == ERR_CUDA:
            msg += ": " + last_cuda_error()
        super().__init__(f"{where} failed: {msg} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2609_10937_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i32 = ctypes.c_void_p, ctypes.c_int
        L.attn_hw_desc_b200.argtypes = [ctypes.POINTER(AttnHwDesc)]
        L.attn_hw_desc_query.argtypes = [i32, ctypes.POINTER(AttnHwDesc)]
        L.attn_plan.argtypes = [ctypes.POINTER(AttnHwDesc), i32, i32, i32, i32, ctypes.POINTER(AttnTiles)]
        L.attn_plan_ex.argtypes = [ctypes.POINTER(AttnHwDesc), i32, i32, i32, i32, i32, ctypes.POINTER(AttnTiles)]
        L.attn_forward_causal.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
        L.attn_workspace_bytes.argtypes = [ctypes.POINTER(AttnTiles), i32, i32, i32, i32]
        L.attn_workspace_bytes.restype = ctypes.c_size_t
        L.attn_set_workspace.argtypes = [i32, vp, ctypes.c_size_t]
        L.attn_forward.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
        L.attn_workspace_init.argtypes = [vp, ctypes.c_size_t, vp, vp]
        L.attn_forward_ws.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, ctypes.c_size_t, vp, vp]
        L.attn_status_read.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_uint32)]
        L.attn_plan_qk.argtypes = [ctypes.POINTER(AttnHwDesc), i32, i32, i32, i32, i32, ctypes.POINTER(AttnTiles)]
        L.attn_forward_qk.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.attn_forward_tiles.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, ctypes.POINTER(AttnTiles), vp]
        L.attn_forward_simple.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
        L.attn_forward_host_workspace_bytes.argtypes = [ctypes.POINTER(AttnHwDesc), i32, i32, i32, i32]
        L.attn_forward_host_workspace_bytes.restype = ctypes.c_size_t
        L.attn_forward_host.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, ctypes.c_size_t, vp]
        L.attn_forward_static_scratch.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
        L.attn_forward_desc.argtypes = [ctypes.POINTER(AttnHwDesc), vp, vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.attn_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
        L.attn_selftest_wait_expiry.argtypes = [vp]
        L.attn_selftest_wait_expiry_to.argtypes = [vp, vp]
        L.attn_last_launch_count.argtypes = []
        L.attn_last_cluster_size.argtypes = []
        L.attn_status_string.argtypes = [i32]
        L.attn_status_string.restype = ctypes.c_char_p
        L.attn_last_cuda_error.argtypes = []
        L.attn_last_cuda_error.restype = ctypes.c_char_p
        L.gemm_plan.argtypes = [ctypes.POINTER(AttnHwDesc), i32, i32, i32, i32, ctypes.POINTER(GemmTiles)]
        L.gemm_forward.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.gemm_forward_tiles.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, ctypes.POINTER(GemmTiles), vp]
        L.softmax_rows_forward.argtypes = [vp, vp, ctypes.c_longlong, i32, ctypes.c_float, vp]
        L.attn_forward_unfused.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t, i32, i32, i32, i32, vp]
        for name in EXPORTED_SYMBOLS:
            getattr(L, name)
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().attn_status_string(int(code)).decode()


def last_cuda_error() -> str:
    return lib().attn_last_cuda_error().decode()


def _check(code: int, where: str) -> None:
    if code != ATTN_OK:
        raise AttnError(code, where)


def hw_desc_b200() -> AttnHwDesc:
    d = AttnHwDesc()
    _check(lib().attn_hw_desc_b200(ctypes.byref(d)), "attn_hw_desc_b200")
    return d


def hw_desc_query(device: int = 0) -> AttnHwDesc:
    d = AttnHwDesc()
    _check(lib().attn_hw_desc_query(int(device), ctypes.byref(d)), "attn_hw_desc_query")
    return d


def plan(desc: AttnHwDesc, B: int, H: int, L: int, d: int, causal: bool = False) -> AttnTiles:
    t = AttnTiles()
    if causal:
        _check(lib().attn_plan_ex(ctypes.byref(desc), B, H, L, d, 1, ctypes.byref(t)), "attn_plan_ex")
    else:
        _check(lib().attn_plan(ctypes.byref(desc), B, H, L, d, ctypes.byref(t)), "attn_plan")
    return t


def workspace_bytes(tiles: AttnTiles, B: int, H: int, L: int, d: int) -> int:
    return int(lib().attn_workspace_bytes(ctypes.byref(tiles), B, H, L, d))


# ---------------------------------------------------------------- torch side
_workspaces = {}   # device index -> torch uint8 tensor registered with the library
_descs = {}


def _device_desc(device_index: int) -> AttnHwDesc:
    if device_index not in _descs:
        _descs[device_index] = hw_desc_query(device_index)
    return _descs[device_index]


def ensure_workspace(device_index: int, nbytes: int) -> None:
    """Keeps a caller-side torch buffer of at least nbytes registered as the workspace."""
    import torch

    cur = _workspaces.get(device_index)
    if nbytes <= 0 or (cur is not None and cur.numel() >= nbytes):
        return
    buf = torch.empty(int(nbytes), dtype=torch.uint8, device=torch.device("cuda", device_index))
    _check(lib().attn_set_workspace(device_index, buf.data_ptr(), buf.numel()), "attn_set_workspace")
    _workspaces[device_index] = buf


def _prep(q, k, v, o):
    import torch

    if q.dtype != torch.bfloat16 or k.dtype != torch.bfloat16 or v.dtype != torch.bfloat16:
        raise TypeError("q, k, v must be torch.bfloat16")
    if q.dim() != 4 or q.shape != k.shape or q.shape != v.shape:
        raise ValueError("q, k, v must share the shape [B, H, L, d]")
    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise ValueError("q, k, v must be CUDA tensors (there is no CPU path)")
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
        raise ValueError("q, k, v must be contiguous [B][H][L][d]")
    if o is None:
        o = torch.empty_like(q)
    elif o.shape != q.shape or o.dtype != torch.bfloat16 or not o.is_contiguous() or o.device != q.device:
        raise ValueError("o must match q in shape, dtype, device and be contiguous")
    B, H, L, d = (int(x) for x in q.shape)
    dev = q.device.index if q.device.index is not None else torch.cuda.current_device()
    stream = torch.cuda.current_stream(q.device).cuda_stream
    return o, B, H, L, d, dev, stream


def forward(q, k, v, o=None, causal=False):
    """O = softmax(Q K^T / sqrt(d)) V with the closed-form default tiles (asynchronous).

    causal=True: row i attends to keys 0..i only."""
    import torch

    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    with torch.cuda.device(dev):
        t = plan(_device_desc(dev), B, H, L, d, causal)
        if t.feasible:
            ensure_workspace(dev, workspace_bytes(t, B, H, L, d))
        fn = lib().attn_forward_causal if causal else lib().attn_forward
        _check(fn(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, L, d, stream),
               "attn_forward_causal" if causal else "attn_forward")
    return o


def workspace_init(workspace, status=None):
    """Queues, on the current stream, the clearing of a workspace's arrival counters (its first 64 KB) and of a
    four-word status tensor; both are caller-owned CUDA tensors (uint8 / int32)."""
    import torch

    dev = workspace.device if workspace is not None else status.device
    with torch.cuda.device(dev):
        stream = torch.cuda.current_stream(dev).cuda_stream
        _check(lib().attn_workspace_init(workspace.data_ptr() if workspace is not None else None,
                                         workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                         status.data_ptr() if status is not None else None, stream),
               "attn_workspace_init")


def forward_ws(q, k, v, o=None, *, workspace=None, status=None, causal=False):
    """forward() with this call's own workspace (a CUDA uint8 tensor, counters cleared by workspace_init) and
    status words (a CUDA int32 tensor of four elements, or None for the device-wide record)."""
    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    import torch

    with torch.cuda.device(dev):
        _check(lib().attn_forward_ws(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, L, d,
                                     1 if causal else 0, workspace.data_ptr() if workspace is not None else None,
                                     workspace.numel() if workspace is not None else 0,
                                     status.data_ptr() if status is not None else None, stream), "attn_forward_ws")
    return o


def status_read(status, workspace=None):
    """Synchronises the current stream; returns (code, detail words) of a call's own status words."""
    import torch

    detail = (ctypes.c_uint32 * 4)()
    with torch.cuda.device(status.device):
        stream = torch.cuda.current_stream(status.device).cuda_stream
        code = lib().attn_status_read(status.data_ptr(), workspace.data_ptr() if workspace is not None else None,
                                      stream, detail)
    return int(code), [int(x) for x in detail]


def forward_static_scratch(q, k, v, o):
    """attn_forward without any allocation: the output tensor must be supplied, and the split-key
    scratch is the array built into the library (shared by all calls on a device; do not overlap calls)."""
    import torch

    if o is None:
        raise ValueError("the allocation-free entry point needs a caller-supplied output tensor")
    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    with torch.cuda.device(dev):
        _check(lib().attn_forward_static_scratch(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                                 B, H, L, d, stream), "attn_forward_static_scratch")
    return o


def forward_desc(desc: AttnHwDesc, q, k, v, o=None, causal=False):
    """forward() with the tiles derived from `desc` (this device or a smaller machine of its architecture)."""
    import torch

    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    with torch.cuda.device(dev):
        t = plan(desc, B, H, L, d, causal=causal)
        if t.feasible:
            ensure_workspace(dev, workspace_bytes(t, B, H, L, d))
        _check(lib().attn_forward_desc(ctypes.byref(desc), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                       B, H, L, d, 1 if causal else 0, stream), "attn_forward_desc")
    return o


def plan_qk(desc: AttnHwDesc, B: int, H: int, Lq: int, Lk: int, d: int) -> AttnTiles:
    t = AttnTiles()
    _check(lib().attn_plan_qk(ctypes.byref(desc), B, H, Lq, Lk, d, ctypes.byref(t)), "attn_plan_qk")
    return t


def forward_qk(q, k, v, o=None):
    """O = softmax(Q K^T / sqrt(d)) V for q [B, H, Lq, d] and k, v [B, H, Lk, d] (contiguous CUDA bf16)."""
    import torch

    for name, x in (("q", q), ("k", k), ("v", v)):
        if x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous() or x.dim() != 4:
            raise ValueError(f"{name} must be a contiguous CUDA bfloat16 tensor [B, H, L, d]")
    B, H, Lq, d = (int(x) for x in q.shape)
    Lk = int(k.shape[2])
    if tuple(k.shape) != (B, H, Lk, d) or tuple(v.shape) != (B, H, Lk, d):
        raise ValueError("k and v must be [B, H, Lk, d] with q's B, H and d")
    if o is None:
        o = torch.empty_like(q)
    dev = q.device.index if q.device.index is not None else torch.cuda.current_device()
    with torch.cuda.device(dev):
        t = plan_qk(_device_desc(dev), B, H, Lq, Lk, d)
        ensure_workspace(dev, workspace_bytes(t, B, H, Lq, d))
        stream = torch.cuda.current_stream(q.device).cuda_stream
        _check(lib().attn_forward_qk(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, Lq, Lk, d, stream),
               "attn_forward_qk")
    return o


def forward_tiles(q, k, v, o=None, *, n_q=0, tile_kv=0, kv_stages=0, kv_splits=0, ctas=0, causal=False):
    """Same with tile fields overridden (0 keeps the closed-form value); tile sweep only.

    kv_splits asks for that many CTAs per Q tile; ctas sets the grid size directly (any value from 1
    up to the number of (Q tile, KV step) units); causal selects causal attention."""
    import torch

    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    with torch.cuda.device(dev):
        desc = _device_desc(dev)
        base = plan(desc, B, H, L, d)
        ov = AttnTiles()
        ov.n_q, ov.tile_kv, ov.kv_stages, ov.kv_splits, ov.ctas = n_q, tile_kv, kv_stages, kv_splits, ctas
        ov.causal = 1 if causal else 0
        eff_nq = n_q or base.n_q
        tiles = B * H * math.ceil(L / (128 * eff_nq))
        w = AttnTiles()          # upper bound of what the call can need
        w.feasible, w.n_q, w.tiles, w.causal = 1, eff_nq, tiles, 1
        w.ctas = max(ctas, tiles * max(kv_splits, 1), desc.num_units, tiles)
        ensure_workspace(dev, workspace_bytes(w, B, H, L, d))
        _check(lib().attn_forward_tiles(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, L, d,
                                        ctypes.byref(ov), stream), "attn_forward_tiles")
    return o


def forward_simple(q, k, v, o=None, *, tile_kv=128, scores_out=None):
    """Non-pipelined variant; scores_out (fp32 [128, tile_kv], CUDA) receives Q_0 K_0^T of head 0."""
    import torch

    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    sp = None
    if scores_out is not None:
        if scores_out.dtype != torch.float32 or scores_out.numel() < 128 * tile_kv or not scores_out.is_cuda:
            raise ValueError("scores_out must be a CUDA fp32 tensor with at least 128*tile_kv elements")
        sp = scores_out.data_ptr()
    with torch.cuda.device(dev):
        _check(lib().attn_forward_simple(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, L, d,
                                         int(tile_kv), sp, stream), "attn_forward_simple")
    return o


def forward_host(q_host, k_host, v_host, o_host, dev_scratch):
    """Host-buffer entry point: pinned host bf16 tensors in, pinned host tensor out.

    dev_scratch is a caller-owned CUDA uint8 tensor of at least 4 * q.nbytes bytes.
    Copies and kernels are queued on the current stream; nothing is synchronised.
    """
    import torch

    B, H, L, d = (int(x) for x in q_host.shape)
    dev = dev_scratch.device.index
    stream = torch.cuda.current_stream(dev_scratch.device).cuda_stream
    with torch.cuda.device(dev):
        desc = _device_desc(dev)
        ensure_workspace(dev, int(lib().attn_forward_host_workspace_bytes(ctypes.byref(desc), B, H, L, d)))
        _check(lib().attn_forward_host(q_host.data_ptr(), k_host.data_ptr(), v_host.data_ptr(), o_host.data_ptr(),
                                       B, H, L, d, dev_scratch.data_ptr(), dev_scratch.numel(), stream),
               "attn_forward_host")
    return o_host


def last_device_status(device=None):
    """Synchronises the current stream; returns (code, detail words)."""
    import torch

    dev = torch.cuda.current_device() if device is None else device
    detail = (ctypes.c_uint32 * 4)()
    with torch.cuda.device(dev):
        stream = torch.cuda.current_stream().cuda_stream
        code = lib().attn_last_device_status(stream, detail)
    return int(code), [int(x) for x in detail]


def last_launch_count() -> int:
    return int(lib().attn_last_launch_count())


def last_cluster_size() -> int:
    """CTAs per thread-block cluster of the last fused launch (0: launched without clusters)."""
    return int(lib().attn_last_cluster_size())


# ----------------------------------------------------------------- unfused path
def gemm_plan(desc: AttnHwDesc, batch: int, M: int, N: int, K: int) -> GemmTiles:
    t = GemmTiles()
    _check(lib().gemm_plan(ctypes.byref(desc), batch, M, N, K, ctypes.byref(t)), "gemm_plan")
    return t


def _mat(x, name):
    import torch

    if x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous() or x.dim() not in (2, 3):
        raise ValueError(f"{name} must be a contiguous CUDA bfloat16 tensor of 2 or 3 dimensions")
    return x if x.dim() == 3 else x.unsqueeze(0)


def gemm(a, b, c=None, *, b_layout="kn", cta_pair=0, tile_n=0, tail_split=0):
    """C = A B ("kn": b is [.., K, N]) or C = A B^T ("nk": b is [.., N, K]); bf16 in and out, fp32 accumulation.

    cta_pair (1 | 2), tile_n (128 | 256) and tail_split (-1: whole tiles in the last wave) override the closed-form
    tiles (tile sweep only; 0 keeps them)."""
    import torch

    a3, b3 = _mat(a, "a"), _mat(b, "b")
    batch, M, K = (int(x) for x in a3.shape)
    if b_layout == "kn":
        kb, N = int(b3.shape[1]), int(b3.shape[2])
    elif b_layout == "nk":
        N, kb = int(b3.shape[1]), int(b3.shape[2])
    else:
        raise ValueError("b_layout is 'kn' or 'nk'")
    if kb != K or int(b3.shape[0]) != batch:
        raise ValueError("a and b do not agree in batch or K")
    if c is None:
        c = torch.empty((batch, M, N) if a.dim() == 3 else (M, N), dtype=torch.bfloat16, device=a.device)
    elif c.dtype != torch.bfloat16 or not c.is_contiguous() or c.numel() != batch * M * N or c.device != a.device:
        raise ValueError("c must be a contiguous bfloat16 tensor of batch*M*N elements on a's device")
    dev = a.device.index if a.device.index is not None else torch.cuda.current_device()
    with torch.cuda.device(dev):
        stream = torch.cuda.current_stream(a.device).cuda_stream
        if cta_pair or tile_n or tail_split:
            ov = GemmTiles()
            ov.cta_pair, ov.tile_n, ov.tail_split = int(cta_pair), int(tile_n), int(tail_split)
            _check(lib().gemm_forward_tiles(a.data_ptr(), b.data_ptr(), c.data_ptr(), batch, M, N, K,
                                            0 if b_layout == "kn" else 1, ctypes.byref(ov), stream), "gemm_forward_tiles")
        else:
            _check(lib().gemm_forward(a.data_ptr(), b.data_ptr(), c.data_ptr(), batch, M, N, K,
                                      0 if b_layout == "kn" else 1, stream), "gemm_forward")
    return c


def softmax_rows(s, scale: float, out=None):
    """Row softmax of scale * s over the last dimension (bf16, CUDA, contiguous); out may be s."""
    import torch

    if s.dtype != torch.bfloat16 or not s.is_cuda or not s.is_contiguous():
        raise ValueError("s must be a contiguous CUDA bfloat16 tensor")
    if out is None:
        out = torch.empty_like(s)
    elif out.shape != s.shape or out.dtype != s.dtype or not out.is_contiguous() or out.device != s.device:
        raise ValueError("out must match s")
    cols = int(s.shape[-1])
    rows = s.numel() // cols
    dev = s.device.index if s.device.index is not None else torch.cuda.current_device()
    with torch.cuda.device(dev):
        stream = torch.cuda.current_stream(s.device).cuda_stream
        _check(lib().softmax_rows_forward(s.data_ptr(), out.data_ptr(), rows, cols, float(scale), stream),
               "softmax_rows_forward")
    return out


def forward_unfused(q, k, v, scores, o=None):
    """The three-kernel path (S = Q K^T materialised in `scores`, softmax in place, P V); comparison only."""
    import torch

    o, B, H, L, d, dev, stream = _prep(q, k, v, o)
    if scores.dtype != torch.bfloat16 or not scores.is_cuda or not scores.is_contiguous() or scores.device != q.device:
        raise ValueError("scores must be a contiguous CUDA bfloat16 tensor on q's device")
    with torch.cuda.device(dev):
        _check(lib().attn_forward_unfused(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), scores.data_ptr(),
                                          scores.numel() * 2, B, H, L, d, stream), "attn_forward_unfused")
    return o
