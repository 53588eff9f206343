#!/usr/bin/env python
"""Benchmark of the fused-attention forward pass (one JSON line on stdout).

Metric: attention TFLOP/s = 4*B*H*L^2*d / time at the paper's headline shape
B=1, H=1, L=16384, d=128 (bf16 in/out, fp32 accumulate, non-causal), with the
closed-form default tiles.  A "step" is one whole forward pass (one kernel launch;
when the plan shares Q tiles between CTAs the partial results are merged inside
that kernel) over one synthetic batch.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun): every rank runs its own copy of the workload (weak
scaling, independent problems, no data-path collective); value is the total
work of all ranks over the slowest rank's time.

--impl reference times the fp64 CPU oracle on the host cores on a bounded row
sample of the same workload (rank 0 only).

Beside the headline the same line carries, each measured outside the headline's
timed region: `sustained` (the headline step back to back for seconds, clocks
sampled throughout), `configs` (every other benchmark configuration: time,
TFLOP/s, fraction of the measured peak, error against the oracle's sampled rows),
`unfused_baseline` and `gemm` (the paper's other workloads), `cpu_baseline`.

Other modes (each prints its own output and exits; used for the summaries under profiles/):
  --case NAME           time one named configuration only (small, for profiler captures)
  --tile-sweep NAME     every compiled tile variant around the closed-form default
  --grid-sweep          CTAs per Q tile and the equal-range grid over short and medium shapes
  --unfused-sweep       fused against the unfused three-kernel path over L, and the matrix product alone
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOAD = "cfg3"
WORKLOAD_TEXT = ("cfg3: attention fwd B=1,H=1,L=16384,d=128, non-causal, bf16 N(0,1), seed 0, scale 1/sqrt(d), "
                 "fp32 accumulate (one such problem per GPU)")
METRIC = "fused_attention_fwd_tflops_L16384_d128"
UNIT = "TFLOP/s"
L2_FLUSH_BYTES = 256 << 20
CONFIG = {"workload": WORKLOAD_TEXT}          # the same object in both arms
DRAM_CAPTURE_FILE = os.path.join("profiles", "attn_fwd_kernel_cfg3_dram_bytes.txt")

# Shapes of the grid sweep: fewer Q tiles than SMs, so the key axis has to be shared out (B, H, L, d).
GRID_SWEEP_SHAPES = [
    (1, 8, 2048, 128), (1, 4, 1024, 128), (1, 4, 2048, 128), (1, 4, 4096, 128), (1, 1, 2048, 128), (1, 1, 4096, 128),
    (1, 1, 8192, 128), (1, 1, 16384, 128), (1, 2, 8192, 128), (1, 3, 3000, 128), (1, 16, 1024, 128), (1, 2, 4096, 128),
    (1, 3, 4096, 128), (1, 4, 1024, 64), (1, 8, 2048, 64), (1, 1, 8192, 64), (1, 2, 4096, 64), (1, 16, 1024, 64),
]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def load_dram_capture():
    """DRAM bytes per launch of the dominant kernel from the profiler capture recorded under profiles/
    (a `key value` text file written beside the capture's summary); None if there is none."""
    path = os.path.join(ROOT, DRAM_CAPTURE_FILE)
    if not os.path.exists(path):
        return None
    rec = {}
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                key, _, val = line.partition(" ")
                rec[key] = val.strip()
    try:
        rec["bytes_per_launch"] = int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])
    except (KeyError, ValueError):
        return None
    return rec


def fused_bytes(B, H, L, d, elem_bytes):
    """Q, K, V read once and the result written once (the paper's HBM accounting for the fused kernel)."""
    return B * H * 4 * L * d * elem_bytes


def unfused_bytes(B, H, L, d, elem_bytes, score_bytes):
    """Scores written and read, probabilities written and read, plus Q, K, V and the result once (the paper's
    accounting for three separate passes: 4,329 MB at L = 16384, d = 128 with 4-byte elements)."""
    return B * H * (4 * L * L * score_bytes + 4 * L * d * elem_bytes)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs (read-only queries)."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index, period_ms=50):
        self.gpu_index = gpu_index
        self.period_ms = period_ms
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def window(self, t0, t1):
        """Summary of the samples taken between t0 and t1 (all samples if none fall inside)."""
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [l for t, l in self.lines if t0 <= t <= t1]
        chosen = inside or [l for t, l in self.lines if t0 - 0.05 <= t <= t1 + 0.1] or [l for _, l in self.lines]
        for line in chosen:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_mhz_min": min(sm) if sm else None, "power_w_max": max(power) if power else None,
                "samples": len(sm), "samples_inside_region": len(inside), "reasons": sorted(reasons)}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def cpu_baseline(case, q, k, v, target_seconds=12.0):
    """The fp64 oracle, as it stands, on the host cores, on a bounded row sample."""
    from oracle import attn_oracle as orc

    cores = orc.threads()
    probe = np.arange(0, case.L, max(1, case.L // 256), dtype=np.int32)[:256]
    t0 = time.perf_counter()
    orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, probe)
    dt = max(time.perf_counter() - t0, 1e-6)
    n_rows = int(min(case.L, max(256, len(probe) * target_seconds / dt)))
    rows = np.unique(np.linspace(0, case.L - 1, n_rows).astype(np.int32))
    # when even all rows take less than the target, the pass is repeated (at most 8 times) and the mean is reported
    reps, dt = 0, 0.0
    while reps < 8 and (reps == 0 or (len(rows) == case.L and dt < 0.8 * target_seconds)):
        t0 = time.perf_counter()
        orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, rows)
        dt += time.perf_counter() - t0
        reps += 1
    flops = 4.0 * case.B * case.H * len(rows) * case.L * case.d * reps
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(rows)} of {case.L} query rows per head, all keys, fp64, {reps} pass(es), {dt:.2f} s in all"}


def run_reference(args):
    """Reference arm: the fp64 CPU oracle on the host cores (rank 0 only), `--steps` steps of a bounded row sample."""
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    from oracle import attn_oracle as orc
    from paper_2609_10937_b200 import synth

    case = synth.CONFIGS[WORKLOAD]
    q, k, v = synth.make_qkv(case, seed=0)
    cores = orc.threads()
    # the sample of one step is sized from a probe so that warm-up plus all steps take about two minutes at most
    probe = np.unique(np.linspace(0, case.L - 1, 256).astype(np.int32))
    orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, probe)
    t0 = time.perf_counter()
    orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, probe)
    per_row = max(time.perf_counter() - t0, 1e-6) / len(probe)
    budget_s = 120.0
    n_rows = int(max(128, min(2048, budget_s / (per_row * (args.steps + args.warmup)))))
    rows = np.unique(np.linspace(0, case.L - 1, n_rows).astype(np.int32))
    flops = 4.0 * case.B * case.H * len(rows) * case.L * case.d
    for _ in range(args.warmup):
        orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, rows)
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, rows)
        times.append(time.perf_counter() - t0)
    ms = 1e3 * sum(times) / len(times)
    value = flops / (ms * 1e-3) / 1e12
    sample = (f"{len(rows)} of {case.L} query rows per head per step, all keys, fp64 (the oracle's time is linear in "
              f"the rows: TFLOP/s is per row processed)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": CONFIG,
        "arithmetic": "the oracle's: fp64 over the same bf16 inputs",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------------ GPU side
class Gpu:
    """Device buffers and timing helpers shared by the modes below."""

    def __init__(self, local):
        import torch

        from paper_2609_10937_b200 import binding

        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: the attention path has no CPU fallback")
        torch.cuda.set_device(local)
        self.torch, self.binding, self.local = torch, binding, local
        binding.lib()
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
        self.stream = torch.cuda.current_stream()
        self.desc = binding.hw_desc_query(local)

    def to_dev(self, bits):
        t = self.torch
        return t.from_numpy(bits.view(np.int16)).view(t.bfloat16).cuda()

    def timed(self, fn, steps, warmup, barrier=None):
        """Mean of per-step CUDA-event times on the launching stream; an L2 flush (a device write larger than L2)
        precedes every step outside its events.  Returns (mean ms, per-step list, wall t0, wall t1)."""
        torch = self.torch
        sync = barrier or torch.cuda.synchronize
        for _ in range(warmup):
            self.flush.fill_(1)
            fn()
        sync()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        t0 = time.time()
        for i in range(steps):
            self.flush.fill_(i & 0xFF)
            starts[i].record(self.stream)
            fn()
            ends[i].record(self.stream)
        sync()
        t1 = time.time()
        per = [s.elapsed_time(e) for s, e in zip(starts, ends)]
        return sum(per) / len(per), per, t0, t1

    def check_status(self):
        code, detail = self.binding.last_device_status()
        if code != 0:
            raise RuntimeError(f"device-side wait expired: {detail}")


def kernel_name(plan, d, cluster):
    """The instantiation a plan runs as: <d, tile_kv, n_q, causal, fixed merge roles, clusters>."""
    uniform = plan.ctas > plan.tiles and plan.ctas % plan.tiles == 0
    fixed = int((uniform and not plan.causal) or (plan.causal and cluster > 0))
    return f"attn_fwd_kernel<{d},{plan.tile_kv},{plan.n_q},{int(plan.causal)},{fixed},{int(cluster > 0)}>"


def measure_config(gpu, name, peaks, iters=None, oracle=True):
    """One benchmark configuration with the closed-form default tiles: time, TFLOP/s, error against the oracle."""
    from paper_2609_10937_b200 import synth

    torch, binding = gpu.torch, gpu.binding
    case = synth.CONFIGS[name]
    q, k, v = synth.make_qkv(case, seed=0)
    dq, dk, dv = (gpu.to_dev(x) for x in (q, k, v))
    do = torch.empty_like(dq)
    plan = binding.plan(gpu.desc, case.B, case.H, case.L, case.d)
    if iters is None:
        iters = 100 if case.flops < 1e9 else 30 if case.flops < 5e11 else 10
    ms_mean, per, _, _ = gpu.timed(lambda: binding.forward(dq, dk, dv, do), iters, 5)
    cluster = binding.last_cluster_size()
    gpu.check_status()
    # the median of the per-launch times: one launch delayed on the host side (the events bracket the launch call)
    # would otherwise carry into a mean over few launches
    ms = statistics.median(per)
    tf = case.flops / (ms * 1e-3) / 1e12
    out = {"shape": [case.B, case.H, case.L, case.d], "ms": ms, "ms_mean": ms_mean, "ms_min": min(per), "tflops": tf,
           "frac_of_measured_burst_peak": tf / peaks["bf16_tflops"], "launches_timed": iters,
           "tiles": {"tile_q": plan.tile_q, "tile_kv": plan.tile_kv, "kv_stages": plan.kv_stages, "q_tiles": plan.tiles,
                     "ctas": plan.ctas, "cluster": cluster, "cost_steps": plan.cost_steps},
           "kernel": kernel_name(plan, case.d, cluster)}
    if oracle:
        from oracle import attn_oracle as orc

        rows = synth.sample_rows(case.L)
        ref = orc.attention_rows(q, k, v, case.B, case.H, case.L, case.d, rows)
        bits = do.view(torch.int16).cpu().numpy().view(np.uint16).reshape(case.B * case.H, case.L, case.d)
        got = orc.bf16_bits_to_f64(np.ascontiguousarray(bits[:, rows]))
        diff = got - ref
        out["max_abs"] = float(np.abs(diff).max())
        out["rel_l2"] = float(np.linalg.norm(diff.ravel()) / np.linalg.norm(ref.ravel()))
        out["rows_checked_per_head"] = int(len(rows))
    del dq, dk, dv, do
    torch.cuda.empty_cache()
    return out


def sustained_leg(gpu, fn, flops, seconds, peaks, sampler, flush=True):
    """The step back to back for `seconds`: one pair of events around the lot plus events around every step."""
    torch = gpu.torch
    for _ in range(5):
        fn()
    torch.cuda.synchronize()
    probe, _, _, _ = gpu.timed(fn, 10, 0)
    per_iter_ms = probe + (L2_FLUSH_BYTES / 3.0e9 if flush else 0.0)     # the flush is a write of 256 MiB at ~3 TB/s
    steps = int(min(40000, max(50, seconds * 1e3 / per_iter_ms)))
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    lot0, lot1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.time()
    lot0.record(gpu.stream)
    for i in range(steps):
        if flush:
            gpu.flush.fill_(i & 0xFF)
        starts[i].record(gpu.stream)
        fn()
        ends[i].record(gpu.stream)
    lot1.record(gpu.stream)
    torch.cuda.synchronize()
    t1 = time.time()
    per = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    tail = per[len(per) // 2:]                                 # the second half: clocks have settled under load
    ms = sum(tail) / len(tail)
    value = flops / (ms * 1e-3) / 1e12
    clk = sampler.window(t0 + 0.2, t1) if sampler else {}
    out = {"ms_per_step": ms, "ms_per_step_first_tenth": sum(per[:max(1, len(per) // 10)]) / max(1, len(per) // 10),
           "value": value, "unit": UNIT, "steps": steps, "seconds": lot0.elapsed_time(lot1) / 1e3,
           "busy_fraction": sum(per) / lot0.elapsed_time(lot1),
           "frac_of_sustained_peak": value / peaks["bf16_tflops_sustained"],
           "frac_of_burst_peak": value / peaks["bf16_tflops"],
           "l2": "flushed between steps" if flush else "not flushed (inputs stay in L2)",
           "sm_mhz_median": clk.get("sm_mhz"), "sm_mhz_min": clk.get("sm_mhz_min"), "samples": clk.get("samples_inside_region"),
           "power_w_max": clk.get("power_w_max"), "reasons": clk.get("reasons"),
           "ms_x_mhz": ms * clk["sm_mhz"] if clk.get("sm_mhz") else None}
    return out


def run_ours(args):
    from paper_2609_10937_b200 import multirank, synth

    rank, world, local = dist_env()
    gpu = Gpu(local)
    torch, binding = gpu.torch, gpu.binding
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    case = synth.CONFIGS[WORKLOAD]
    q, k, v = synth.make_qkv(case, seed=multirank.rank_seed(0, rank))   # every rank its own problem of the same shape
    as_t = lambda b: torch.from_numpy(b.view(np.int16)).view(torch.bfloat16)
    hq, hk, hv = (as_t(x).pin_memory() for x in (q, k, v))
    ho = torch.empty_like(hq).pin_memory()
    dq, dk, dv = (x.cuda(non_blocking=True) for x in (hq, hk, hv))
    do = torch.empty_like(dq)
    scratch = torch.empty(4 * dq.numel() * 2, dtype=torch.uint8, device="cuda")
    plan = binding.plan(gpu.desc, case.B, case.H, case.L, case.d)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.15)
    step = lambda: binding.forward(dq, dk, dv, do)
    ms, per, t0, t1 = gpu.timed(step, args.steps, args.warmup, barrier)
    ms = multirank.max_over_ranks(ms, dist, "cuda")      # the slowest rank sets the step time
    launches_per_step = binding.last_launch_count()
    cluster = binding.last_cluster_size()
    clocks = sampler.window(t0, t1) if sampler else None
    gpu.check_status()
    e2e_steps = max(3, min(args.steps, 10))
    e2e_ms, _, _, _ = gpu.timed(lambda: binding.forward_host(hq, hk, hv, ho, scratch), e2e_steps, 3, barrier)
    e2e_ms = multirank.max_over_ranks(e2e_ms, dist, "cuda")

    flops = case.flops
    value = world * flops / (ms * 1e-3) / 1e12
    e2e_value = world * flops / (e2e_ms * 1e-3) / 1e12
    nbytes = dq.numel() * 2

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    peaks = load_peaks()
    achieved = flops / (ms * 1e-3) / 1e12
    capture = load_dram_capture()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": CONFIG,
        "tiles": {"tile_q": plan.tile_q, "tile_kv": plan.tile_kv, "kv_stages": plan.kv_stages, "q_tiles": plan.tiles,
                  "kv_splits": plan.kv_splits, "ctas": plan.ctas, "cluster": cluster, "cost_steps": plan.cost_steps,
                  "predicted_us_at_descriptor_peak": plan.predicted_us, "closed_form_default": True},
        "timing": {"l2": f"{L2_FLUSH_BYTES >> 20} MiB device write between timed steps (outside the step's events)",
                   "how": "CUDA events on the launching stream around every step; mean of per-step times; max over ranks",
                   "ms_per_step_min": min(per), "ms_per_step_max": max(per),
                   "note": "a burst number: the timed region is milliseconds long, compare with the burst peak"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 3 * nbytes, "d2h_bytes_per_step": nbytes,
                "ms_per_step": e2e_ms, "steps": e2e_steps,
                "path": "attn_forward_host: pinned host q,k,v -> device, forward (two blocks of query rows, copies overlapped with the kernels), o -> pinned host, all in the timed region"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {
            "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": UNIT,
            "frac": achieved / peaks["bf16_tflops"],
            "traffic": capture["bytes_per_launch"] if capture else None,
            "traffic_source": ({k_: capture.get(k_) for k_ in ("capture", "commit", "kernel")} if capture else None),
            "peak_source": f"{peaks['source']} cuBLAS bf16 burst (kernel timed alone)",
            "frac_of_nominal_2250": achieved / 2250.0,
            "kernel": kernel_name(plan, case.d, cluster) + " (one launch per step; split-key partials are merged in the same kernel)",
            "algorithmic_flops_per_launch": flops,
            "unfused_traffic_bytes_bf16_scores": unfused_bytes(case.B, case.H, case.L, case.d, 2, 2),
            "compulsory_traffic_bytes": fused_bytes(case.B, case.H, case.L, case.d, 2),
        },
    }
    if world == 1 and not args.no_sustained:
        # What the same step does once the power limit bites: seconds of back-to-back steps, clocks sampled throughout.
        line["sustained"] = sustained_leg(gpu, step, flops, args.sustained_seconds, peaks, sampler, flush=True)
        line["sustained_no_flush"] = sustained_leg(gpu, step, flops, min(1.0, args.sustained_seconds), peaks, sampler,
                                                   flush=False)
    if sampler:
        sampler.stop()
    if world == 1 and not args.no_extras:
        # Context beside the headline (not part of the timed region above): the same problem through the
        # unfused three-kernel path, and the paper's other workload, the 4096^3 matrix product.
        scores = torch.empty(case.B * case.H * case.L * case.L, dtype=torch.bfloat16, device="cuda")
        u_ms, _, _, _ = gpu.timed(lambda: binding.forward_unfused(dq, dk, dv, scores, do), 10, 3)
        del scores
        line["unfused_baseline"] = {
            "ms_per_step": u_ms, "value": flops / (u_ms * 1e-3) / 1e12, "unit": UNIT, "kernels_per_step": 3,
            "fused_speedup": u_ms / ms,
            "path": "attn_forward_unfused: S = Q K^T to HBM (bf16), row softmax in place, P V; same inputs",
            "analytic_traffic_bytes": unfused_bytes(case.B, case.H, case.L, case.d, 2, 2)}
        ga = torch.randn(4096, 4096, device="cuda").to(torch.bfloat16)
        gb = torch.randn(4096, 4096, device="cuda").to(torch.bfloat16)
        gc = torch.empty(4096, 4096, dtype=torch.bfloat16, device="cuda")
        g_ms, _, _, _ = gpu.timed(lambda: binding.gemm(ga, gb, gc), 20, 3)
        g_tf = 2.0 * 4096 ** 3 / (g_ms * 1e-3) / 1e12
        line["gemm"] = {"workload": "C = A B, 4096 x 4096 x 4096, bf16 in/out, fp32 accumulate, closed-form tiles",
                        "ms_per_step": g_ms, "value": g_tf, "unit": UNIT, "frac_of_measured_peak": g_tf / peaks["bf16_tflops"]}
        del ga, gb, gc
    if world == 1 and not args.no_configs:
        del scratch
        torch.cuda.empty_cache()
        names = [n for n in synth.CONFIGS if n != WORKLOAD]
        line["configs"] = {n: measure_config(gpu, n, peaks) for n in names}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(case, q, k, v)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------------------------------------ other modes
def run_case(args):
    """One named configuration, timed alone (few launches: the command profiler captures are taken on).  `gemmN` is
    the N x N x N matrix product, `gemmMxNxK` any other.  Beside it the library product on the same inputs."""
    gpu = Gpu(0)
    if args.case.startswith("gemm"):
        dims = [int(x) for x in args.case[4:].split("x")]
        m, n, k = dims if len(dims) == 3 else (dims[0],) * 3
        torch, binding = gpu.torch, gpu.binding
        a = torch.randn(m, k, device="cuda").to(torch.bfloat16)
        b = torch.randn(k, n, device="cuda").to(torch.bfloat16)
        c = torch.empty(m, n, dtype=torch.bfloat16, device="cuda")
        ms, _, _, _ = gpu.timed(lambda: binding.gemm(a, b, c), args.steps, 3)
        ms_lib, _, _, _ = gpu.timed(lambda: torch.matmul(a, b, out=c), args.steps, 3)
        print(json.dumps({"case": args.case, "ms": ms, "tflops": 2.0 * m * n * k / ms / 1e9,
                          "c_write_gbs": 2.0 * m * n / ms / 1e6, "torch_matmul_ms": ms_lib,
                          "tiles": binding.gemm_plan(gpu.desc, 1, m, n, k).as_dict()}), flush=True)
        return 0
    out = measure_config(gpu, args.case, load_peaks(), iters=args.steps, oracle=False)
    print(json.dumps({"case": args.case, **out}), flush=True)
    return 0


def run_tile_sweep(args):
    """Every compiled tile variant (n_q in {1, 2}, tile_kv in {64, 128}, ring depth default and default - 1, grid sizes
    around the planner's choice) against the closed-form default: the default's time, the best point, default / best."""
    from paper_2609_10937_b200 import synth

    gpu = Gpu(0)
    torch, binding, desc = gpu.torch, gpu.binding, gpu.desc
    case = synth.CONFIGS[args.tile_sweep]
    q, k, v = (gpu.to_dev(x) for x in synth.make_qkv(case, 0))
    o = torch.empty_like(q)
    plan = binding.plan(desc, case.B, case.H, case.L, case.d)
    iters = args.steps
    t = lambda fn: gpu.timed(fn, iters, 3)[0]
    t(lambda: binding.forward(q, k, v, o))          # settle clocks; the default is timed after the sweep points
    points = []
    for n_q in (2, 1):
        for tile_kv in (128, 64):
            tiles = case.B * case.H * -(-case.L // (128 * n_q))
            steps = case.L // tile_kv
            grids = sorted({tiles, min(tiles * max(1, desc.num_units // tiles), tiles * steps),
                            min(max(desc.num_units, tiles), tiles * steps)})
            for stages_delta in (0, 1):
                for ctas in grids:
                    q_bytes, stage = n_q * 128 * case.d * 2, tile_kv * case.d * 2
                    max_stages = min(8, (desc.local_mem_bytes - q_bytes - n_q * 128 * 128 - 3072) // stage)
                    stages = max_stages - stages_delta
                    if stages < 2:
                        continue
                    kw = dict(n_q=n_q, tile_kv=tile_kv, kv_stages=stages, ctas=ctas)
                    try:
                        ms = t(lambda: binding.forward_tiles(q, k, v, o, **kw))
                    except binding.AttnError:
                        continue
                    points.append(dict(kw, ms=ms, tflops=case.flops / ms / 1e9))
    default_ms = t(lambda: binding.forward(q, k, v, o))
    best = min(points, key=lambda p: p["ms"])
    print(json.dumps({
        "workload": args.tile_sweep,
        "default": {"tile_q": plan.tile_q, "tile_kv": plan.tile_kv, "kv_stages": plan.kv_stages, "ctas": plan.ctas,
                    "ms": default_ms, "tflops": case.flops / default_ms / 1e9},
        "best": best, "default_over_best_time": default_ms / best["ms"],
        "points": sorted(points, key=lambda p: p["ms"])}), flush=True)
    return 0


def run_grid_sweep(args):
    """For shapes with fewer Q tiles than SMs: the time of every grid the occupancy step chooses among -- k = 1..8
    CTAs per Q tile (as one thread-block cluster where the launcher can, else through the workspace) and equal ranges
    of the (tile, step) line over min(SMs, units / 4) CTAs -- and the grid the closed form picks.  One text row per
    (shape, grid): B H L d ctas k cluster us picked."""
    from paper_2609_10937_b200 import synth

    gpu = Gpu(0)
    torch, binding, desc = gpu.torch, gpu.binding, gpu.desc
    print("# B H L d q_tiles steps ctas k cluster_size mean_us picked_by_closed_form")
    for (B, H, L, d) in GRID_SWEEP_SHAPES:
        case = synth.AttnCase("grid", B, H, L, d, cfg_id=70)
        q, k, v = (gpu.to_dev(x) for x in synth.make_qkv(case, 0))
        o = torch.empty_like(q)
        plan = binding.plan(desc, B, H, L, d)
        tiles, steps = plan.tiles, -(-L // plan.tile_kv)
        grids = {}
        for kk in range(1, 9):
            if tiles * kk <= desc.num_units and steps // kk >= 1:
                grids[tiles * kk] = kk
        g = min(desc.num_units, tiles * steps // 4)
        if g > tiles and g not in grids:
            grids[g] = 0
        if plan.ctas not in grids:
            grids[plan.ctas] = 0
        gpu.timed(lambda: binding.forward(q, k, v, o), 5, 3)
        for ctas in sorted(grids):
            fn = lambda: binding.forward_tiles(q, k, v, o, ctas=ctas)
            try:
                ms, _, _, _ = gpu.timed(fn, args.steps, 3)
            except binding.AttnError:
                continue
            print(f"{B} {H} {L} {d} {tiles} {steps} {ctas} {grids[ctas]} {binding.last_cluster_size()} {ms * 1e3:.2f} "
                  f"{int(ctas == plan.ctas)}", flush=True)
        gpu.check_status()
    return 0


def run_unfused_sweep(args):
    """Fused attention against the unfused three-kernel path over L (one head, d = 128), the three kernels also timed
    separately, and the matrix product alone: one JSON object per line."""
    gpu = Gpu(0)
    torch, binding = gpu.torch, gpu.binding
    t = lambda fn: gpu.timed(fn, args.steps, 3)[0]
    gen = torch.Generator(device="cuda").manual_seed(0)
    rnd = lambda *shape: torch.randn(*shape, device="cuda", generator=gen).to(torch.bfloat16)
    d = 128
    for L in (4096, 8192, 16384, 32768):
        q, k, v = rnd(1, 1, L, d), rnd(1, 1, L, d), rnd(1, 1, L, d)
        o = torch.empty_like(q)
        s = torch.empty(L, L, dtype=torch.bfloat16, device="cuda")
        t_f = t(lambda: binding.forward(q, k, v, o))
        t_u = t(lambda: binding.forward_unfused(q, k, v, s, o))
        t_qk = t(lambda: binding.gemm(q[0, 0], k[0, 0], s, b_layout="nk"))
        t_sm = t(lambda: binding.softmax_rows(s, d ** -0.5, out=s))
        t_pv = t(lambda: binding.gemm(s, v[0, 0], o[0, 0], b_layout="kn"))
        flops = 4.0 * L * L * d
        print(json.dumps({
            "workload": f"attention B=1 H=1 L={L} d={d}", "fused_ms": t_f, "fused_tflops": flops / t_f / 1e9,
            "unfused_ms": t_u, "unfused_tflops": flops / t_u / 1e9, "fused_speedup": t_u / t_f,
            "unfused_kernels_ms": {"qk": t_qk, "softmax": t_sm, "pv": t_pv},
            "softmax_gbs": 2.0 * L * L * 2 / t_sm / 1e6,
            "unfused_analytic_traffic_bytes": unfused_bytes(1, 1, L, d, 2, 2),
            "fused_compulsory_traffic_bytes": fused_bytes(1, 1, L, d, 2)}), flush=True)
        del s
    for n in (4096, 8192):
        a, b = rnd(n, n), rnd(n, n)
        c = torch.empty(n, n, dtype=torch.bfloat16, device="cuda")
        ms = t(lambda: binding.gemm(a, b, c))
        ms_lib = t(lambda: torch.matmul(a, b, out=c))
        print(json.dumps({"workload": f"gemm {n}x{n}x{n} bf16", "ms": ms, "tflops": 2.0 * n ** 3 / ms / 1e9,
                          "torch_matmul_ms": ms_lib, "torch_matmul_tflops": 2.0 * n ** 3 / ms_lib / 1e9,
                          "tiles": binding.gemm_plan(gpu.desc, 1, n, n, n).as_dict()}), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--sustained-seconds", type=float, default=2.5)
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--no-extras", action="store_true", help="skip the unfused-path and matrix-product context numbers")
    ap.add_argument("--no-configs", action="store_true", help="skip the other benchmark configurations")
    ap.add_argument("--no-sustained", action="store_true", help="skip the seconds-long back-to-back leg")
    ap.add_argument("--case", default=None, help="time one named configuration only (cfg1, cfg2, cfg4_L1024, ..., cfg5b, gemm4096, gemm16384x16384x128)")
    ap.add_argument("--tile-sweep", default=None, metavar="NAME", help="tile sweep around the closed-form default")
    ap.add_argument("--grid-sweep", action="store_true", help="grid-size sweep over short and medium shapes")
    ap.add_argument("--unfused-sweep", action="store_true", help="fused against unfused over L; matrix product alone")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.case or args.tile_sweep or args.grid_sweep or args.unfused_sweep:
        args.steps = args.steps or (3 if args.case else 20 if args.grid_sweep else 10)
        if args.case:
            return run_case(args)
        if args.tile_sweep:
            return run_tile_sweep(args)
        if args.grid_sweep:
            return run_grid_sweep(args)
        return run_unfused_sweep(args)
    if args.impl == "reference":
        args.steps = args.steps or 10
        return run_reference(args)
    args.steps = args.steps or 100
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
