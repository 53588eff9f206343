"""Fused attention against the unfused three-kernel path, and the matrix product alone.

  python -m paper_2609_10937_b200.unfused_bench [--L 4096,8192,16384] [--d 128] [--gemm 4096] [--iters 10]

Prints one JSON object per line: for every L the time of attn_forward and of attn_forward_unfused
(S = Q K^T materialised in HBM, row softmax in place, P V) with its three kernels timed separately, and
for every --gemm size n the n x n x n matrix product.  Times are means of CUDA-event times with a
256 MiB device write between launches (cold L2).  The paper's sequence-length sweep (its Table 3) has
this shape; its numbers are for other hardware.
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def main(argv=None) -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--L", default="4096,8192,16384")
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--gemm", default="4096")
    ap.add_argument("--iters", type=int, default=10)
    args = ap.parse_args(argv)

    import torch

    from . import binding, traffic

    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device: there is no CPU path")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(args.iters):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return float(np.mean(ts))

    gen = torch.Generator(device="cuda").manual_seed(0)
    rnd = lambda *shape: torch.randn(*shape, device="cuda", generator=gen).to(torch.bfloat16)
    d = args.d
    for L in [int(x) for x in args.L.split(",") if x]:
        q, k, v = rnd(1, 1, L, d), rnd(1, 1, L, d), rnd(1, 1, L, d)
        o = torch.empty_like(q)
        s = torch.empty(L, L, dtype=torch.bfloat16, device="cuda")
        t_f = timed(lambda: binding.forward(q, k, v, o))
        t_u = timed(lambda: binding.forward_unfused(q, k, v, s, o))
        t_qk = timed(lambda: binding.gemm(q[0, 0], k[0, 0], s, b_layout="nk"))
        t_sm = timed(lambda: binding.softmax_rows(s, d ** -0.5, out=s))
        t_pv = timed(lambda: binding.gemm(s, v[0, 0], o[0, 0], b_layout="kn"))
        flops = 4.0 * L * L * d
        print(json.dumps({
            "workload": f"attention B=1 H=1 L={L} d={d}", "fused_ms": t_f, "fused_tflops": flops / t_f / 1e9,
            "unfused_ms": t_u, "unfused_tflops": flops / t_u / 1e9, "fused_speedup": t_u / t_f,
            "unfused_kernels_ms": {"qk": t_qk, "softmax": t_sm, "pv": t_pv},
            "softmax_gbs": 2.0 * L * L * 2 / t_sm / 1e6,
            "unfused_analytic_traffic_bytes": traffic.unfused_bytes(1, 1, L, d, 2, 2),
            "fused_compulsory_traffic_bytes": traffic.fused_bytes(1, 1, L, d, 2)}), flush=True)
        del s
    for n in [int(x) for x in args.gemm.split(",") if x]:
        a, b = rnd(n, n), rnd(n, n)
        c = torch.empty(n, n, dtype=torch.bfloat16, device="cuda")
        t = timed(lambda: binding.gemm(a, b, c))
        print(json.dumps({"workload": f"gemm {n}x{n}x{n} bf16", "ms": t, "tflops": 2.0 * n ** 3 / t / 1e9,
                          "tiles": binding.gemm_plan(binding.hw_desc_query(0), 1, n, n, n).as_dict()}), flush=True)
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
