"""HBM-traffic accounting for fused attention (the paper's Section "Results",
paragraph "HBM traffic", and its savings equation L/(4d)).

fused_bytes:   Q, K, V read once and the result written once.
unfused_bytes: three separate passes with the L x L matrix materialised between
               them -- scores written and read, probabilities written and read --
               plus Q, K, V and the result once.  With 4-byte elements and scores
               this reproduces the paper's 34 MB / 4,329 MB / 129x at L = 16384.
"""
from __future__ import annotations

# DRAM bytes (read + write) of one launch of the dominant kernel, from an ncu
# capture of the benchmark workload (dram__bytes_read.sum + dram__bytes_write.sum);
# None until a capture has been taken.  The capture summaries live in profiles/.
MEASURED_DRAM_BYTES_PER_LAUNCH = {
    "cfg3": 12_799_488 + 34_048,    # 12.80 MB read + 0.03 MB written, mean of two launches (the output was still in L2 when the kernel ended)
}


def fused_bytes(B: int, H: int, L: int, d: int, elem_bytes: int) -> int:
    return B * H * 4 * L * d * elem_bytes


def unfused_bytes(B: int, H: int, L: int, d: int, elem_bytes: int, score_bytes: int) -> int:
    return B * H * (4 * L * L * score_bytes + 4 * L * d * elem_bytes)


def savings(L: int, d: int) -> float:
    return L / (4.0 * d)


def measured_dram_bytes_per_launch(_root=None, workload: str = "cfg3"):
    return MEASURED_DRAM_BYTES_PER_LAUNCH.get(workload)
