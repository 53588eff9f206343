"""Helpers for the GPU parity tests: bf16 bit patterns <-> torch tensors, error measures."""
import numpy as np

MAX_ABS_TOL = 1e-2      # stated tolerance of the build target on bf16 outputs
REL_L2_TOL = 5e-3


def to_cuda_bf16(bits: np.ndarray):
    import torch

    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.cuda()


def to_host_f64(t) -> np.ndarray:
    """bf16 CUDA tensor -> fp64 numpy (exact widening)."""
    import torch

    bits = t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def errors(got: np.ndarray, ref: np.ndarray):
    diff = got - ref
    max_abs = float(np.abs(diff).max())
    rel_l2 = float(np.linalg.norm(diff.ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300))
    return max_abs, rel_l2


def assert_close(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """max-abs <= 1e-2 and relative L2 <= 5e-3; an element whose reference magnitude is
    >= 4 is judged by one bf16 ulp of the reference instead (half an ulp there already
    exceeds 1e-2)."""
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    diff = np.abs(got - ref)
    big = np.abs(ref) >= 4.0
    if big.any():
        ulp = 2.0 ** (np.floor(np.log2(np.abs(ref[big]))) - 7)
        assert (diff[big] <= np.maximum(MAX_ABS_TOL, ulp)).all(), f"{what}: large-magnitude element off by > 1 ulp"
    max_abs = float(diff[~big].max()) if (~big).any() else 0.0
    rel_l2 = errors(got, ref)[1]
    assert max_abs <= MAX_ABS_TOL, f"{what}: max_abs {max_abs:.3e} > {MAX_ABS_TOL}"
    assert rel_l2 <= REL_L2_TOL, f"{what}: rel_l2 {rel_l2:.3e} > {REL_L2_TOL}"
    return max_abs, rel_l2
