"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

RTOL_SUMABS = 2e-3      # |y_gpu - y_ref| <= RTOL_SUMABS * sum_k |w x| + ATOL   (per output element)
ATOL = 1e-5


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host_f64(t: torch.Tensor) -> np.ndarray:
    """fp16/fp32 CUDA tensor -> float64 numpy (exact widening)."""
    return t.detach().cpu().numpy().astype(np.float64)


def assert_within_tol(y_gpu: np.ndarray, y_ref: np.ndarray, B: np.ndarray, what: str = ""):
    tol = RTOL_SUMABS * B + ATOL
    err = np.abs(y_gpu - y_ref)
    worst = float(np.max(err / tol)) if err.size else 0.0
    assert np.all(np.isfinite(y_gpu)), what
    assert worst <= 1.0, "%s: max |err|/tol = %.3f" % (what, worst)
    return worst


def random_blocks(synth, fmt, N, K, seed, special_scales=True):
    """Random codes over the full code range and random fp16 scales (some negative,
    zero and subnormal) as canonical blocks; returns (blocks, codes, scale_bits)."""
    rng = np.random.default_rng(seed)
    lo, hi = (-8, 8) if fmt == 4 else (-128, 128)
    codes = rng.integers(lo, hi, size=(N, K))
    sb = rng.integers(0x1400, 0x3400, size=(N, K // 32)).astype(np.uint16)     # ~ 2^-10 .. 0.25
    if special_scales:
        flat = sb.reshape(-1)
        pick = rng.permutation(flat.size)[: max(8, flat.size // 16)]
        kinds = rng.integers(0, 4, size=pick.size)
        flat[pick[kinds == 0]] |= 0x8000                                        # negative
        flat[pick[kinds == 1]] = 0                                              # zero
        flat[pick[kinds == 2]] = rng.integers(1, 0x400, size=(kinds == 2).sum())  # subnormal
        flat[pick[kinds == 3]] = 0x8000                                         # -0
    return synth.blocks_from_codes(fmt, sb, codes), codes, sb
