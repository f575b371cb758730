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


def random_blocks(synth, fmt, N, K, seed, special_scales=True, scale_bits=(0x1400, 0x3400)):
    """Random codes over the full code range and random fp16 scales as canonical blocks;
    returns (blocks, codes, scale_bits).  Scales are drawn from the bit-pattern range
    `scale_bits` (default ~ 2^-10 .. 0.25).  special_scales: True replaces one block in 16 by a
    negative, zero, subnormal or -0 scale; "no_subnormal" leaves the subnormal kind out."""
    rng = np.random.default_rng(seed)
    lo, hi = {4: (-8, 8), 5: (-16, 16), 6: (-32, 32), 8: (-128, 128)}[fmt]
    codes = rng.integers(lo, hi, size=(N, K))
    sb = rng.integers(scale_bits[0], scale_bits[1], size=(N, K // 32)).astype(np.uint16)
    if special_scales:
        flat = sb.reshape(-1)
        pick = rng.permutation(flat.size)[: max(8, flat.size // 16)]
        kinds = rng.integers(0, 4, size=pick.size)
        flat[pick[kinds == 0]] |= 0x8000                                        # negative
        flat[pick[kinds == 1]] = 0                                              # zero
        if special_scales != "no_subnormal":
            flat[pick[kinds == 2]] = rng.integers(1, 0x400, size=(kinds == 2).sum())  # subnormal
        flat[pick[kinds == 3]] = 0x8000                                         # -0
    return synth.blocks_from_codes(fmt, sb, codes), codes, sb


def subnormal_weight_term(W: np.ndarray, X: np.ndarray) -> np.ndarray:
    """The extra term of the tensor-core products' documented bound: a weight with
    0 < |d q| < 2^-14 enters the contraction as a subnormal fp16 with an absolute error of up
    to 2^-25, so output [m, n] may be off by another 2^-25 * sum of |X[m, k]| over such k.
    W: dequantised weights [N, K]; X: activations [M, K].  Returns [M, N]."""
    tiny = ((np.abs(W) > 0) & (np.abs(W) < 2.0**-14)).astype(np.float64)
    return 2.0**-25 * (np.abs(X.astype(np.float64)) @ tiny.T)


def moe_composed_bound(oracle, fmt, logits, X, gate, up, down, H, I, E, topk, tokens):
    """Error bound of a whole mixture-of-experts layer output against the all-fp64 layer, composed
    from the per-product tolerance tol(B) = 2e-3 * B + 1e-5 of each stage (B = sum |w x|).

    For token t and slot j (expert e, weight p_j), with G, U, B_G, B_U the exact gate / up products:
      h = silu(G) * U;  E_h = 1.1 tol(B_G) |U| + |silu(G)| tol(B_U) + 1.1 tol(B_G) tol(B_U) + 2^-11 |h|
                               (|silu'| <= 1.1; the last term is the fp16 rounding of the stored h)
      D_j = Wdown h;    E_D = 2e-3 * sum_i |Wdown[c,i] h_i| + 1.002 * sum_i |Wdown[c,i]| E_h,i + 1e-5
                               (the down product's own tolerance on the rounded h, plus the propagated E_h)
      out = sum_j p_j D_j;  bound = sum_j p_j E_D,j                        (propagated)
                                  + 2e-3 * sum_j p_j (|D_j| + E_D,j) + 1e-5   (the combine's own tolerance)
                                  + 1e-6 * sum_j (|D_j| + E_D,j)            (routing weights within 1e-6)
    Returns (out_ref, bound), each [len(tokens), H]; out_ref agrees with oracle.moe_tokens."""
    gu_bytes, dn_bytes = len(gate) // E, len(down) // E
    idx, p = oracle.route(logits, topk)
    tol = lambda B: RTOL_SUMABS * B + ATOL
    out_ref = np.zeros((len(tokens), H))
    bound = np.zeros((len(tokens), H))
    for n, t in enumerate(tokens):
        prop = np.zeros(H)
        mag = np.zeros(H)
        for j in range(topk):
            e = int(idx[t, j])
            G, BG = oracle.gemm(fmt, gate[e * gu_bytes:(e + 1) * gu_bytes], I, H, X[t:t + 1])
            U, BU = oracle.gemm(fmt, up[e * gu_bytes:(e + 1) * gu_bytes], I, H, X[t:t + 1])
            sG = oracle.silu(G)
            h = sG * U
            E_h = 1.1 * tol(BG) * np.abs(U) + np.abs(sG) * tol(BU) + 1.1 * tol(BG) * tol(BU) + 2.0**-11 * np.abs(h)
            wd = down[e * dn_bytes:(e + 1) * dn_bytes]
            D, B_dh = oracle.gemm_f64(fmt, wd, H, I, h)
            _, B_dE = oracle.gemm_f64(fmt, wd, H, I, E_h)
            E_D = RTOL_SUMABS * B_dh[0] + 1.002 * B_dE[0] + ATOL
            out_ref[n] += p[t, j] * D[0]
            prop += p[t, j] * E_D
            mag += np.abs(D[0]) + E_D
            bound[n] += RTOL_SUMABS * p[t, j] * (np.abs(D[0]) + E_D)
        bound[n] += prop + ATOL + 1e-6 * mag
    return out_ref, bound
