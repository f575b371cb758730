"""Seeded synthetic inputs for the block-quantised matmul library.

This module only *makes inputs*: random weights, activations and router
logits with the shapes and value distributions of the benchmark workloads, and
the offline step that turns fp32 weights into canonical quantised blocks
(scales + codes are an input of the library; the library never quantises).
It holds none of the dequantise-and-multiply arithmetic and imports neither
the CUDA binding nor the CPU oracle, so both sides can be fed from it.

Recipe: tensor ``i`` of workload ``c`` is drawn from
``numpy.random.default_rng([seed_c, i])``; weights are
``standard_normal(float32) * 0.02`` (standard deviation 0.02), activations and
router logits ``standard_normal(float32)`` (activations then rounded to fp16).

Canonical block format (32 elements along K):
  Q4: uint16 fp16 scale, then 16 bytes; element i has code q_i in [-8,7] stored
      as u_i = q_i + 8, byte j = u_{2j} | (u_{2j+1} << 4).            (18 bytes)
  Q8: uint16 fp16 scale, then 32 int8 codes in [-127,127].          (34 bytes)
  Q5: uint16 fp16 scale, 4 bytes of fifth bits (bit i of the little-endian word:
      element i), 16 bytes of low nibbles as in Q4; u_i = q_i + 16, q in [-16,15]. (22 bytes)
  Q6: uint16 fp16 scale, 8 bytes of high bit pairs (bits 2(i%4), 2(i%4)+1 of byte
      i/4: element i), 16 bytes of low nibbles; u_i = q_i + 32, q in [-32,31].     (26 bytes)
Row n of W[N,K] holds K/32 consecutive blocks; rows are consecutive.
"""
from __future__ import annotations

import numpy as np

Q4 = 4
Q5 = 5
Q6 = 6
Q8 = 8
BLOCK = 32
BLOCK_BYTES = {Q4: 18, Q5: 22, Q6: 26, Q8: 34}
QRANGE = {Q4: (-8, 7), Q5: (-16, 15), Q6: (-32, 31), Q8: (-127, 127)}     # what the quantiser emits (Q8 decodes -128 too)


def canonical_bytes(fmt: int, N: int, K: int) -> int:
    assert K % BLOCK == 0
    return N * (K // BLOCK) * BLOCK_BYTES[fmt]


def rng(seed: int, tensor: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tensor)])


def weights(seed: int, tensor: int, N: int, K: int, std: float = 0.02) -> np.ndarray:
    """fp32 W[N,K] ~ N(0, std^2)."""
    w = rng(seed, tensor).standard_normal((N, K), dtype=np.float32)
    w *= np.float32(std)
    return w


def activations(seed: int, tensor: int, *shape: int) -> np.ndarray:
    """fp16 activations ~ N(0,1)."""
    return rng(seed, tensor).standard_normal(shape, dtype=np.float32).astype(np.float16)


def logits(seed: int, tensor: int, T: int, E: int) -> np.ndarray:
    """fp32 router logits ~ N(0,1)."""
    return rng(seed, tensor).standard_normal((T, E), dtype=np.float32)


def quantize(fmt: int, w: np.ndarray, chunk_rows: int = 4096) -> np.ndarray:
    """fp32 W[N,K] -> canonical blocks as a flat uint8 array.

    Per block in fp32: scale = fp16(max|w| / QMAX) with QMAX 7 (Q4) or 127
    (Q8); codes = clip(round_half_even(w / float(scale))); a zero scale gives
    all-zero codes.
    """
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    assert K % BLOCK == 0
    nb = K // BLOCK
    bb = BLOCK_BYTES[fmt]
    qmin, qmax = (np.float32(v) for v in QRANGE[fmt])
    out = np.empty((N * nb, bb), dtype=np.uint8)
    for r0 in range(0, N, chunk_rows):
        r1 = min(N, r0 + chunk_rows)
        wb = w[r0:r1].reshape(-1, BLOCK)
        amax = np.abs(wb).max(axis=1)
        d = (amax / qmax).astype(np.float16)
        df = d.astype(np.float32)
        zero = df == 0
        div = np.where(zero, np.float32(1), df)
        q = np.rint(wb / div[:, None])
        np.clip(q, qmin, qmax, out=q)
        q[zero] = 0
        qi = q.astype(np.int8)
        o = out[r0 * nb:r1 * nb]
        o[:, 0:2] = d.view(np.uint16).astype("<u2").view(np.uint8).reshape(-1, 2)
        _store_codes(fmt, o, qi)
    return out.reshape(-1)


def _store_codes(fmt: int, o: np.ndarray, q: np.ndarray) -> None:
    """Write integer codes q [blocks, 32] into the code bytes of canonical blocks o [blocks, block bytes]."""
    if fmt == Q8:
        o[:, 2:] = q.astype(np.int8).view(np.uint8)
        return
    u = (q.astype(np.int16) - QRANGE[fmt][0]).astype(np.uint8)               # offset binary
    lo = u & 15
    nib = lo[:, 0::2] | (lo[:, 1::2] << 4)
    if fmt == Q4:
        o[:, 2:] = nib
    elif fmt == Q5:
        bit = (u >> 4).astype(np.uint32)
        word = (bit << np.arange(32, dtype=np.uint32)[None, :]).sum(axis=1, dtype=np.uint32)
        o[:, 2:6] = word.astype("<u4").view(np.uint8).reshape(-1, 4)
        o[:, 6:] = nib
    else:
        two = (u >> 4).reshape(-1, 8, 4)
        o[:, 2:10] = (two[:, :, 0] | (two[:, :, 1] << 2) | (two[:, :, 2] << 4) | (two[:, :, 3] << 6)).astype(np.uint8)
        o[:, 10:] = nib


def blocks_from_codes(fmt: int, scales_bits: np.ndarray, codes: np.ndarray) -> np.ndarray:
    """Assemble canonical blocks from explicit fp16 scale bit patterns
    (uint16 [N, K/32]) and integer codes (int [N, K])."""
    scales_bits = np.ascontiguousarray(scales_bits, dtype=np.uint16)
    N, nb = scales_bits.shape
    codes = np.asarray(codes).reshape(N * nb, BLOCK)
    out = np.empty((N * nb, BLOCK_BYTES[fmt]), dtype=np.uint8)
    out[:, 0:2] = scales_bits.reshape(-1).astype("<u2").view(np.uint8).reshape(-1, 2)
    lo, hi = (-128, 127) if fmt == Q8 else QRANGE[fmt]
    assert codes.min() >= lo and codes.max() <= hi
    _store_codes(fmt, out, codes)
    return out.reshape(-1)


# --------------------------------------------------------------------------
# Workloads.  Shapes follow the layer shapes of 0.6B-30B class transformer
# checkpoints; the values are synthetic.
# --------------------------------------------------------------------------

CFG0 = dict(seed=0, fmt=Q4, N=3072, K=1024)

# (name, N, K, activation vector it reads)
CFG1_LAYER = (
    ("q", 2048, 2048, "x_attn"),
    ("k", 512, 2048, "x_attn"),
    ("v", 512, 2048, "x_attn"),
    ("o", 2048, 2048, "x_o"),
    ("gate", 8192, 2048, "x_ffn"),
    ("up", 8192, 2048, "x_ffn"),
    ("down", 2048, 8192, "x_down"),
)
CFG1 = dict(seed=1, layers=16, fmts=(Q4, Q8))
CFG1_ACTS = (("x_attn", 2048), ("x_o", 2048), ("x_ffn", 2048), ("x_down", 8192))

CFG2 = dict(seed=2, fmt=Q8, N=128256, K=3072)

CFG3 = dict(seed=3, fmt=Q4, Ms=(128, 256, 512, 1024, 2048),
            shapes=(("gate_up", 8192, 3072), ("down", 3072, 8192)))

CFG4 = dict(seed=4, fmt=Q4, H=2048, I=768, E=128, topk=8, Ts=(1, 128, 512, 2048))


def cfg1_weight_id(layer: int, mat: int) -> int:
    return layer * 16 + mat


def cfg1_act_id(layer: int, act: int) -> int:
    return 1000 + layer * 4 + act


def cfg1_layer_weights(layer: int):
    """Yield (name, N, K, act_name, fp32 weights) for one layer of the decode stack."""
    for mi, (name, N, K, act) in enumerate(CFG1_LAYER):
        yield name, N, K, act, weights(CFG1["seed"], cfg1_weight_id(layer, mi), N, K)


def cfg1_layer_acts(layer: int):
    return {name: activations(CFG1["seed"], cfg1_act_id(layer, ai), K)
            for ai, (name, K) in enumerate(CFG1_ACTS)}


def moe_expert_weights(seed: int, fmt: int, E: int, H: int, I: int):
    """Canonical blocks for E experts: (gate [E*I,H], up [E*I,H], down [E*H,I]).

    Expert e's matrix is rows [e*I,(e+1)*I) of gate/up and [e*H,(e+1)*H) of
    down, so each expert's blocks follow the previous expert's.
    """
    gate = quantize(fmt, weights(seed, 10, E * I, H))
    up = quantize(fmt, weights(seed, 11, E * I, H))
    down = quantize(fmt, weights(seed, 12, E * H, I))
    return gate, up, down
