"""Pins for the CPU oracle (no GPU).

Each test fixes the oracle to something other than itself: hand-derived values
(tests/golden/handbuilt.json), library fp16, integer matrix products, triple
loops in plain Python, an independent numpy decoder, or an invariant of the
mathematics.  A dropped term, a wrong sign or index, swapped nibbles or a
transposed operand fails at least one of them.
"""
import json
import math
import os

import numpy as np
import pytest

from paper_2607_00501_b200 import synth
from tests import npref

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "handbuilt.json")))
Q4, Q5, Q6, Q8 = 4, 5, 6, 8
FMTS = [Q4, Q5, Q6, Q8]
QLO = {Q4: -8, Q5: -16, Q6: -32, Q8: -128}      # lowest code a block can hold
QMAX = {Q4: 7, Q5: 15, Q6: 31, Q8: 127}


def bits16(x):
    return int(x, 16)


# ------------------------------------------------------------------ fp16

def test_fp16_roundtrip_exhaustive(oracle):
    for b in range(65536):
        e = (b >> 10) & 0x1F
        m = b & 0x3FF
        if e == 31 and m != 0:
            assert math.isnan(oracle.h2f(b))
            continue
        assert oracle.f2h(oracle.h2f(b)) == b, hex(b)


def test_h2f_matches_numpy_float16_everywhere(oracle):
    allb = np.arange(65536, dtype=np.uint16)
    ref = allb.view(np.float16).astype(np.float32)
    for b in range(0, 65536, 1):
        r = ref[b]
        v = np.float32(oracle.h2f(b))
        if np.isnan(r):
            assert np.isnan(v)
        else:
            assert v.tobytes() == r.tobytes(), hex(b)


def test_f2h_matches_numpy_on_random_and_boundary_values(oracle):
    rng = np.random.default_rng(123)
    vals = [rng.standard_normal(20000, dtype=np.float32) * np.float32(s)
            for s in (1.0, 1e-3, 1e-5, 3e-8, 100.0, 7e4)]
    # random bit patterns (all magnitudes), ties and near-ties around fp16 grid points
    rb = rng.integers(0, 2**32, size=40000, dtype=np.uint64).astype(np.uint32).view(np.float32)
    grid = np.arange(1, 0x7C00, 37, dtype=np.uint16).view(np.float16).astype(np.float32)
    nxt = (np.arange(1, 0x7C00, 37, dtype=np.uint16) + 1).view(np.float16).astype(np.float32)
    mid = ((grid.astype(np.float64) + nxt.astype(np.float64)) / 2).astype(np.float32)
    ties = [mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(np.inf))]
    edge = np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 65536.0, 1e30, -1e30, np.inf, -np.inf,
                     2.0**-24, 2.0**-25, 2.0**-25 * 1.0000001, 2.0**-26, 2.0**-14, 2.0**-14 * 0.9999],
                    dtype=np.float32)
    x = np.concatenate(vals + [rb[np.isfinite(rb)]] + ties + [edge])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    for v, r in zip(x.tolist(), ref.tolist()):
        assert oracle.f2h(v) == r, (v, hex(r))


# --------------------------------------------------------- hand-built blocks

def _v1_block():
    q = (np.arange(32) % 16) - 8
    return synth.blocks_from_codes(Q4, np.array([[0x3800]], dtype=np.uint16), q.reshape(1, 32)), q


def test_v1_q4_block_bytes_and_products(oracle):
    g = GOLD["V1_q4_block"]
    blk, q = _v1_block()
    assert blk.tobytes().hex() == g["canonical_hex"]
    w = oracle.dequant(Q4, blk, 1, 32)
    assert np.array_equal(w[0], (0.5 * q).astype(np.float32))
    ones = np.ones(32, dtype=np.float16)
    y, B = oracle.gemv(Q4, blk, 1, 32, ones)
    assert y[0] == g["x_ones"]["y"] and B[0] == g["x_ones"]["sum_abs"]
    iota = np.arange(32, dtype=np.float16)
    y, B = oracle.gemv(Q4, blk, 1, 32, iota)
    assert y[0] == g["x_iota"]["y"] and B[0] == g["x_iota"]["sum_abs"]


def test_v1_handwritten_bytes_decode(oracle):
    # The golden hex typed by hand, decoded by the oracle: nibble order and offset.
    raw = np.frombuffer(bytes.fromhex(GOLD["V1_q4_block"]["canonical_hex"]), dtype=np.uint8)
    w = oracle.dequant(Q4, raw, 1, 32)
    assert w[0].tolist() == [0.5 * ((i % 16) - 8) for i in range(32)]


def test_v2_q8_block(oracle):
    g = GOLD["V2_q8_block"]
    q = np.arange(32) - 16
    blk = synth.blocks_from_codes(Q8, np.array([[bits16(g["scale_bits"])]], dtype=np.uint16), q.reshape(1, 32))
    w = oracle.dequant(Q8, blk, 1, 32)
    assert w[0].tolist() == [g["scale_value"] * v for v in q.tolist()]
    y, _ = oracle.gemv(Q8, blk, 1, 32, np.ones(32, dtype=np.float16))
    assert y[0] == g["x_ones"]["y"]
    y, B = oracle.gemv(Q8, blk, 1, 32, np.arange(32, dtype=np.float16))
    assert y[0] == g["x_iota"]["y"] and B[0] == g["x_iota"]["sum_abs"]


@pytest.mark.parametrize("fmt,key,step", [(Q5, "V7_q5_block", 1), (Q6, "V8_q6_block", 2)])
def test_v7_v8_q5_q6_blocks_bytes_and_products(oracle, fmt, key, step):
    """Hand-typed bytes of a 5-bit and a 6-bit block: where the low nibbles and the high bits sit, the
    offset, and the products the block gives with x = ones and x_i = i (derivations in the fixture)."""
    g = GOLD[key]
    raw = np.frombuffer(bytes.fromhex(g["canonical_hex"]), dtype=np.uint8)
    assert raw.size == {Q5: 22, Q6: 26}[fmt]
    d = float(np.array([bits16(g["scale_bits"])], dtype=np.uint16).view(np.float16)[0])
    q = step * np.arange(32) - (16 if fmt == Q5 else 32)
    assert oracle.dequant(fmt, raw, 1, 32)[0].tolist() == [d * v for v in q.tolist()]
    # the block builders produce the same bytes from the codes
    assert synth.blocks_from_codes(fmt, np.array([[bits16(g["scale_bits"])]], dtype=np.uint16), q.reshape(1, 32)).tobytes().hex() == g["canonical_hex"]
    y, B = oracle.gemv(fmt, raw, 1, 32, np.ones(32, dtype=np.float16))
    assert y[0] == g["x_ones"]["y"] and B[0] == g["x_ones"]["sum_abs"]
    y, B = oracle.gemv(fmt, raw, 1, 32, np.arange(32, dtype=np.float16))
    assert y[0] == g["x_iota"]["y"] and B[0] == g["x_iota"]["sum_abs"]


def test_v8_q6_extreme_codes(oracle):
    g = GOLD["V8_q6_block"]["extremes"]
    raw = np.frombuffer(bytes.fromhex(g["hex"]), dtype=np.uint8)
    w = oracle.dequant(Q6, raw, 1, 32)[0]
    assert w[0] == g["w0"] and w[1] == g["w1"] and w[31] == g["w31"]
    assert np.all(w[2:31] == -32.0)


@pytest.mark.parametrize("fmt,key", [(Q5, "q5"), (Q6, "q6")])
def test_v9_q5_q6_ties_to_even(oracle, fmt, key):
    g = GOLD["V9_q5_q6_ties"][key]
    d = float(np.array([bits16(g["scale_bits"])], dtype=np.uint16).view(np.float16)[0])
    w = np.zeros((1, 32), dtype=np.float32)
    w[0, :len(g["w_over_half_step"])] = np.array(g["w_over_half_step"], dtype=np.float32) * np.float32(d / 2)
    for name, quant in _quantisers(oracle):
        blk = quant(fmt, w)
        assert npref.scales_bits(fmt, blk, 1, 32)[0, 0] == bits16(g["scale_bits"]), name
        assert npref.codes(fmt, blk, 1, 32)[0, :len(g["codes"])].tolist() == g["codes"], name
        assert not npref.codes(fmt, blk, 1, 32)[0, len(g["codes"]):].any(), name


def test_q8_minus128_decodes(oracle):
    q = np.full((1, 32), -128)
    blk = synth.blocks_from_codes(Q8, np.array([[0x3C00]], dtype=np.uint16), q)
    assert oracle.dequant(Q8, blk, 1, 32)[0].tolist() == [-128.0] * 32


def test_scale_special_values(oracle):
    q = np.tile(np.arange(-8, 8), 2).reshape(1, 32)
    for bits, val in ((0x0001, 2.0**-24), (0x8001, -(2.0**-24)), (0x0000, 0.0), (0xBC00, -1.0), (0x03FF, 1023 * 2.0**-24)):
        blk = synth.blocks_from_codes(Q4, np.array([[bits]], dtype=np.uint16), q)
        w = oracle.dequant(Q4, blk, 1, 32)[0].astype(np.float64)
        assert np.array_equal(w, val * q[0]), hex(bits)
    for bits in (0x7C00, 0xFC00, 0x7E00):
        blk = synth.blocks_from_codes(Q4, np.array([[bits]], dtype=np.uint16), q)
        with pytest.raises(ValueError):
            oracle.dequant(Q4, blk, 1, 32)


# ---------------------------------------------------------------- quantiser

def _quantisers(oracle):
    return (("oracle", oracle.quantize), ("synth", synth.quantize))


def test_v3_ties_to_even(oracle):
    g = GOLD["V3_q4_ties"]
    w = (np.clip(np.arange(32) - 16, -14, 14) * 2.0**-7).astype(np.float32).reshape(1, 32)
    for name, quant in _quantisers(oracle):
        blk = quant(Q4, w)
        assert npref.scales_bits(Q4, blk, 1, 32)[0, 0] == bits16(g["scale_bits"]), name
        assert npref.codes(Q4, blk, 1, 32)[0].tolist() == g["codes"], name


def test_v4_scale_is_rounded_before_codes(oracle):
    g = GOLD["V4_scale_rounding"]
    w = np.zeros((1, 32), dtype=np.float32)
    for k, v in g["w_nonzero"].items():
        w[0, int(k)] = v
    for fmt, key in ((Q4, "q4"), (Q8, "q8")):
        for name, quant in _quantisers(oracle):
            blk = quant(fmt, w)
            assert npref.scales_bits(fmt, blk, 1, 32)[0, 0] == bits16(g[key]["scale_bits"]), (name, key)
            c = npref.codes(fmt, blk, 1, 32)[0]
            assert c[5:10].tolist() == g[key]["codes_5_to_9"], (name, key)
            assert not c[:5].any() and not c[10:].any()
            assert oracle.h2f(bits16(g[key]["scale_bits"])) == g[key]["scale_value"]


def test_zero_block_quantises_to_zero(oracle):
    w = np.zeros((2, 64), dtype=np.float32)
    w[1, 40] = 1e-9     # amax/7 underflows fp16 -> scale 0 -> codes 0
    for fmt in (Q4, Q8):
        for name, quant in _quantisers(oracle):
            blk = quant(fmt, w)
            assert not npref.codes(fmt, blk, 2, 64).any(), name
            assert not npref.scales_bits(fmt, blk, 2, 64).any(), name


@pytest.mark.parametrize("fmt", FMTS)
def test_two_quantisers_agree_bit_for_bit(oracle, fmt):
    w = synth.weights(77, fmt, 96, 256)
    w[3, 5] = 0.31      # an outlier block
    assert np.array_equal(oracle.quantize(fmt, w), synth.quantize(fmt, w))


@pytest.mark.parametrize("fmt", FMTS)
def test_roundtrip_within_half_step(oracle, fmt):
    w = synth.weights(5, fmt, 64, 512)
    blk = oracle.quantize(fmt, w)
    wq = oracle.dequant(fmt, blk, 64, 512).astype(np.float64)
    d = npref.scales_bits(fmt, blk, 64, 512).view(np.float16).astype(np.float64)
    step = np.repeat(d, 32, axis=1)
    assert np.all(np.abs(w.astype(np.float64) - wq) <= step / 2 * (1 + 2.0**-10))
    c = npref.codes(fmt, blk, 64, 512).reshape(64, 16, 32)
    qmax = QMAX[fmt]
    assert np.all(np.abs(c).max(axis=2) == qmax)        # the arg-max element gets +-QMAX
    assert c.min() >= -qmax                              # this quantiser never emits the lowest code


def test_dequant_product_is_exact_in_fp32():
    # float(d) * q needs at most 11 + 8 significant bits: the fp32 product equals the exact one.
    d = np.arange(0, 0x7C00, dtype=np.uint16).view(np.float16)
    q = np.arange(-128, 128, dtype=np.int32)
    p32 = d.astype(np.float32)[:, None] * q.astype(np.float32)[None, :]
    p64 = d.astype(np.float64)[:, None] * q.astype(np.float64)[None, :]
    assert np.array_equal(p32.astype(np.float64), p64)


# ------------------------------------------------------------------ products

@pytest.mark.parametrize("fmt", FMTS)
def test_dequant_matches_independent_decoder(oracle, fmt):
    N, K = 48, 160
    w = synth.weights(9, fmt, N, K)
    blk = oracle.quantize(fmt, w)
    assert np.array_equal(oracle.dequant(fmt, blk, N, K).astype(np.float64), npref.decode(fmt, blk, N, K))


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("N,K,M", [(32, 32, 1), (64, 96, 3), (96, 64, 5)])
def test_gemm_matches_brute_force_loops(oracle, fmt, N, K, M):
    rng = np.random.default_rng(N * 1000 + K + M + fmt)
    codes = rng.integers(QLO[fmt], QMAX[fmt] + 1, size=(N, K))
    sb = rng.integers(0x1800, 0x3000, size=(N, K // 32)).astype(np.uint16)
    sb[0, 0] |= 0x8000                                  # one negative scale
    blk = synth.blocks_from_codes(fmt, sb, codes)
    X = rng.standard_normal((M, K)).astype(np.float16)
    Y, B = oracle.gemm(fmt, blk, N, K, X)
    scale = sb.view(np.float16).astype(np.float64)
    Xf = [[float(v) for v in row] for row in X]
    for m in range(M):
        for n in range(N):
            s = a = 0.0
            for k in range(K):
                t = scale[n, k // 32] * int(codes[n, k]) * Xf[m][k]
                s += t
                a += abs(t)
            assert Y[m, n] == s and B[m, n] == a


@pytest.mark.parametrize("fmt", FMTS)
def test_unit_scales_reduce_to_integer_matmul(oracle, fmt):
    # scales = 1.0, small integer activations: the product is an integer matrix product.
    rng = np.random.default_rng(11 + fmt)
    N, K, M = 64, 128, 4
    codes = rng.integers(QLO[fmt], QMAX[fmt] + 1, size=(N, K))
    blk = synth.blocks_from_codes(fmt, np.full((N, K // 32), 0x3C00, dtype=np.uint16), codes)
    Xi = rng.integers(-4, 5, size=(M, K))
    Y, B = oracle.gemm(fmt, blk, N, K, Xi.astype(np.float16))
    assert np.array_equal(Y, (Xi.astype(np.int64) @ codes.T.astype(np.int64)).astype(np.float64))
    assert np.array_equal(B, (np.abs(Xi) @ np.abs(codes).T).astype(np.float64))


@pytest.mark.parametrize("fmt", FMTS)
def test_gemm_matches_numpy_float64_matmul(oracle, fmt):
    N, K, M = 128, 512, 7
    blk = oracle.quantize(fmt, synth.weights(21, fmt, N, K))
    X = synth.activations(21, 50 + fmt, M, K)
    Y, B = oracle.gemm(fmt, blk, N, K, X)
    W = npref.decode(fmt, blk, N, K)
    Yn = X.astype(np.float64) @ W.T
    assert np.max(np.abs(Y - Yn) / B) < 1e-12
    Bn = np.abs(X.astype(np.float64)) @ np.abs(W).T
    assert np.allclose(B, Bn, rtol=1e-12, atol=0)


@pytest.mark.parametrize("fmt", FMTS)
def test_gemv_invariants(oracle, fmt):
    N, K = 64, 256
    blk = oracle.quantize(fmt, synth.weights(31, fmt, N, K))
    x = synth.activations(31, 9, K)
    y, B = oracle.gemv(fmt, blk, N, K, x)
    # homogeneity under an exact power-of-two scaling of x
    y4, B4 = oracle.gemv(fmt, blk, N, K, (x.astype(np.float32) * 4).astype(np.float16))
    assert np.array_equal(y4, 4 * y) and np.array_equal(B4, 4 * B)
    # a one-hot activation returns a column of the dequantised matrix exactly
    W = oracle.dequant(fmt, blk, N, K)
    for k in (0, 31, 32, 255):
        e = np.zeros(K, dtype=np.float16)
        e[k] = 1
        yk, Bk = oracle.gemv(fmt, blk, N, K, e)
        assert np.array_equal(yk, W[:, k].astype(np.float64))
        assert np.array_equal(Bk, np.abs(W[:, k]).astype(np.float64))
    # all-zero codes give exactly zero; doubling every scale doubles y
    sb = npref.scales_bits(fmt, blk, N, K)
    z = synth.blocks_from_codes(fmt, sb, np.zeros((N, K), dtype=np.int64))
    yz, Bz = oracle.gemv(fmt, z, N, K, x)
    assert not yz.any() and not Bz.any()
    sb2 = (sb.view(np.float16) * np.float16(2)).view(np.uint16)
    y2, _ = oracle.gemv(fmt, synth.blocks_from_codes(fmt, sb2, npref.codes(fmt, blk, N, K)), N, K, x)
    assert np.array_equal(y2, 2 * y)


def test_gemm_rows_are_independent_gemvs(oracle):
    N, K, M = 32, 64, 3
    blk = oracle.quantize(Q4, synth.weights(41, 0, N, K))
    X = synth.activations(41, 1, M, K)
    Y, B = oracle.gemm(Q4, blk, N, K, X)
    for m in range(M):
        y, b = oracle.gemv(Q4, blk, N, K, X[m])
        assert np.array_equal(Y[m], y) and np.array_equal(B[m], b)


def test_gemm_f64_agrees_with_fp16_entry(oracle):
    N, K, M = 32, 96, 2
    blk = oracle.quantize(Q8, synth.weights(42, 0, N, K))
    X = synth.activations(42, 1, M, K)
    Y, B = oracle.gemm(Q8, blk, N, K, X)
    Y2, B2 = oracle.gemm_f64(Q8, blk, N, K, X.astype(np.float64))
    assert np.array_equal(Y, Y2) and np.array_equal(B, B2)


# ---------------------------------------------------------------- MoE pieces

def test_v5_routing_example(oracle):
    g = GOLD["V5_routing"]
    idx, p = oracle.route(np.array([g["logits"]], dtype=np.float32), g["topk"])
    assert idx[0].tolist() == g["idx"]
    assert np.allclose(p[0], g["p"], rtol=0, atol=5e-11)


def test_v5b_permutation_example(oracle):
    g = GOLD["V5b_permutation"]
    perm, offs = oracle.permute(np.array(g["idx"], dtype=np.int32), 4)
    assert perm.tolist() == g["perm"] and offs.tolist() == g["offsets"]


def test_routing_ties_and_signed_zero(oracle):
    l = np.zeros((1, 8), dtype=np.float32)
    l[0, 3] = -0.0
    idx, p = oracle.route(l, 3)
    assert idx[0].tolist() == [0, 1, 2] and np.allclose(p[0], 1 / 3)
    l = np.array([[1, 5, 5, 5, 0, 5]], dtype=np.float32)
    assert oracle.route(l, 3)[0][0].tolist() == [1, 2, 3]
    with pytest.raises(ValueError):
        oracle.route(np.array([[0, np.nan, 1]], dtype=np.float32), 2)


def test_routing_matches_sort_and_invariants(oracle):
    T, E, k = 257, 128, 8
    lg = synth.logits(4, 99, T, E)
    lg[5, 7] = lg[5, 90]                               # force a tie
    idx, p = oracle.route(lg, k)
    # independent statement: stable argsort of -logit (stable keeps the lower index first)
    ref = np.argsort(-lg.astype(np.float64), axis=1, kind="stable")[:, :k]
    assert np.array_equal(idx, ref.astype(np.int32))
    sel = np.take_along_axis(lg.astype(np.float64), ref, axis=1)
    full = np.exp(lg.astype(np.float64) - lg.max(axis=1, keepdims=True))
    full /= full.sum(axis=1, keepdims=True)
    renorm = np.take_along_axis(full, ref, axis=1)
    renorm /= renorm.sum(axis=1, keepdims=True)       # full softmax then renormalise: same thing
    assert np.allclose(p, renorm, rtol=1e-12, atol=0)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(np.diff(p, axis=1) <= 0)
    assert np.all(np.diff(sel, axis=1) <= 0)
    perm, offs = oracle.permute(idx, E)
    assert sorted(perm.tolist()) == list(range(T * k))
    assert offs[0] == 0 and offs[-1] == T * k and np.all(np.diff(offs) >= 0)
    flat = idx.reshape(-1)
    assert np.array_equal(np.bincount(flat, minlength=E), np.diff(offs))
    for e in range(E):
        seg = perm[offs[e]:offs[e + 1]]
        assert np.all(flat[seg] == e)
        assert np.all(np.diff(seg // k) > 0)           # ascending token index, each token once
    # the sort-based statement of the permutation
    key = flat.astype(np.int64) * (T * k) + np.arange(T * k)
    assert np.array_equal(perm, np.argsort(key, kind="stable").astype(np.int32))


def test_v6_silu(oracle):
    g = GOLD["V6_silu"]
    assert abs(oracle.silu(g["gate"])[()] * g["up"] - g["h"]) < 1e-15
    assert oracle.silu(0.0)[()] == 0.0
    assert abs(oracle.silu(-30.0)[()] + 30.0 * math.exp(-30.0)) < 1e-20
    assert abs(oracle.silu(40.0)[()] - 40.0) < 1e-14


def test_moe_tokens_matches_plain_python_loops(oracle):
    T, H, I, E, k = 4, 64, 32, 8, 2
    seed = 404
    gate, up, down = synth.moe_expert_weights(seed, Q4, E, H, I)
    X = synth.activations(seed, 1, T, H)
    lg = synth.logits(seed, 2, T, E)
    out = oracle.moe_tokens(Q4, lg, X, gate, up, down, H, I, E, k, np.arange(T))
    Wg = npref.decode(Q4, gate, E * I, H).reshape(E, I, H)
    Wu = npref.decode(Q4, up, E * I, H).reshape(E, I, H)
    Wd = npref.decode(Q4, down, E * H, I).reshape(E, H, I)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-float(lg[t, e]), e))[:k]
        ex = [math.exp(float(lg[t, e]) - float(lg[t, order[0]])) for e in order]
        ref = np.zeros(H)
        x = X[t].astype(np.float64)
        for e, w in zip(order, ex):
            gv, uv = Wg[e] @ x, Wu[e] @ x
            h = gv / (1 + np.exp(-gv)) * uv
            ref += (w / sum(ex)) * (Wd[e] @ h)
        assert np.allclose(out[t], ref, rtol=1e-11, atol=1e-14)


def test_moe_tokens_subset_equals_full(oracle):
    T, H, I, E, k = 6, 64, 32, 8, 2
    gate, up, down = synth.moe_expert_weights(405, Q8, E, H, I)
    X = synth.activations(405, 1, T, H)
    lg = synth.logits(405, 2, T, E)
    full = oracle.moe_tokens(Q8, lg, X, gate, up, down, H, I, E, k, np.arange(T))
    sub = oracle.moe_tokens(Q8, lg, X, gate, up, down, H, I, E, k, np.array([4, 1]))
    assert np.array_equal(sub, full[[4, 1]])


# ------------------------------------------------------- property tests

from hypothesis import assume, given, settings, strategies as st  # noqa: E402


@settings(max_examples=60, deadline=None)
@given(st.lists(st.floats(min_value=-4.0, max_value=4.0, allow_nan=False, width=32), min_size=32, max_size=32),
       st.sampled_from(FMTS))
def test_property_quantise_block_roundtrip(oracle, vals, fmt):
    w = np.array(vals, dtype=np.float32).reshape(1, 32)
    blk = oracle.quantize(fmt, w)
    assert np.array_equal(blk, synth.quantize(fmt, w))               # both quantisers, any block
    assume(np.abs(w).max() >= 1e-2)                                  # half-step bound: scales in fp16's normal range
    d = float(npref.scales_bits(fmt, blk, 1, 32).view(np.float16)[0, 0])
    wq = oracle.dequant(fmt, blk, 1, 32).astype(np.float64)
    assert np.all(np.abs(w.astype(np.float64) - wq) <= d / 2 * (1 + 2.0**-10) + 1e-30)
    assert np.array_equal(wq, npref.decode(fmt, blk, 1, 32))


@settings(max_examples=40, deadline=None)
@given(st.integers(1, 9), st.integers(2, 12), st.integers(0, 2**31 - 1))
def test_property_routing_and_permutation(oracle, T, E, seed):
    rng = np.random.default_rng(seed)
    k = int(rng.integers(1, E + 1))
    lg = rng.integers(-3, 4, size=(T, E)).astype(np.float32)          # small integers: many ties
    idx, p = oracle.route(lg, k)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-float(lg[t, e]), e))[:k]
        assert idx[t].tolist() == order
        assert abs(p[t].sum() - 1.0) < 1e-12
    perm, offs = oracle.permute(idx, E)
    flat = idx.reshape(-1)
    assert sorted(perm.tolist()) == list(range(T * k))
    keys = [(int(flat[i]), int(i)) for i in perm]
    assert keys == sorted(keys)
    assert offs.tolist() == [int((flat < e).sum()) for e in range(E + 1)]


def test_composed_moe_bound_reproduces_the_layer_and_scales_with_the_tolerance(oracle):
    """The helper that composes the end-to-end bound of a mixture-of-experts layer from the per-product
    tolerances recomputes the layer stage by stage: its reference must be the oracle's all-fp64 layer, and
    its bound must be positive, dominated by the propagated gate/up term, and small against the output."""
    from tests import util
    fmt, T, E, topk, H, I = 4, 5, 8, 2, 256, 256
    gate, up, down = synth.moe_expert_weights(901, fmt, E, H, I)
    X = synth.activations(901, 1, T, H)
    lg = synth.logits(901, 2, T, E)
    tokens = np.arange(T)
    ref = oracle.moe_tokens(fmt, lg, X, gate, up, down, H, I, E, topk, tokens)
    ref2, bound = util.moe_composed_bound(oracle, fmt, lg, X, gate, up, down, H, I, E, topk, tokens)
    assert np.allclose(ref, ref2, rtol=1e-12, atol=1e-15)
    assert np.all(bound > 1e-5)
    # never tighter than the combine's own tolerance, and not vacuous
    assert np.all(bound >= 2e-3 * np.abs(ref) + 1e-5)
    assert np.median(bound) < np.abs(ref).max()
    # token 0 once more with the independent numpy decoder and plain matrix products
    from tests import npref
    idx, p = oracle.route(lg, topk)
    x = X[0].astype(np.float64)
    tol = lambda B: 2e-3 * B + 1e-5
    want = np.zeros(H)
    gu, dn = len(gate) // E, len(down) // E
    mag = np.zeros(H)
    for j in range(topk):
        e = int(idx[0, j])
        Wg, Wu = npref.decode(fmt, gate[e * gu:(e + 1) * gu], I, H), npref.decode(fmt, up[e * gu:(e + 1) * gu], I, H)
        Wd = npref.decode(fmt, down[e * dn:(e + 1) * dn], H, I)
        G, U = Wg @ x, Wu @ x
        BG, BU = np.abs(Wg) @ np.abs(x), np.abs(Wu) @ np.abs(x)
        sG = G / (1 + np.exp(-G))
        h = sG * U
        E_h = 1.1 * tol(BG) * np.abs(U) + np.abs(sG) * tol(BU) + 1.1 * tol(BG) * tol(BU) + 2.0**-11 * np.abs(h)
        E_D = 2e-3 * (np.abs(Wd) @ np.abs(h)) + 1.002 * (np.abs(Wd) @ E_h) + 1e-5
        D = Wd @ h
        want += p[0, j] * E_D + 2e-3 * p[0, j] * (np.abs(D) + E_D)
        mag += np.abs(D) + E_D
    want += 1e-5 + 1e-6 * mag
    assert np.allclose(bound[0], want, rtol=1e-9, atol=0)
