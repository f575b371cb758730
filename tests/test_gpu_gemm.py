"""GPU parity: qmm_gemm (tcgen05 tensor cores, weights expanded through tensor
memory) against the CPU oracle.  Every output must satisfy
|Y_gpu - Y_ref| <= 2e-3 * sum_k |w x| + 1e-5."""
import numpy as np
import pytest
import torch

from paper_2607_00501_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
Q4, Q8 = 4, 8


@pytest.fixture(scope="module")
def qmm():
    from paper_2607_00501_b200 import qmm as _qmm
    assert torch.cuda.is_available()
    _qmm.lib()
    return _qmm


def run_gemm(qmm, oracle, fmt, blocks, N, K, X, what, rows=None):
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    ws = torch.zeros(qmm.gemm_workspace_bytes(fmt, X.shape[0], N, K), dtype=torch.uint8, device="cuda")
    Y = qmm.gemm(fmt, packed, N, K, util.dev(X), ws=ws)
    qmm.status_check(ws)
    Yh = util.host_f64(Y)
    sel = np.arange(X.shape[0]) if rows is None else np.asarray(rows)
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X[sel])
    return util.assert_within_tol(Yh[sel], Y_ref, B, what)


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("M,N,K", [(128, 128, 256), (32, 256, 256), (1, 128, 512), (77, 384, 768), (130, 256, 1024),
                                   (200, 640, 512), (64, 128, 4096), (700, 6400, 512), (1000, 1280, 256), (4100, 256, 256)])
def test_gemm_small_shapes(qmm, oracle, fmt, M, N, K):
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=M + 3 * N + K + fmt, special_scales=False)
    X = synth.activations(70, M + N + K, M, K)
    run_gemm(qmm, oracle, fmt, blocks, N, K, X, "gemm M=%d N=%d K=%d fmt=%d" % (M, N, K, fmt))


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("M,N,K", [(96, 256, 512), (33, 128, 2048), (300, 384, 1024), (700, 1280, 512), (150, 256, 8192)])
def test_gemm_negative_zero_and_subnormal_scales(qmm, oracle, fmt, M, N, K):
    """One block in 16 has a negative, zero, -0 or subnormal scale.  Negative and zero scales are
    covered by the stated tolerance; a weight whose product d*q is a subnormal fp16 adds the
    documented 2^-25 |x| per such weight (it enters the tensor core with an absolute error)."""
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=11 * M + N + K + fmt, special_scales=True)
    X = synth.activations(75, M + N + K, M, K)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    ws = torch.zeros(qmm.gemm_workspace_bytes(fmt, M, N, K), dtype=torch.uint8, device="cuda")
    Y = util.host_f64(qmm.gemm(fmt, packed, N, K, util.dev(X), ws=ws))
    qmm.status_check(ws)
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
    extra = util.subnormal_weight_term(oracle.dequant(fmt, blocks, N, K), X)
    assert extra.max() > 0                                       # the case does contain such weights
    assert np.all(np.isfinite(Y))
    worst = float(np.max(np.abs(Y - Y_ref) / (util.RTOL_SUMABS * B + util.ATOL + extra)))
    assert worst <= 1.0, "max |err| / documented bound = %.3f" % worst
    # the same blocks without the subnormal kind: the plain tolerance, nothing added
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=11 * M + N + K + fmt, special_scales="no_subnormal")
    run_gemm(qmm, oracle, fmt, blocks, N, K, X, "negative / zero scales M=%d N=%d K=%d fmt=%d" % (M, N, K, fmt))


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("side", ["normal", "subnormal"])
def test_gemm_on_both_sides_of_the_fp16_subnormal_limit(qmm, oracle, fmt, side):
    """Every scale just above 2^-14 (each non-zero product d*q is a normal fp16: the stated tolerance
    holds as it stands), then every scale subnormal (each product below 2^-14 has an absolute error of
    up to 2^-25: the documented wider bound holds, and the stated one is not promised)."""
    M, N, K = 64, 256, 1024
    bits = (0x0400, 0x0800) if side == "normal" else (0x0001, 0x0400)
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=77 + fmt, special_scales=False, scale_bits=bits)
    X = synth.activations(76, fmt, M, K)
    Y = util.host_f64(qmm.gemm(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(X)))
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
    W = oracle.dequant(fmt, blocks, N, K)
    extra = util.subnormal_weight_term(W, X)
    if side == "normal":
        assert extra.max() == 0
        util.assert_within_tol(Y, Y_ref, B, "scales just above 2^-14")
    else:
        assert extra.min() > 0
        assert np.all(np.abs(Y - Y_ref) <= util.RTOL_SUMABS * B + util.ATOL + extra)
    # the GEMV multiplies codes exactly and scales in fp32: the stated tolerance on both sides
    y = util.host_f64(qmm.gemv(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(X[0])))
    util.assert_within_tol(y, Y_ref[0], B[0], "gemv, " + side)


def test_gemm_large_scales_up_to_the_documented_limit(qmm, oracle):
    """|d| * max|q| just below 65504 stays finite and inside the tolerance; qmm_packed_check accepts it
    and rejects a scale beyond the limit, an inf scale, canonical bytes passed as packed and a buffer of
    the other format."""
    M, N, K = 40, 128, 256
    rng = np.random.default_rng(3)
    for fmt, top in ((Q4, 8184.0), (Q8, 511.0)):
        codes = rng.integers(-8 if fmt == Q4 else -128, 8 if fmt == Q4 else 128, size=(N, K))
        sb = np.full((N, K // 32), np.float16(top).view(np.uint16), dtype=np.uint16)
        blocks = synth.blocks_from_codes(fmt, sb, codes)
        X = (synth.activations(78, fmt, M, K).astype(np.float32) * 2.0**-9).astype(np.float16)   # keeps |Y| inside fp16
        packed = qmm.pack(fmt, util.dev(blocks), N, K)
        ws = torch.zeros(qmm.gemm_workspace_bytes(fmt, M, N, K), dtype=torch.uint8, device="cuda")
        Y = util.host_f64(qmm.gemm(fmt, packed, N, K, util.dev(X), ws=ws))
        Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
        assert np.abs(Y_ref).max() < 60000
        util.assert_within_tol(Y, Y_ref, B, "large scales fmt=%d" % fmt)
        qmm.packed_check(fmt, packed, N, K, ws)
        qmm.status_check(ws)                                     # accepted
        for bad_bits in (np.float16(top * 1.01).view(np.uint16), 0x7C00, 0xFE00):
            sb2 = sb.copy()
            sb2[77, 3] = bad_bits
            bad = qmm.pack(fmt, util.dev(synth.blocks_from_codes(fmt, sb2, codes)), N, K)
            qmm.packed_check(fmt, bad, N, K, ws)
            with pytest.raises(qmm.QmmError) as ei:
                qmm.status_check(ws)
            assert ei.value.status == 8
            qmm.status_check(ws)                                 # reported once, then clear
    # realistic weights: the packed buffer passes; its canonical bytes, and the buffer read as the other
    # format, do not
    N, K = 512, 1024
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for fmt, other in ((Q4, Q8), (Q8, Q4)):
        canon = util.dev(synth.quantize(fmt, synth.weights(79, fmt, N, K)))
        packed = qmm.pack(fmt, canon, N, K)
        qmm.packed_check(fmt, packed, N, K, ws)
        qmm.status_check(ws)
        qmm.packed_check(fmt, canon, N, K, ws)
        with pytest.raises(qmm.QmmError) as ei:
            qmm.status_check(ws)
        assert ei.value.status == 8 and "packed" in ei.value.message
        N2 = N * (18 if fmt == Q4 else 34) // (18 if other == Q4 else 34) // 128 * 128    # rows of the other format that fit
        qmm.packed_check(other, packed, N2, K, ws)
        with pytest.raises(qmm.QmmError):
            qmm.status_check(ws)


def test_bounded_wait_gives_up_and_the_context_stays_usable(qmm, oracle):
    """A wait on a barrier that nothing completes runs into its limit (about a millisecond here), the
    kernel records QMM_ERR_DEVICE_TIMEOUT in the status word and returns; the host reads status 7, and a
    product on the same workspace then runs normally."""
    M, N, K = 100, 256, 512
    blocks = synth.quantize(Q4, synth.weights(80, 0, N, K))
    X = synth.activations(80, 1, M, K)
    packed = qmm.pack(Q4, util.dev(blocks), N, K)
    ws = torch.zeros(qmm.gemm_workspace_bytes(Q4, M, N, K), dtype=torch.uint8, device="cuda")
    qmm.debug_wait_give_up(ws, 2_000_000)
    with pytest.raises(qmm.QmmError) as ei:
        qmm.status_check(ws)
    assert ei.value.status == 7 and "bounded wait" in ei.value.message
    Y = qmm.gemm(Q4, packed, N, K, util.dev(X), ws=ws)
    qmm.status_check(ws)
    Y_ref, B = oracle.gemm(Q4, blocks, N, K, X)
    util.assert_within_tol(util.host_f64(Y), Y_ref, B, "gemm after a give-up")


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemm_integer_case_is_exact(qmm, fmt):
    # unit scales, small integer activations: every product and partial sum is an exact integer
    rng = np.random.default_rng(17 + fmt)
    M, N, K = 96, 256, 512
    lo, hi = (-8, 8) if fmt == Q4 else (-127, 128)
    codes = np.where(rng.random((N, K)) < (0.25 if fmt == Q4 else 0.01), rng.integers(lo, hi, size=(N, K)), 0)
    Xi = rng.integers(-2, 3, size=(M, K))
    ref = Xi.astype(np.int64) @ codes.T.astype(np.int64)
    assert np.abs(ref).max() < 2048
    blocks = synth.blocks_from_codes(fmt, np.full((N, K // 32), 0x3C00, dtype=np.uint16), codes)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    Y = qmm.gemm(fmt, packed, N, K, util.dev(Xi.astype(np.float16)))
    assert np.array_equal(util.host_f64(Y), ref.astype(np.float64))


def test_gemm_strided_inputs_and_guard_bytes(qmm, oracle):
    M, N, K = 100, 256, 512
    blocks = synth.quantize(Q4, synth.weights(71, 0, N, K))
    packed = qmm.pack(Q4, util.dev(blocks), N, K)
    X = synth.activations(71, 1, M, K)
    Xbuf = torch.full((M, K + 64), 9.0, dtype=torch.float16, device="cuda")
    Xbuf[:, :K] = util.dev(X)
    Ybuf = torch.full((M + 2, N + 16), 5.0, dtype=torch.float16, device="cuda")
    qmm.gemm(Q4, packed, N, K, Xbuf[:, :K], Y=Ybuf[1:M + 1, :N])
    Y_ref, B = oracle.gemm(Q4, blocks, N, K, X)
    util.assert_within_tol(util.host_f64(Ybuf[1:M + 1, :N]), Y_ref, B, "strided")
    assert torch.all(Ybuf[0] == 5.0) and torch.all(Ybuf[M + 1] == 5.0) and torch.all(Ybuf[:, N:] == 5.0)


def test_status_word_is_decoded_and_cleared(qmm):
    # the kernels write QMM_ERR_DEVICE_TIMEOUT (7) into the workspace's status word when a bounded wait
    # gives up; here the word is set by hand to check the host side: report once, then clear
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    qmm.status_check(ws)
    ws.view(torch.int32)[0] = 7
    with pytest.raises(qmm.QmmError) as ei:
        qmm.status_check(ws)
    assert ei.value.status == 7 and "bounded wait" in ei.value.message
    qmm.status_check(ws)
    assert int(ws.view(torch.int32)[0]) == 0


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("force,M,N,K", [("128,5", 100, 256, 2048), ("32,3", 7, 128, 4096), ("256,7", 300, 384, 1024),
                                         ("160,9", 170, 512, 1024), ("192,9", 200, 512, 1024), ("64,1", 33, 128, 256),
                                         (None, 48, 256, 8192), (None, 256, 128, 4096), (None, 520, 2432, 1024)])
def test_gemm_tiles_cut_across_blocks(qmm, oracle, fmt, force, M, N, K):
    """Blocks own equal shares of the (tile, k-block) units (forced to odd sizes here); a tile cut by a
    share boundary is summed from fp32 partial results, in contributor order, by a second kernel."""
    qmm.debug_config("gemm_force", force)
    assert qmm.gemm_workspace_bytes(fmt, M, N, K) > 8192          # these shapes do cut tiles
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=M + N + K + fmt, special_scales=False)
    X = synth.activations(71, M + N + K, M, K)
    run_gemm(qmm, oracle, fmt, blocks, N, K, X, "cut-tile gemm M=%d N=%d K=%d fmt=%d" % (M, N, K, fmt))
    # same bits on every call
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    Xd = util.dev(X)
    first = qmm.gemm(fmt, packed, N, K, Xd).cpu()
    for _ in range(3):
        assert torch.equal(first, qmm.gemm(fmt, packed, N, K, Xd).cpu())


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemm_last_round_cut_into_shares(qmm, oracle, fmt):
    """Many tiles, a nearly empty last round and a long K: every block takes its whole tiles, then an
    equal share of the units of the last round's tiles (here 152 tiles on 148 SMs: 4 tiles in shares
    of 8 of their 128 k-blocks), which the second kernel adds up.  Rows of the cut tiles and of whole tiles are checked."""
    qmm.debug_config(None)
    M, N, K = 2048, 2432, 8192
    assert qmm.gemm_workspace_bytes(fmt, M, N, K) == 8192 + 2 * 148 * 256 * 128 * 4
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=5 + fmt, special_scales=False)
    X = synth.activations(73, fmt, M, K)
    rows = np.array([0, 255, 256, 1000, 1791, 1792, 1800, 1919, 2000, 2047])     # the last token tile holds the cut tiles
    run_gemm(qmm, oracle, fmt, blocks, N, K, X, "cut last round fmt=%d" % fmt, rows=rows)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    Xd = util.dev(X)
    first = qmm.gemm(fmt, packed, N, K, Xd).cpu()
    for _ in range(2):
        assert torch.equal(first, qmm.gemm(fmt, packed, N, K, Xd).cpu())
    # the same product with the last round left whole agrees to fp16 rounding of nearly equal fp32 sums
    qmm.debug_config("gemm_no_tail_cut", "1")
    assert qmm.gemm_workspace_bytes(fmt, M, N, K) == 8192
    whole = qmm.gemm(fmt, packed, N, K, Xd).cpu()
    assert torch.equal(first[:1792], whole[:1792])                                # whole tiles: identical
    assert float((first.float() - whole.float()).abs().max()) <= 2e-3 * float(whole.float().abs().max())


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("M", [2048, 1990, 1900])
def test_gemm_last_round_as_half_tiles(qmm, oracle, fmt, M):
    """152 tiles of 256 tokens on 148 SMs, short K: the four tiles of the second round run as eight
    half tiles (MMAs of 128 token columns), each a product of its own -- so the result is the same
    bits as with whole tiles.  M = 1990 leaves the second half of the last token tile ragged,
    M = 1900 leaves it empty."""
    qmm.debug_config(None)
    N, K = 2432, 512
    assert qmm.gemm_workspace_bytes(fmt, M, N, K) == 8192                         # no partial sums
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=9 + fmt, special_scales=False)
    X = synth.activations(74, fmt, M, K)
    rows = np.unique(np.concatenate([[0, 255, 1000, 1791], np.arange(1792, M, 7), [M - 1]]))
    run_gemm(qmm, oracle, fmt, blocks, N, K, X, "half tiles fmt=%d M=%d" % (fmt, M), rows=rows)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    Xd = util.dev(X)
    halves = qmm.gemm(fmt, packed, N, K, Xd).cpu()
    qmm.debug_config("gemm_no_tail_cut", "1")
    whole = qmm.gemm(fmt, packed, N, K, Xd).cpu()
    assert torch.equal(halves, whole)


def test_gemm_matches_gemv_rows(qmm):
    # the M = 1 product through both kernels agrees to fp16 rounding of nearly equal fp32 sums
    N, K = 384, 1024
    blocks = synth.quantize(Q8, synth.weights(72, 0, N, K))
    packed = qmm.pack(Q8, util.dev(blocks), N, K)
    x = util.dev(synth.activations(72, 1, K))
    y1 = qmm.gemv(Q8, packed, N, K, x).float()
    y2 = qmm.gemm(Q8, packed, N, K, x.reshape(1, K)).float()[0]
    assert torch.allclose(y1, y2, rtol=4e-3, atol=1e-3)


@pytest.mark.parametrize("shape", synth.CFG3["shapes"])
@pytest.mark.parametrize("M", synth.CFG3["Ms"])
def test_cfg3_prefill_full_size_sampled_rows(qmm, oracle, shape, M):
    name, N, K = shape
    c = synth.CFG3
    blocks = synth.quantize(c["fmt"], synth.weights(c["seed"], 0 if name == "gate_up" else 1, N, K))
    X = synth.activations(c["seed"], 10 + M, M, K)
    rng = np.random.default_rng(M + N)
    rows = np.unique(np.concatenate([[0, M - 1, M // 2], rng.integers(0, M, size=13)]))
    run_gemm(qmm, oracle, c["fmt"], blocks, N, K, X, "cfg3 %s M=%d" % (name, M), rows=rows)
