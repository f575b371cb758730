"""GPU parity: qmm_gemm for a handful of tokens (M <= 8), which streams the codes
into registers like the decode kernels and multiplies eight tokens per warp-level MMA, rather than
running on the tensor-memory prefill kernel.  Every output must satisfy
|Y_gpu - Y_ref| <= 2e-3 * sum_k |w x| + 1e-5 against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2607_00501_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
FMTS = [4, 5, 6, 8]


@pytest.fixture(scope="module")
def qmm():
    from paper_2607_00501_b200 import qmm as _qmm
    assert torch.cuda.is_available()
    _qmm.lib()
    return _qmm


def gemm(qmm, fmt, packed, N, K, Xd, **kw):
    ws = torch.zeros(qmm.gemm_workspace_bytes(fmt, Xd.shape[0], N, K), dtype=torch.uint8, device="cuda")
    Y = qmm.gemm(fmt, packed, N, K, Xd, ws=ws, **kw)
    qmm.status_check(ws)
    return Y


# (N, K): one item, ragged warp shares (K / tile not a multiple of the warps), K split over a cluster
# (few row groups, long rows), many items per block (more pairs than resident blocks)
SHAPES = [(128, 256), (384, 768), (256, 2048), (128, 8192), (1280, 512), (19200, 256)]


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 6, 7, 8])
def test_few_tokens_every_m(qmm, oracle, fmt, M):
    for N, K in SHAPES[:4]:
        blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=7 * M + N + K + fmt, special_scales=True)
        X = synth.activations(81, M + N + K, M, K)
        packed = qmm.pack(fmt, util.dev(blocks), N, K)
        Y = util.host_f64(gemm(qmm, fmt, packed, N, K, util.dev(X)))
        Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
        util.assert_within_tol(Y, Y_ref, B, "few tokens M=%d N=%d K=%d fmt=%d" % (M, N, K, fmt))


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("N,K", SHAPES[4:])
def test_few_tokens_many_items_per_block(qmm, oracle, fmt, N, K):
    M = 7
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=N + K + fmt, special_scales=True)
    X = synth.activations(82, N + K, M, K)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    Y = util.host_f64(gemm(qmm, fmt, packed, N, K, util.dev(X)))
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
    util.assert_within_tol(Y, Y_ref, B, "few tokens, many items N=%d K=%d fmt=%d" % (N, K, fmt))


@pytest.mark.parametrize("fmt", [4, 8])
def test_a_token_row_does_not_depend_on_the_other_tokens(qmm, fmt):
    """Row m of Y is the same bits whatever M is (3..8) and whichever slot of the token group it rides in:
    the order of its fp32 additions is fixed by the shape alone.  A repeated call gives the same bits.
    One and two tokens run on the single-token kernel: their rows are the bits of qmm_gemv."""
    for N, K in ((256, 2048), (128, 8192), (640, 512)):
        blocks = synth.quantize(fmt, synth.weights(83, fmt, N, K))
        packed = qmm.pack(fmt, util.dev(blocks), N, K)
        X = util.dev(synth.activations(83, N + K, 8, K))
        Y8 = gemm(qmm, fmt, packed, N, K, X)
        assert torch.equal(Y8, gemm(qmm, fmt, packed, N, K, X))
        for M in (3, 5, 7):
            assert torch.equal(gemm(qmm, fmt, packed, N, K, X[:M]), Y8[:M])
        # token 5 in the first slot of the group, and in the third slot behind tokens 0 and 1
        assert torch.equal(gemm(qmm, fmt, packed, N, K, X[5:8])[0], Y8[5])
        assert torch.equal(gemm(qmm, fmt, packed, N, K, X[[0, 1, 5]].contiguous())[2], Y8[5])
        # two tokens: each row as qmm_gemv computes it, whichever of the two it is
        y3, y6 = qmm.gemv(fmt, packed, N, K, X[3].contiguous()), qmm.gemv(fmt, packed, N, K, X[6].contiguous())
        Y2 = gemm(qmm, fmt, packed, N, K, X[[3, 6]].contiguous())
        assert torch.equal(Y2[0], y3) and torch.equal(Y2[1], y6)
        Y2 = gemm(qmm, fmt, packed, N, K, X[[6, 3]].contiguous())
        assert torch.equal(Y2[0], y6) and torch.equal(Y2[1], y3)
        assert torch.equal(gemm(qmm, fmt, packed, N, K, X[3:4])[0], y3)


@pytest.mark.parametrize("fmt", FMTS)
def test_few_tokens_integer_case_is_exact(qmm, fmt):
    rng = np.random.default_rng(23 + fmt)
    M, N, K = 6, 256, 1024
    lo, hi = {4: (-8, 8), 5: (-16, 16), 6: (-32, 32), 8: (-127, 128)}[fmt]
    codes = np.where(rng.random((N, K)) < (0.2 if fmt != 8 else 0.01), rng.integers(lo, hi, size=(N, K)), 0)
    Xi = rng.integers(-2, 3, size=(M, K))
    ref = Xi.astype(np.int64) @ codes.T.astype(np.int64)
    assert np.abs(ref).max() < 2048
    blocks = synth.blocks_from_codes(fmt, np.full((N, K // 32), 0x3C00, dtype=np.uint16), codes)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    Y = gemm(qmm, fmt, packed, N, K, util.dev(Xi.astype(np.float16)))
    assert np.array_equal(util.host_f64(Y), ref.astype(np.float64))


def test_few_tokens_strided_inputs_and_guard_bytes(qmm, oracle):
    M, N, K = 5, 256, 768
    blocks = synth.quantize(4, synth.weights(84, 0, N, K))
    packed = qmm.pack(4, util.dev(blocks), N, K)
    X = synth.activations(84, 1, M, K)
    Xbuf = torch.full((M, K + 64), 9.0, dtype=torch.float16, device="cuda")
    Xbuf[:, :K] = util.dev(X)
    Ybuf = torch.full((M + 2, N + 16), 5.0, dtype=torch.float16, device="cuda")
    qmm.gemm(4, packed, N, K, Xbuf[:, :K], Y=Ybuf[1:M + 1, :N])
    Y_ref, B = oracle.gemm(4, blocks, N, K, X)
    util.assert_within_tol(util.host_f64(Ybuf[1:M + 1, :N]), Y_ref, B, "strided")
    assert torch.all(Ybuf[0] == 5.0) and torch.all(Ybuf[M + 1] == 5.0) and torch.all(Ybuf[:, N:] == 5.0)


@pytest.mark.parametrize("fmt", [4, 8])
@pytest.mark.parametrize("M", [1, 3, 8])
def test_tensor_core_kernel_still_takes_few_tokens_when_asked(qmm, oracle, fmt, M):
    """qmm_debug_config("gemm_no_small") sends M <= 8 through the prefill kernel: both kernels meet the
    tolerance on the same inputs."""
    N, K = 384, 1024
    blocks = synth.quantize(fmt, synth.weights(85, fmt, N, K))
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    X = synth.activations(85, M, M, K)
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
    util.assert_within_tol(util.host_f64(gemm(qmm, fmt, packed, N, K, util.dev(X))), Y_ref, B, "few-token kernel")
    qmm.debug_config("gemm_no_small", "1")
    util.assert_within_tol(util.host_f64(gemm(qmm, fmt, packed, N, K, util.dev(X))), Y_ref, B, "prefill kernel")


@pytest.mark.parametrize("shape", synth.CFG3["shapes"])
@pytest.mark.parametrize("M", [2, 5, 8])
def test_few_tokens_on_the_full_size_prefill_shapes(qmm, oracle, shape, M):
    name, N, K = shape
    c = synth.CFG3
    blocks = synth.quantize(c["fmt"], synth.weights(c["seed"], 0 if name == "gate_up" else 1, N, K))
    X = synth.activations(c["seed"], 20 + M, M, K)
    packed = qmm.pack(c["fmt"], util.dev(blocks), N, K)
    Y = util.host_f64(gemm(qmm, c["fmt"], packed, N, K, util.dev(X)))
    Y_ref, B = oracle.gemm(c["fmt"], blocks, N, K, X)
    util.assert_within_tol(Y, Y_ref, B, "cfg3 %s M=%d" % (name, M))


# ------------------------------------------------------------------ qmm_gemm_batch

@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("M", [1, 2, 3, 8])
def test_gemm_batch_mixed_shapes(qmm, oracle, fmt, M):
    """One launch over problems that differ in N and K (short K: fewer tiles than warps; long K; many
    row groups), strided X and Y with guard values; every output against the oracle; repeatable."""
    shapes = [(128, 256), (384, 1024), (128, 8192), (640, 512), (256, 2048), (128, 256), (2176, 1280)]
    probs, refs, bufs = [], [], []
    for i, (N, K) in enumerate(shapes):
        blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=97 + 10 * fmt + i, special_scales=True)
        X = synth.activations(97, 100 + i, M, K)
        Xbuf = torch.full((M, K + 8 * (i % 3)), 7.0, dtype=torch.float16, device="cuda")
        Xbuf[:, :K] = util.dev(X)
        Ybuf = torch.full((M, N + 16), 9.0, dtype=torch.float16, device="cuda")
        probs.append((qmm.pack(fmt, util.dev(blocks), N, K), N, K, Xbuf[:, :K], Ybuf[:, :N]))
        refs.append(oracle.gemm(fmt, blocks, N, K, X))
        bufs.append(Ybuf)
    arr = qmm.gemm_batch_problems(probs)
    qmm.gemm_batch(fmt, arr)
    torch.cuda.synchronize()
    for (p, N, K, X, Y), (Y_ref, B), Ybuf in zip(probs, refs, bufs):
        util.assert_within_tol(util.host_f64(Y), Y_ref, B, "batch %dx%d M=%d fmt=%d" % (N, K, M, fmt))
        assert torch.all(Ybuf[:, N:] == 9.0)
    first = [b.clone() for b in bufs]
    qmm.gemm_batch(fmt, arr)
    for f, b in zip(first, bufs):
        assert torch.equal(f, b)


@pytest.mark.parametrize("fmt", [4, 8])
def test_gemm_batch_rows_equal_qmm_gemm(qmm, fmt):
    """Where qmm_gemm does not split K across blocks (many row groups) the two calls add in the same order:
    the batched launch gives the same bits, and a row does not depend on M (3 <= M <= 8: one and two
    tokens run on the single-token kernels, which add in another order)."""
    N, K, M = 38400, 512, 6
    blocks = synth.quantize(fmt, synth.weights(98, fmt, N, K))
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    X = util.dev(synth.activations(98, 1, M, K))
    Y1 = gemm(qmm, fmt, packed, N, K, X)
    Y2 = torch.empty_like(Y1)
    qmm.gemm_batch(fmt, qmm.gemm_batch_problems([(packed, N, K, X, Y2)]))
    assert torch.equal(Y1, Y2)
    Y3 = torch.empty((3, N), dtype=torch.float16, device="cuda")
    qmm.gemm_batch(fmt, qmm.gemm_batch_problems([(packed, N, K, X[3:6], Y3)]))
    assert torch.equal(Y3, Y1[3:6])


@pytest.mark.parametrize("fmt", [4, 8])
@pytest.mark.parametrize("M", [2, 8])
def test_cfg1_two_layers_full_size_for_a_batch_of_sequences(qmm, oracle, fmt, M):
    """All 14 matrices of two decoder layers at their real sizes for 2 / 8 sequences in one launch (two
    sequences ride in the single-token kernel's MMAs, eight run on the few-token ring kernel)."""
    probs, refs = [], []
    for layer in (0, 15):
        for name, N, K, act, w in synth.cfg1_layer_weights(layer):
            blocks = synth.quantize(fmt, w)
            X = synth.activations(99, 16 * layer + len(probs), M, K)
            Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            probs.append((qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(X), Y))
            refs.append((name, oracle.gemm(fmt, blocks, N, K, X)))
    qmm.gemm_batch(fmt, qmm.gemm_batch_problems(probs))
    torch.cuda.synchronize()
    for (p, N, K, X, Y), (name, (Y_ref, B)) in zip(probs, refs):
        util.assert_within_tol(util.host_f64(Y), Y_ref, B, "cfg1 batch of %d, %s" % (M, name))


def test_gemm_batch_more_problems_than_one_launch_holds(qmm, oracle):
    fmt, M = 4, 4
    shapes = [(128, 256), (256, 512), (128, 1024)]
    probs, refs = [], []
    for i in range(150):
        N, K = shapes[i % 3]
        blocks = synth.quantize(fmt, synth.weights(96, i % 7, N, K))
        X = synth.activations(96, 300 + i, M, K)
        probs.append((qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(X), torch.empty((M, N), dtype=torch.float16, device="cuda")))
        refs.append(oracle.gemm(fmt, blocks, N, K, X))
    qmm.gemm_batch(fmt, qmm.gemm_batch_problems(probs))
    torch.cuda.synchronize()
    for (p, N, K, X, Y), (Y_ref, B) in zip(probs, refs):
        util.assert_within_tol(util.host_f64(Y), Y_ref, B, "150 problems")


def test_gemm_batch_argument_checks(qmm):
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    Y = torch.zeros((4, 128), dtype=torch.float16, device="cuda")
    X = torch.zeros((4, 256), dtype=torch.float16, device="cuda")
    L = qmm.lib()
    P = qmm.GemmProblem
    good = qmm.gemm_batch_problems([(buf, 128, 256, X, Y)])
    assert L.qmm_gemm_batch(4, good, 1, 4, None) == 0
    assert L.qmm_gemm_batch(4, good, 0, 4, None) == 0 and L.qmm_gemm_batch(4, good, 1, 0, None) == 0
    assert L.qmm_gemm_batch(4, good, -1, 4, None) == 1 and L.qmm_gemm_batch(4, good, 1, -1, None) == 1
    assert L.qmm_gemm_batch(4, good, 1, 9, None) == 5                                    # more than eight tokens
    assert L.qmm_gemm_batch(4, None, 1, 4, None) == 1
    assert L.qmm_gemm_batch(7, good, 1, 4, None) == 1                                    # unknown format
    bad = (P * 1)(P(buf.data_ptr() + 8, X.data_ptr(), Y.data_ptr(), 128, 256, 256, 128))
    assert L.qmm_gemm_batch(4, bad, 1, 4, None) == 3                                     # packed not 32-byte aligned
    bad = (P * 1)(P(buf.data_ptr(), X.data_ptr(), Y.data_ptr(), 100, 256, 256, 128))
    assert L.qmm_gemm_batch(4, bad, 1, 4, None) == 5                                     # N not a multiple of 128
    bad = (P * 1)(P(buf.data_ptr(), X.data_ptr(), Y.data_ptr(), 128, 256, 128, 128))
    assert L.qmm_gemm_batch(4, bad, 1, 4, None) == 2                                     # ldx < K
    bad = (P * 1)(P(buf.data_ptr(), X.data_ptr(), Y.data_ptr(), 128, 256, 260, 128))
    assert L.qmm_gemm_batch(4, bad, 1, 4, None) == 3                                     # ldx not a multiple of 8
    bad = (P * 1)(P(buf.data_ptr(), 0, Y.data_ptr(), 128, 256, 256, 128))
    assert L.qmm_gemm_batch(4, bad, 1, 4, None) == 1                                     # null X
    torch.cuda.synchronize()
