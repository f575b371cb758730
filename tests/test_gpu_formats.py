"""GPU parity of the 5-bit and 6-bit block formats (pack, dequant, GEMV, dense GEMM) against the CPU
oracle: dequantised weights bit-exact, every product within 2e-3 * sum|w x| + 1e-5."""
import numpy as np
import pytest
import torch

from paper_2607_00501_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
Q5, Q6 = 5, 6
RANGE = {5: (-16, 16), 6: (-32, 32)}


@pytest.fixture(scope="module")
def qmm():
    from paper_2607_00501_b200 import qmm as _qmm
    assert torch.cuda.is_available()
    _qmm.lib()
    return _qmm


@pytest.mark.parametrize("fmt", [Q5, Q6])
def test_sizes_and_dequant_bit_exact(qmm, oracle, fmt):
    assert qmm.canonical_bytes(fmt, 128, 256) == 128 * 8 * {5: 22, 6: 26}[fmt] == qmm.packed_bytes(fmt, 128, 256)
    for N, K, seed in ((128, 256, 1), (384, 768, 2), (256, 2048, 3)):
        blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=seed + fmt)          # incl. negative, zero, subnormal scales
        w = qmm.dequant(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K).cpu().numpy()
        assert w.tobytes() == oracle.dequant(fmt, blocks, N, K).tobytes()
    # every code value in every position of a word, every scale class
    N, K = 128, 256
    lo, hi = RANGE[fmt]
    codes = np.stack([np.roll(np.resize(np.arange(lo, hi), K), n) for n in range(N)])
    sb = np.resize(np.array([0x0001, 0x03FF, 0x0400, 0x2000, 0x3C00, 0x77FF, 0x8001, 0xBC00, 0x0000, 0x8000], dtype=np.uint16), (N, K // 32))
    blocks = synth.blocks_from_codes(fmt, sb, codes)
    w = qmm.dequant(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K).cpu().numpy()
    assert w.tobytes() == oracle.dequant(fmt, blocks, N, K).tobytes()


@pytest.mark.parametrize("fmt", [Q5, Q6])
@pytest.mark.parametrize("N,K", [(128, 256), (384, 512), (128, 8192), (2176, 1280), (512, 4096)])
def test_gemv(qmm, oracle, fmt, N, K):
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=7 * N + K + fmt)
    x = synth.activations(96, N + K, K)
    y = qmm.gemv(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(x))
    y_ref, B = oracle.gemv(fmt, blocks, N, K, x)
    util.assert_within_tol(util.host_f64(y), y_ref, B, "gemv fmt=%d %dx%d" % (fmt, N, K))


@pytest.mark.parametrize("fmt", [Q5, Q6])
@pytest.mark.parametrize("force,two_kernels", [("8,1", False), ("8,4", False), ("16,2", False), ("8,4", True), ("8,16", False)])
def test_gemv_launch_geometries_and_static(qmm, oracle, fmt, force, two_kernels):
    qmm.debug_config("gemv_force", force)
    qmm.debug_config("gemv_no_cluster", "1" if two_kernels else None)
    N, K = 512, 4096
    blocks = synth.quantize(fmt, synth.weights(97, fmt, N, K))
    x = synth.activations(97, 7, K)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    y = qmm.gemv(fmt, packed, N, K, util.dev(x))
    y_ref, B = oracle.gemv(fmt, blocks, N, K, x)
    util.assert_within_tol(util.host_f64(y), y_ref, B, "gemv forced " + force)
    assert torch.equal(y, qmm.gemv(fmt, packed, N, K, util.dev(x)))
    qmm.debug_config(None)
    ys = torch.empty(N, dtype=torch.float16, device="cuda")
    qmm.gemv_static(fmt, packed, N, K, util.dev(x), ys)
    util.assert_within_tol(util.host_f64(ys), y_ref, B, "gemv_static")


@pytest.mark.parametrize("fmt", [Q5, Q6])
def test_integer_case_is_exact_and_one_hot_returns_columns(qmm, oracle, fmt):
    rng = np.random.default_rng(5 + fmt)
    N, K, M = 256, 512, 96
    lo, hi = RANGE[fmt]
    codes = np.where(rng.random((N, K)) < 0.08, rng.integers(lo, hi, size=(N, K)), 0)
    blocks = synth.blocks_from_codes(fmt, np.full((N, K // 32), 0x3C00, dtype=np.uint16), codes)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    xi = rng.integers(-2, 3, size=K)
    ref = codes.astype(np.int64) @ xi.astype(np.int64)
    assert np.abs(ref).max() < 2048
    assert np.array_equal(util.host_f64(qmm.gemv(fmt, packed, N, K, util.dev(xi.astype(np.float16)))), ref.astype(np.float64))
    Xi = rng.integers(-2, 3, size=(M, K))
    refm = Xi.astype(np.int64) @ codes.T.astype(np.int64)
    assert np.abs(refm).max() < 2048
    assert np.array_equal(util.host_f64(qmm.gemm(fmt, packed, N, K, util.dev(Xi.astype(np.float16)))), refm.astype(np.float64))
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=44 + fmt, special_scales=False)
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    W = oracle.dequant(fmt, blocks, N, K)
    for k in (0, 1, 7, 8, 31, 32, 63, 64, 255, 511):
        e = np.zeros(K, dtype=np.float16)
        e[k] = 1
        assert np.array_equal(qmm.gemv(fmt, packed, N, K, util.dev(e)).cpu().numpy(), W[:, k].astype(np.float16)), k


@pytest.mark.parametrize("fmt", [Q5, Q6])
@pytest.mark.parametrize("M,N,K", [(128, 128, 256), (1, 128, 512), (77, 384, 768), (200, 640, 512), (64, 128, 4096), (700, 6400, 512),
                                   (300, 384, 1024), (2048, 2432, 512)])
def test_gemm(qmm, oracle, fmt, M, N, K):
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=M + 3 * N + K + fmt, special_scales="no_subnormal")
    X = synth.activations(98, M + N + K, M, K)
    ws = torch.zeros(qmm.gemm_workspace_bytes(fmt, M, N, K), dtype=torch.uint8, device="cuda")
    Y = qmm.gemm(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(X), ws=ws)
    qmm.status_check(ws)
    rows = np.arange(M) if M <= 700 else np.unique(np.concatenate([[0, M - 1], np.arange(1792, M, 5)]))
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X[rows])
    util.assert_within_tol(util.host_f64(Y)[rows], Y_ref, B, "gemm fmt=%d M=%d N=%d K=%d" % (fmt, M, N, K))


@pytest.mark.parametrize("fmt", [Q5, Q6])
def test_prefill_and_decode_shapes_of_the_configs(qmm, oracle, fmt):
    c = synth.CFG3
    _, N, K = c["shapes"][0]
    blocks = synth.quantize(fmt, synth.weights(c["seed"], 0, N, K))
    packed = qmm.pack(fmt, util.dev(blocks), N, K)
    M = 512
    X = synth.activations(c["seed"], 10 + M, M, K)
    Y = qmm.gemm(fmt, packed, N, K, util.dev(X))
    rows = np.array([0, 100, 255, 256, 511])
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X[rows])
    util.assert_within_tol(util.host_f64(Y)[rows], Y_ref, B, "cfg3-shaped gemm fmt=%d" % fmt)
    y = qmm.gemv(fmt, packed, N, K, util.dev(X[3]))
    util.assert_within_tol(util.host_f64(y), *oracle.gemv(fmt, blocks, N, K, X[3]), "cfg3-shaped gemv fmt=%d" % fmt)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    qmm.packed_check(fmt, packed, N, K, ws)
    qmm.status_check(ws)
    qmm.packed_check(fmt, util.dev(blocks), N, K, ws)                 # canonical bytes are not a packed buffer
    with pytest.raises(qmm.QmmError):
        qmm.status_check(ws)


@pytest.mark.parametrize("fmt", [Q5, Q6])
def test_gemv_batch(qmm, oracle, fmt):
    shapes = [(128, 256), (384, 1024), (128, 8192), (640, 512), (2176, 1280), (2048, 2048)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        blocks = synth.quantize(fmt, synth.weights(94, 10 * fmt + i, N, K))
        x = synth.activations(94, 100 + i, K)
        y = torch.full((N,), 9.0, dtype=torch.float16, device="cuda")
        probs.append((qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(x), y))
        refs.append(oracle.gemv(fmt, blocks, N, K, x))
    qmm.gemv_batch(fmt, qmm.gemv_batch_problems(probs))
    torch.cuda.synchronize()
    for (p, N, K, x, y), (y_ref, B) in zip(probs, refs):
        util.assert_within_tol(util.host_f64(y), y_ref, B, "batch fmt=%d %dx%d" % (fmt, N, K))


def test_calls_not_built_for_these_formats_say_so(qmm):
    L = qmm.lib()
    w = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    y = torch.zeros(128, dtype=torch.float16, device="cuda")
    for fmt in (Q5, Q6):
        assert L.qmm_gemv_gate_up(fmt, w.data_ptr(), w.data_ptr(), 128, 256, x.data_ptr(), y.data_ptr(), None) == 5
        st = (qmm.ChainStage * 1)(qmm.ChainStage(0, -1, 0, x.data_ptr(), w.data_ptr(), None, 128, 256, None))
        assert L.qmm_chain_plan_bytes(fmt, st, 1) == 0 and "not built" in qmm.last_error()
        a = qmm.moe_args(fmt, 4, 256, 256, 8, 2, x, x, w, w, w, y)
        assert L.qmm_moe_workspace_bytes(a) == 0
