"""GPU parity on seeded random shapes: every supported (N % 128 == 0, K % 256 == 0, any M / T)
combination goes through the same tolerance as the fixed cases -- shapes nobody picked by hand."""
import numpy as np
import pytest
import torch

from paper_2607_00501_b200 import synth
from tests import util
from tests.test_gpu_moe import Layer, check_stages, run_layer

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qmm():
    from paper_2607_00501_b200 import qmm as _qmm
    assert torch.cuda.is_available()
    _qmm.lib()
    return _qmm



@pytest.mark.parametrize("case", range(12))
def test_random_gemv_shapes(qmm, oracle, case):
    rng = np.random.default_rng([811, case])
    fmt = int(rng.choice([4, 8]))
    N, K = int(rng.integers(1, 24)) * 128, int(rng.integers(1, 33)) * 256
    blocks = synth.quantize(fmt, synth.weights(812, case, N, K))
    x = synth.activations(813, case, K)
    y = qmm.gemv(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(x))
    y_ref, B = oracle.gemv(fmt, blocks, N, K, x)
    util.assert_within_tol(util.host_f64(y), y_ref, B, "gemv fmt=%d N=%d K=%d" % (fmt, N, K))


@pytest.mark.parametrize("case", range(16))
def test_random_gemm_shapes(qmm, oracle, case):
    rng = np.random.default_rng([821, case])
    fmt = int(rng.choice([4, 8]))
    M, N, K = int(rng.integers(1, 700)), int(rng.integers(1, 20)) * 128, int(rng.integers(1, 17)) * 256
    blocks = synth.quantize(fmt, synth.weights(822, case, N, K))
    X = synth.activations(823, case, M, K)
    ws = torch.zeros(qmm.gemm_workspace_bytes(fmt, M, N, K), dtype=torch.uint8, device="cuda")
    Y = qmm.gemm(fmt, qmm.pack(fmt, util.dev(blocks), N, K), N, K, util.dev(X), ws=ws)
    qmm.status_check(ws)
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X)
    util.assert_within_tol(util.host_f64(Y), Y_ref, B, "gemm fmt=%d M=%d N=%d K=%d" % (fmt, M, N, K))


@pytest.mark.parametrize("case", range(16))
def test_random_few_token_products(qmm, oracle, case):
    """M <= 8 through qmm_gemm (even cases) and through qmm_gemm_batch over a random list (odd cases), all
    four formats, special scales, padded rows with guard values.  (One-off runs of ~8 000 such cases found
    no failure.)"""
    rng = np.random.default_rng([851, case])
    fmt, M = int(rng.choice([4, 5, 6, 8])), int(rng.integers(1, 9))
    probs, refs, bufs = [], [], []
    for i in range(1 if case % 2 == 0 else int(rng.integers(2, 10))):
        N, K = 128 * int(rng.integers(1, 30)), 256 * int(rng.integers(1, 20))
        blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=int(rng.integers(1 << 30)), special_scales=bool(rng.random() < 0.5))
        X = synth.activations(852, 100 * case + i, M, K)
        Xb = torch.full((M, K + 8 * int(rng.integers(0, 3))), 2.0, dtype=torch.float16, device="cuda")
        Xb[:, :K] = util.dev(X)
        Yb = torch.full((M, N + 8 * int(rng.integers(0, 3))), 3.0, dtype=torch.float16, device="cuda")
        probs.append((qmm.pack(fmt, util.dev(blocks), N, K), N, K, Xb[:, :K], Yb[:, :N]))
        refs.append(oracle.gemm(fmt, blocks, N, K, X))
        bufs.append(Yb)
    if case % 2 == 0:
        p, N, K, X, Y = probs[0]
        qmm.gemm(fmt, p, N, K, X, Y=Y)
    else:
        qmm.gemm_batch(fmt, qmm.gemm_batch_problems(probs))
    torch.cuda.synchronize()
    for (p, N, K, X, Y), (Y_ref, B), Yb in zip(probs, refs, bufs):
        util.assert_within_tol(util.host_f64(Y), Y_ref, B, "few tokens fmt=%d M=%d N=%d K=%d" % (fmt, M, N, K))
        assert bool(torch.all(Yb[:, N:] == 3.0))


@pytest.mark.parametrize("case", range(10))
def test_random_many_tile_gemm_plans_agree(qmm, oracle, case):
    """Shapes with more output tiles than SMs: the plan gives every block whole tiles and treats the
    last, partly filled round in one of three ways (whole tiles, half tiles, shares of the K range with
    partial sums).  Whatever it picks must agree with the whole-tile plan -- bit for bit unless partial
    sums are added in another order -- be the same on every call, and pass the oracle on sampled rows."""
    rng = np.random.default_rng([841, case])
    fmt = int(rng.choice([4, 8]))
    while True:
        M, N, K = int(rng.integers(600, 4600)), int(rng.integers(4, 40)) * 128, int(rng.integers(1, 33)) * 256
        if (N // 128) * ((M + 255) // 256) > 148:
            break
    qmm.debug_config(None)
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=842 + case, special_scales=False)
    X = synth.activations(843, case, M, K)
    packed, Xd = qmm.pack(fmt, util.dev(blocks), N, K), util.dev(X)
    need = qmm.gemm_workspace_bytes(fmt, M, N, K)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    Y = qmm.gemm(fmt, packed, N, K, Xd, ws=ws)
    qmm.status_check(ws)
    assert torch.equal(Y, qmm.gemm(fmt, packed, N, K, Xd, ws=ws))
    rows = np.unique(np.concatenate([[0, M - 1, M - 129 if M > 129 else 0], rng.integers(0, M, size=5)]))
    Y_ref, B = oracle.gemm(fmt, blocks, N, K, X[rows])
    util.assert_within_tol(util.host_f64(Y)[rows], Y_ref, B, "gemm fmt=%d M=%d N=%d K=%d" % (fmt, M, N, K))
    qmm.debug_config("gemm_no_tail_cut", "1")
    need_whole = qmm.gemm_workspace_bytes(fmt, M, N, K)
    ws2 = torch.zeros(need_whole, dtype=torch.uint8, device="cuda")
    Y2 = qmm.gemm(fmt, packed, N, K, Xd, ws=ws2)
    qmm.status_check(ws2)
    if need == need_whole:                                                        # no partial sums: same arithmetic
        assert torch.equal(Y, Y2)
    else:
        assert float((Y.float() - Y2.float()).abs().max()) <= 2e-3 * float(Y2.float().abs().max())


@pytest.mark.parametrize("case", range(6))
def test_random_moe_layers(qmm, oracle, case):
    rng = np.random.default_rng([831, case])
    fmt = int(rng.choice([4, 8]))
    E = int(rng.choice([4, 8, 32, 128]))
    topk = int(rng.integers(1, min(E, 8) + 1))
    T, H, I = int(rng.integers(1, 300)), int(rng.integers(1, 5)) * 256, int(rng.integers(1, 5)) * 256
    L = Layer(qmm, fmt, 832 + case, E, H, I)
    X = synth.activations(833, case, T, H)
    logits = synth.logits(834, case, T, E)
    res = run_layer(qmm, L, logits, X, topk)
    experts = sorted({int(e) for e in rng.integers(0, E, size=min(E, 6))})
    check_stages(oracle, L, res, logits, X, topk, experts=experts, rows_per_expert=8, tokens=list(range(min(T, 5))))
