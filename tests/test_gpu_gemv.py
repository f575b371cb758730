"""GPU parity: qmm_pack / qmm_dequant / qmm_gemv against the CPU oracle.

Weights must dequantise bit-exactly; every GEMV output must satisfy
|y_gpu - y_ref| <= 2e-3 * sum_k |w x| + 1e-5 with y_ref, sum|w x| from the
oracle's fp64 accumulation.
"""
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


def packed_from(qmm, fmt, blocks, N, K):
    return qmm.pack(fmt, util.dev(blocks), N, K)


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("N,K", [(128, 256), (384, 768), (256, 2048)])
def test_dequant_bit_exact(qmm, oracle, fmt, N, K):
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=N + K + fmt)
    w_gpu = qmm.dequant(fmt, packed_from(qmm, fmt, blocks, N, K), N, K).cpu().numpy()
    w_ref = oracle.dequant(fmt, blocks, N, K)
    assert w_gpu.tobytes() == w_ref.tobytes()


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_dequant_every_code_and_scale_class(qmm, oracle, fmt):
    # each row repeats every code value; scales sweep normal, subnormal, negative, zero
    N, K = 128, 256
    lo, hi = (-8, 8) if fmt == Q4 else (-128, 128)
    codes = np.resize(np.arange(lo, hi), (N, K))
    codes = np.roll(codes, np.arange(N)[:, None] % 7, axis=1) if False else codes
    sb = np.resize(np.array([0x0001, 0x03FF, 0x0400, 0x2000, 0x3C00, 0x7BFF, 0x8001, 0xBC00, 0x0000, 0x8000],
                            dtype=np.uint16), (N, K // 32))
    blocks = synth.blocks_from_codes(fmt, sb, codes)
    w_gpu = qmm.dequant(fmt, packed_from(qmm, fmt, blocks, N, K), N, K).cpu().numpy()
    assert w_gpu.tobytes() == oracle.dequant(fmt, blocks, N, K).tobytes()


def run_gemv(qmm, oracle, fmt, blocks, N, K, x, what):
    y = qmm.gemv(fmt, packed_from(qmm, fmt, blocks, N, K), N, K, util.dev(x))
    torch.cuda.synchronize()
    y_ref, B = oracle.gemv(fmt, blocks, N, K, x)
    return util.assert_within_tol(util.host_f64(y), y_ref, B, what), y


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("N,K", [(128, 256), (384, 512), (128, 8192), (2176, 1280)])
def test_gemv_small_shapes(qmm, oracle, fmt, N, K):
    blocks, _, _ = util.random_blocks(synth, fmt, N, K, seed=7 * N + K + fmt)
    x = synth.activations(90, N + K, K)
    run_gemv(qmm, oracle, fmt, blocks, N, K, x, "gemv %dx%d fmt %d" % (N, K, fmt))


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("force", ["8,1", "8,2", "8,8", "16,1", "16,2", "16,4", "8,16"])
@pytest.mark.parametrize("two_kernels", [False, True])
def test_gemv_every_launch_geometry(qmm, oracle, fmt, force, two_kernels):
    # the same product through each block size and K split; a K split over up to 8 blocks adds the
    # blocks' sums through the shared memory of a thread-block cluster, otherwise (more splits, or
    # on request) through fp32 partials in the workspace and a second kernel -- both in a fixed order
    qmm.debug_config("gemv_force", force)
    qmm.debug_config("gemv_no_cluster", "1" if two_kernels else None)
    N, K = 512, 4096
    blocks = synth.quantize(fmt, synth.weights(91, fmt, N, K))
    x = synth.activations(91, 7, K)
    _, y = run_gemv(qmm, oracle, fmt, blocks, N, K, x, "gemv forced " + force)
    _, y2 = run_gemv(qmm, oracle, fmt, blocks, N, K, x, "gemv forced " + force)
    assert torch.equal(y, y2)                              # same bits on every call


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemv_integer_case_is_exact(qmm, fmt):
    # unit scales and small integer activations: an integer matrix-vector product, exact in fp16 output
    rng = np.random.default_rng(5 + fmt)
    N, K = 256, 512
    lo, hi = (-8, 8) if fmt == Q4 else (-127, 128)
    codes = rng.integers(lo, hi, size=(N, K))
    keep = rng.random((N, K)) < (0.25 if fmt == Q4 else 0.01)       # keep |y| < 2048
    codes = np.where(keep, codes, 0)
    xi = rng.integers(-2, 3, size=K)
    ref = codes.astype(np.int64) @ xi.astype(np.int64)
    assert np.abs(ref).max() < 2048
    blocks = synth.blocks_from_codes(fmt, np.full((N, K // 32), 0x3C00, dtype=np.uint16), codes)
    y = qmm.gemv(fmt, packed_from(qmm, fmt, blocks, N, K), N, K, util.dev(xi.astype(np.float16)))
    assert np.array_equal(util.host_f64(y), ref.astype(np.float64))


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemv_one_hot_returns_column_and_zero_codes_give_zero(qmm, oracle, fmt):
    N, K = 128, 512
    blocks, codes, sb = util.random_blocks(synth, fmt, N, K, seed=33 + fmt, special_scales=False)
    packed = packed_from(qmm, fmt, blocks, N, K)
    W = oracle.dequant(fmt, blocks, N, K)
    for k in (0, 1, 31, 32, 63, 64, 255, 511):
        e = np.zeros(K, dtype=np.float16)
        e[k] = 1
        y = qmm.gemv(fmt, packed, N, K, util.dev(e)).cpu().numpy()
        assert np.array_equal(y, W[:, k].astype(np.float16)), k
    z = synth.blocks_from_codes(fmt, sb, np.zeros_like(codes))
    y = qmm.gemv(fmt, packed_from(qmm, fmt, z, N, K), N, K, util.dev(synth.activations(1, 1, K)))
    assert not y.cpu().numpy().any()


@pytest.mark.parametrize("two_kernels", [False, True])
def test_gemv_is_deterministic_and_stays_in_bounds(qmm, two_kernels):
    qmm.debug_config("gemv_force", "8,4")
    qmm.debug_config("gemv_no_cluster", "1" if two_kernels else None)
    N, K = 256, 2048
    blocks = synth.quantize(Q4, synth.weights(92, 0, N, K))
    packed = packed_from(qmm, Q4, blocks, N, K)
    x = util.dev(synth.activations(92, 1, K))
    guard = 64
    buf = torch.full((N + 2 * guard,), 7.0, dtype=torch.float16, device="cuda")
    need = qmm.gemv_workspace_bytes(Q4, N, K)
    assert need == (4 * N * 4 if two_kernels else 0)       # the cluster form adds its sums in shared memory
    wsbuf = torch.full((need + 512,), 0x5A, dtype=torch.uint8, device="cuda")
    y = buf[guard:guard + N]
    qmm.gemv(Q4, packed, N, K, x, y=y, ws=wsbuf[256:256 + need])
    first = y.clone()
    for _ in range(5):
        qmm.gemv(Q4, packed, N, K, x, y=y, ws=wsbuf[256:256 + need])
        assert torch.equal(first, y)
    assert torch.all(buf[:guard] == 7.0) and torch.all(buf[guard + N:] == 7.0)
    assert torch.all(wsbuf[:256] == 0x5A) and torch.all(wsbuf[256 + need:] == 0x5A)


def test_cfg0_q4_gemv_full_size(qmm, oracle):
    c = synth.CFG0
    blocks = synth.quantize(c["fmt"], synth.weights(c["seed"], 0, c["N"], c["K"]))
    x = synth.activations(c["seed"], 1, c["K"])
    run_gemv(qmm, oracle, c["fmt"], blocks, c["N"], c["K"], x, "cfg0")


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_cfg1_one_layer_full_size_unfused_and_fused(qmm, oracle, fmt):
    layer = 3
    acts = synth.cfg1_layer_acts(layer)
    packed, refs = {}, {}
    for name, N, K, act, w in synth.cfg1_layer_weights(layer):
        blocks = synth.quantize(fmt, w)
        packed[name] = packed_from(qmm, fmt, blocks, N, K)
        y = qmm.gemv(fmt, packed[name], N, K, util.dev(acts[act]))
        refs[name] = oracle.gemv(fmt, blocks, N, K, acts[act])
        util.assert_within_tol(util.host_f64(y), refs[name][0], refs[name][1], "cfg1 %s" % name)
    # fused launches: packed buffers with the same K concatenate into one matrix
    for names, act in ((("q", "k", "v"), "x_attn"), (("gate", "up"), "x_ffn")):
        Ntot = sum(packed[n].numel() for n in names) // (qmm.packed_bytes(fmt, 128, 2048) // 128)
        y = qmm.gemv(fmt, torch.cat([packed[n] for n in names]), Ntot, 2048, util.dev(acts[act]))
        y_ref = np.concatenate([refs[n][0] for n in names])
        B = np.concatenate([refs[n][1] for n in names])
        util.assert_within_tol(util.host_f64(y), y_ref, B, "cfg1 fused " + "+".join(names))


def check_gate_up(qmm, oracle, fmt, gate_blocks, up_blocks, N, K, x, what):
    """h = silu(Wg x) * (Wu x): both products held to the per-product tolerance through the bound
    it implies for h (|silu'| <= 1.1), plus the fp16 rounding of h."""
    h = qmm.gemv_gate_up(fmt, packed_from(qmm, fmt, gate_blocks, N, K), packed_from(qmm, fmt, up_blocks, N, K), N, K, util.dev(x))
    G, BG = oracle.gemv(fmt, gate_blocks, N, K, x)
    U, BU = oracle.gemv(fmt, up_blocks, N, K, x)
    tolG, tolU = util.RTOL_SUMABS * BG + util.ATOL, util.RTOL_SUMABS * BU + util.ATOL
    sG = oracle.silu(G)
    h_ref = sG * U
    bound = 1.1 * tolG * np.abs(U) + np.abs(sG) * tolU + 1.1 * tolG * tolU + 2.0**-11 * np.abs(h_ref)
    worst = float(np.max(np.abs(util.host_f64(h) - h_ref) / bound))
    assert worst <= 1.0, "%s: %.3f of bound" % (what, worst)
    return worst


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("N,K", [(128, 256), (384, 1280), (2176, 512)])
def test_gemv_gate_up_small_shapes(qmm, oracle, fmt, N, K):
    # (weights of the configs' distribution: with arbitrary scales silu(g) * u leaves the fp16 range)
    gate = synth.quantize(fmt, synth.weights(92, N + K, N, K))
    up = synth.quantize(fmt, synth.weights(93, N + K, N, K))
    x = synth.activations(91, N + K, K)
    check_gate_up(qmm, oracle, fmt, gate, up, N, K, x, "gate_up %dx%d fmt %d" % (N, K, fmt))


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemv_gate_up_cfg1_layer_full_size(qmm, oracle, fmt):
    layer = 5
    acts = synth.cfg1_layer_acts(layer)
    w = {name: (N, K, synth.quantize(fmt, wt)) for name, N, K, act, wt in synth.cfg1_layer_weights(layer) if name in ("gate", "up")}
    N, K, gate = w["gate"]
    check_gate_up(qmm, oracle, fmt, gate, w["up"][2], N, K, acts["x_ffn"], "cfg1 gate_up fused with SiLU*mul")


def test_gemv_gate_up_argument_checks(qmm):
    a = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    h = torch.zeros(128, dtype=torch.float16, device="cuda")
    L = qmm.lib()
    assert L.qmm_gemv_gate_up(Q4, a.data_ptr(), a.data_ptr(), 128, 200, x.data_ptr(), h.data_ptr(), None) in (2, 5)   # K % 256
    assert L.qmm_gemv_gate_up(Q4, a.data_ptr() + 8, a.data_ptr(), 128, 256, x.data_ptr(), h.data_ptr(), None) == 3    # alignment
    assert L.qmm_gemv_gate_up(Q4, a.data_ptr(), None, 128, 256, x.data_ptr(), h.data_ptr(), None) == 1                # null
    assert "null" in qmm.last_error()


def test_cfg2_q8_lm_head_full_size(qmm, oracle):
    c = synth.CFG2
    blocks = synth.quantize(c["fmt"], synth.weights(c["seed"], 0, c["N"], c["K"]))
    x = synth.activations(c["seed"], 1, c["K"])
    run_gemv(qmm, oracle, c["fmt"], blocks, c["N"], c["K"], x, "cfg2")


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemv_batch_mixed_shapes(qmm, oracle, fmt):
    # one launch over problems that differ in N and K; each result held to the GEMV tolerance
    shapes = [(128, 256), (384, 1024), (128, 8192), (640, 512), (256, 2048), (128, 256), (2176, 1280)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        blocks = synth.quantize(fmt, synth.weights(95, 10 * fmt + i, N, K))
        x = synth.activations(95, 100 + i, K)
        y = torch.full((N,), 9.0, dtype=torch.float16, device="cuda")
        probs.append((packed_from(qmm, fmt, blocks, N, K), N, K, util.dev(x), y))
        refs.append(oracle.gemv(fmt, blocks, N, K, x))
    arr = qmm.gemv_batch_problems(probs)
    qmm.gemv_batch(fmt, arr)
    torch.cuda.synchronize()
    for (p, N, K, x, y), (y_ref, B) in zip(probs, refs):
        util.assert_within_tol(util.host_f64(y), y_ref, B, "batch %dx%d" % (N, K))
    first = [p[4].clone() for p in probs]
    qmm.gemv_batch(fmt, arr)                                # deterministic
    for f, p in zip(first, probs):
        assert torch.equal(f, p[4])


def test_gemv_batch_argument_checks(qmm):
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    y = torch.zeros(128, dtype=torch.float16, device="cuda")
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    L = qmm.lib()
    good = qmm.gemv_batch_problems([(buf, 128, 256, x, y)])
    assert L.qmm_gemv_batch(4, good, 0, None) == 0
    assert L.qmm_gemv_batch(4, good, -1, None) == 1
    assert L.qmm_gemv_batch(4, None, 1, None) == 1
    bad = (qmm.GemvProblem * 1)(qmm.GemvProblem(buf.data_ptr() + 8, x.data_ptr(), y.data_ptr(), 128, 256))
    assert L.qmm_gemv_batch(4, bad, 1, None) == 3
    bad = (qmm.GemvProblem * 1)(qmm.GemvProblem(buf.data_ptr(), x.data_ptr(), y.data_ptr(), 100, 256))
    assert L.qmm_gemv_batch(4, bad, 1, None) == 5


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_cfg1_two_layers_full_size_in_one_batch(qmm, oracle, fmt):
    probs, refs = [], []
    for layer in (0, 15):
        acts = synth.cfg1_layer_acts(layer)
        for name, N, K, act, w in synth.cfg1_layer_weights(layer):
            blocks = synth.quantize(fmt, w)
            y = torch.empty(N, dtype=torch.float16, device="cuda")
            probs.append((packed_from(qmm, fmt, blocks, N, K), N, K, util.dev(acts[act]), y))
            refs.append((name, oracle.gemv(fmt, blocks, N, K, acts[act])))
    qmm.gemv_batch(fmt, qmm.gemv_batch_problems(probs))
    torch.cuda.synchronize()
    for (p, N, K, x, y), (name, (y_ref, B)) in zip(probs, refs):
        util.assert_within_tol(util.host_f64(y), y_ref, B, "cfg1 batch %s" % name)


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_cfg1_whole_stack_in_one_batch_as_benchmarked(qmm, oracle, fmt):
    """The launch the benchmark times: all 112 matrices of the 16-layer stack as one qmm_gemv_batch
    call, every output of every problem held to the GEMV tolerance against the oracle."""
    from concurrent.futures import ThreadPoolExecutor
    layers = synth.CFG1["layers"]

    def host_layer(layer):
        return [(name, N, K, act, synth.quantize(fmt, w)) for name, N, K, act, w in synth.cfg1_layer_weights(layer)]

    with ThreadPoolExecutor(max_workers=8) as ex:
        host = list(ex.map(host_layer, range(layers)))
    probs, meta = [], []
    for layer in range(layers):
        acts = synth.cfg1_layer_acts(layer)
        for name, N, K, act, blocks in host[layer]:
            y = torch.full((N,), 9.0, dtype=torch.float16, device="cuda")
            probs.append((packed_from(qmm, fmt, blocks, N, K), N, K, util.dev(acts[act]), y))
            meta.append((layer, name, N, K, blocks, acts[act]))
    assert len(probs) == 112
    qmm.gemv_batch(fmt, qmm.gemv_batch_problems(probs))
    torch.cuda.synchronize()
    worst = 0.0
    for (p, N, K, x, y), (layer, name, _, _, blocks, xh) in zip(probs, meta):
        y_ref, B = oracle.gemv(fmt, blocks, N, K, xh)
        worst = max(worst, util.assert_within_tol(util.host_f64(y), y_ref, B, "cfg1 stack, layer %d %s" % (layer, name)))
    assert worst > 0


def test_row_sharded_gemv_on_one_rank_is_the_plain_product(qmm, oracle):
    """Without a process group the sharded operator holds every row and no collective runs (the
    two-rank form is tested with gloo on CPU)."""
    from paper_2607_00501_b200 import sharded
    N, K = 640, 1024
    blocks = synth.quantize(Q8, synth.weights(99, 0, N, K))
    x = synth.activations(99, 1, K)
    op = sharded.RowShardedGemv(Q8, blocks, N, K)
    assert (op.r0, op.r1, op.world) == (0, N, 1)
    y = op(util.dev(x))
    y_ref, B = oracle.gemv(Q8, blocks, N, K, x)
    util.assert_within_tol(util.host_f64(y), y_ref, B, "sharded, one rank")


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_gemv_batch_of_many_short_products(qmm, oracle, fmt):
    """Enough short-K products for every warp of the grid to own units of its own (the one-warp-per-unit
    form of the batched kernel): 100 products of mixed shapes, every output against the oracle."""
    shapes = [(3072, 1024), (512, 256), (1024, 512), (640, 1024 if fmt == Q4 else 512)]
    probs, refs = [], []
    for i in range(100):
        N, K = shapes[i % len(shapes)]
        blocks = synth.quantize(fmt, synth.weights(120, 1000 * fmt + i, N, K))
        x = synth.activations(121, i, K)
        y = torch.full((N,), 9.0, dtype=torch.float16, device="cuda")
        probs.append((packed_from(qmm, fmt, blocks, N, K), N, K, util.dev(x), y))
        refs.append(oracle.gemv(fmt, blocks, N, K, x))
    arr = qmm.gemv_batch_problems(probs)
    qmm.gemv_batch(fmt, arr)
    torch.cuda.synchronize()
    for (p, N, K, x, y), (y_ref, B) in zip(probs, refs):
        util.assert_within_tol(util.host_f64(y), y_ref, B, "short batch %dx%d" % (N, K))
    first = [p[4].clone() for p in probs]
    qmm.gemv_batch(fmt, arr)
    torch.cuda.synchronize()
    for f, p in zip(first, probs):
        assert torch.equal(f, p[4])
