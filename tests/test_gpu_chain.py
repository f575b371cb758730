"""GPU parity: qmm_chain_* (a list of decode products, dependent or not, as one launch) against the
CPU oracle.  A stage that reads an earlier stage is checked against the oracle applied to the GPU's
own fp16 output of that stage, so every product is held to |y - y_ref| <= 2e-3 * sum|w x| + 1e-5."""
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


def build_chain(qmm, fmt, spec, seed, unit_variance=False):
    """spec: list of (op, N, K, source) with source = None (own caller vector) or (stage, offset).
    Returns (chain, host data per stage)."""
    stages, host = [], []
    for i, (op, N, K, src) in enumerate(spec):
        h = {"op": op, "N": N, "K": K, "src": src}
        std = K ** -0.5 if unit_variance else 0.02                    # (unit variance: magnitudes survive long chains)
        h["w"] = synth.quantize(fmt, synth.weights(seed, 10 * i, N, K, std=std))
        d = {"op": op, "N": N, "K": K, "packed": qmm.pack(fmt, util.dev(h["w"]), N, K),
             "y": torch.full((N,), 7.0, dtype=torch.float16, device="cuda")}
        if op == qmm.CHAIN_GATE_UP_SILU:
            h["w_up"] = synth.quantize(fmt, synth.weights(seed, 10 * i + 1, N, K, std=std))
            d["packed_up"] = qmm.pack(fmt, util.dev(h["w_up"]), N, K)
        if src is None:
            h["x"] = synth.activations(seed, 1000 + i, K)
            d["x"] = util.dev(h["x"])
        else:
            d["x_stage"], d["x_offset"] = src
        stages.append(d)
        host.append(h)
    return qmm.Chain(fmt, stages), stages, host


def check_chain(qmm, oracle, fmt, stages, host, what):
    ys = [s["y"].cpu().numpy() for s in stages]
    worst = 0.0
    for i, h in enumerate(host):
        x = h["x"] if h["src"] is None else ys[h["src"][0]][h["src"][1]:h["src"][1] + h["K"]]
        got = ys[i].astype(np.float64)
        assert np.all(np.isfinite(got)), "%s stage %d" % (what, i)
        if h["op"] == qmm.CHAIN_LINEAR:
            y_ref, B = oracle.gemv(fmt, h["w"], h["N"], h["K"], x)
            worst = max(worst, util.assert_within_tol(got, y_ref, B, "%s stage %d" % (what, i)))
        else:
            G, BG = oracle.gemv(fmt, h["w"], h["N"], h["K"], x)
            U, BU = oracle.gemv(fmt, h["w_up"], h["N"], h["K"], x)
            tolG, tolU = util.RTOL_SUMABS * BG + util.ATOL, util.RTOL_SUMABS * BU + util.ATOL
            sG = oracle.silu(G)
            h_ref = sG * U
            bound = 1.1 * tolG * np.abs(U) + np.abs(sG) * tolU + 1.1 * tolG * tolU + 2.0**-11 * np.abs(h_ref)
            w = float(np.max(np.abs(got - h_ref) / bound))
            assert w <= 1.0, "%s stage %d (gate/up): %.3f of bound" % (what, i, w)
            worst = max(worst, w)
    return worst


LIN, GU = 0, 1


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_chain_of_dependent_stages_small(qmm, oracle, fmt):
    spec = [(LIN, 512, 256, None), (LIN, 768, 512, (0, 0)), (GU, 256, 768, (1, 0)), (LIN, 128, 256, (2, 0)),
            (LIN, 256, 256, (1, 256)), (LIN, 384, 256, None), (LIN, 128, 1280, (1, 0) if False else None)]
    chain, stages, host = build_chain(qmm, fmt, spec, 900 + fmt)
    chain.run()
    qmm.status_check(chain.ws)
    check_chain(qmm, oracle, fmt, stages, host, "small chain")
    first = [s["y"].clone() for s in stages]
    for _ in range(3):                                     # every launch takes a new tag; same bits every time
        for s in stages:
            s["y"].fill_(3.0)
        chain.run()
        torch.cuda.synchronize()
        for a, s in zip(first, stages):
            assert torch.equal(a, s["y"])
    qmm.status_check(chain.ws)


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_chain_two_decoder_layers_full_size(qmm, oracle, fmt):
    """Two layers of the 1B-class decode stack as a dependent chain: q/k/v (one matrix) -> o on the first
    2048 outputs -> gate/up with SiLU*mul -> down -> next layer.  Small stages are cut along K."""
    spec = []
    for layer in range(2):
        base = 4 * layer
        spec += [(LIN, 3072, 2048, None if layer == 0 else (base - 1, 0)), (LIN, 2048, 2048, (base, 0)),
                 (GU, 8192, 2048, (base + 1, 0)), (LIN, 2048, 8192, (base + 2, 0))]
    chain, stages, host = build_chain(qmm, fmt, spec, 910 + fmt)
    chain.run()
    qmm.status_check(chain.ws)
    check_chain(qmm, oracle, fmt, stages, host, "two layers")
    again = [s["y"].clone() for s in stages]
    chain.run()
    torch.cuda.synchronize()
    for a, s in zip(again, stages):
        assert torch.equal(a, s["y"])


@pytest.mark.parametrize("fmt", [Q4, Q8])
def test_chain_of_independent_products_is_a_batch(qmm, oracle, fmt):
    shapes = [(128, 256), (384, 1024), (128, 8192), (640, 512), (256, 2048), (128, 256), (2176, 1280), (2048, 2048), (512, 2048)]
    spec = [(LIN, N, K, None) for N, K in shapes] + [(GU, 512, 1024, None)]
    chain, stages, host = build_chain(qmm, fmt, spec, 920 + fmt)
    chain.run()
    qmm.status_check(chain.ws)
    check_chain(qmm, oracle, fmt, stages, host, "independent")


@pytest.mark.parametrize("case", range(8))
def test_random_stage_graphs(qmm, oracle, case):
    """Seeded random lists of stages: random shapes and operators, each stage reading a caller vector or a
    random window of a random earlier stage -- levels of several stages, fan-out, K splits and whole
    units mixed -- every stage against the oracle on the GPU's own intermediates, twice (same bits)."""
    rng = np.random.default_rng([951, case])
    fmt = int(rng.choice([4, 8]))
    spec = []
    for i in range(int(rng.integers(3, 14))):
        op = GU if rng.random() < 0.25 else LIN
        N = int(rng.integers(1, 17)) * 128
        feasible = [j for j in range(i) if spec[j][1] >= 256]
        if feasible and rng.random() < 0.7:
            j = int(rng.choice(feasible))
            K = int(rng.integers(1, min(spec[j][1], 4096) // 256 + 1)) * 256
            off = int(rng.integers(0, (spec[j][1] - K) // 8 + 1)) * 8
            spec.append((op, N, K, (j, off)))
        else:
            spec.append((op, N, int(rng.integers(1, 17)) * 256, None))
    chain, stages, host = build_chain(qmm, fmt, spec, 960 + case, unit_variance=True)
    chain.run()
    qmm.status_check(chain.ws)
    check_chain(qmm, oracle, fmt, stages, host, "random graph %d" % case)
    first = [s["y"].clone() for s in stages]
    chain.run()
    torch.cuda.synchronize()
    for a, s in zip(first, stages):
        assert torch.equal(a, s["y"])


def test_chain_argument_checks(qmm):
    L = qmm.lib()
    w = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    ok = qmm.ChainStage(0, -1, 0, x.data_ptr(), w.data_ptr(), None, 128, 256, None)
    arr = (qmm.ChainStage * 2)(ok, qmm.ChainStage(0, 0, 0, None, w.data_ptr(), None, 128, 128 * 2, None))
    assert L.qmm_chain_plan_bytes(4, arr, 2) == 0 and "inside stage" in qmm.last_error()       # reads 256 of 128 outputs
    arr[1] = qmm.ChainStage(0, 1, 0, None, w.data_ptr(), None, 128, 256, None)
    assert L.qmm_chain_workspace_bytes(4, arr, 2) == 0 and "earlier stage" in qmm.last_error()
    arr[1] = qmm.ChainStage(1, -1, 0, x.data_ptr(), w.data_ptr(), None, 128, 256, None)
    assert L.qmm_chain_plan_bytes(4, arr, 2) == 0                                               # gate/up without W_up
    arr[1] = qmm.ChainStage(0, -1, 0, x.data_ptr(), w.data_ptr(), None, 100, 256, None)
    assert L.qmm_chain_plan_bytes(4, arr, 2) == 0
    assert L.qmm_chain_plan_bytes(4, arr, 1) > 0 and L.qmm_chain_workspace_bytes(4, arr, 1) > 0
    info = qmm.ChainInfo()
    assert L.qmm_chain_run(info, None) == 1                                                     # not built
