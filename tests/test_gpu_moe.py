"""GPU parity: qmm_moe / qmm_moe_route against the CPU oracle, stage by stage.

Routing indices, permutation and expert offsets must be bit-exact; routing
weights within 1e-6.  Each matrix product is held to the per-product bound
|err| <= 2e-3 * sum|w x| + 1e-5: the gate/up stage through the bound it
implies for silu(G)*U, the down stage against the oracle applied to the GPU's
own intermediate, the combine against the oracle applied to the GPU's own
expert outputs; an all-fp64 end-to-end reference guards against compensating
errors.
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


class Layer:
    """Expert weights of one MoE layer on host (canonical) and device (packed)."""

    def __init__(self, qmm, fmt, seed, E, H, I, blocks=None):
        self.fmt, self.E, self.H, self.I = fmt, E, H, I
        self.gate, self.up, self.down = blocks if blocks is not None else synth.moe_expert_weights(seed, fmt, E, H, I)
        self.p_gate = qmm.pack(fmt, util.dev(self.gate), E * I, H)
        self.p_up = qmm.pack(fmt, util.dev(self.up), E * I, H)
        self.p_down = qmm.pack(fmt, util.dev(self.down), E * H, I)
        self.gu_bytes = synth.canonical_bytes(fmt, I, H)
        self.dn_bytes = synth.canonical_bytes(fmt, H, I)

    def expert_blocks(self, which, e):
        arr, n = {"gate": (self.gate, self.gu_bytes), "up": (self.up, self.gu_bytes), "down": (self.down, self.dn_bytes)}[which]
        return arr[e * n:(e + 1) * n]


def run_layer(qmm, L, logits, X, topk, route_only=False):
    T = logits.shape[0]
    dev = "cuda"
    out = torch.full((T, L.H), 3.0, dtype=torch.float16, device=dev)
    o = dict(
        topk_idx=torch.full((T, topk), -1, dtype=torch.int32, device=dev),
        topk_w=torch.zeros((T, topk), dtype=torch.float32, device=dev),
        perm=torch.full((T * topk,), -1, dtype=torch.int32, device=dev),
        expert_offsets=torch.full((L.E + 1,), -1, dtype=torch.int32, device=dev),
        dbg_H=torch.zeros((T * topk, L.I), dtype=torch.float16, device=dev),
        dbg_D=torch.zeros((T * topk, L.H), dtype=torch.float16, device=dev),
    )
    lg, Xd = util.dev(logits), util.dev(X)
    args = qmm.moe_args(L.fmt, T, L.H, L.I, L.E, topk, lg, Xd, L.p_gate, L.p_up, L.p_down, out, **o)
    ws = torch.zeros(qmm.moe_workspace_bytes(args), dtype=torch.uint8, device=dev)
    (qmm.moe_route if route_only else qmm.moe)(args, ws)
    qmm.status_check(ws)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in o.items()}
    res["out"] = out.cpu().numpy()
    return res


def check_routing(oracle, res, logits, topk, E):
    idx_ref, p_ref = oracle.route(logits, topk)
    perm_ref, offs_ref = oracle.permute(idx_ref, E)
    assert np.array_equal(res["topk_idx"], idx_ref)
    assert np.array_equal(res["perm"], perm_ref)
    assert np.array_equal(res["expert_offsets"], offs_ref)
    assert np.max(np.abs(res["topk_w"].astype(np.float64) - p_ref)) <= 1e-6
    return idx_ref, p_ref, perm_ref, offs_ref


def check_stages(oracle, L, res, logits, X, topk, experts, rows_per_expert=None, tokens=None):
    """Stage-wise parity on the listed experts (all their rows, or a sample) and tokens."""
    fmt, H, I, E = L.fmt, L.H, L.I, L.E
    idx_ref, p_ref, perm_ref, offs_ref = check_routing(oracle, res, logits, topk, E)
    Hg = res["dbg_H"].astype(np.float64)
    Dg = res["dbg_D"].astype(np.float64)
    rng = np.random.default_rng(1)
    worst = {}
    for e in experts:
        r0, r1 = int(offs_ref[e]), int(offs_ref[e + 1])
        if r1 == r0:
            continue
        rows = np.arange(r0, r1)
        if rows_per_expert is not None and rows.size > rows_per_expert:
            rows = np.unique(np.concatenate([[r0, r1 - 1], rng.choice(rows, rows_per_expert - 2, replace=False)]))
        tok = perm_ref[rows] // topk
        Xe = X[tok]
        G, BG = oracle.gemm(fmt, L.expert_blocks("gate", e), I, H, Xe)
        U, BU = oracle.gemm(fmt, L.expert_blocks("up", e), I, H, Xe)
        tolG, tolU = util.RTOL_SUMABS * BG + util.ATOL, util.RTOL_SUMABS * BU + util.ATOL
        sG = oracle.silu(G)
        h_ref = sG * U
        bound = 1.1 * tolG * np.abs(U) + np.abs(sG) * tolU + 1.1 * tolG * tolU + 2.0**-11 * np.abs(h_ref)
        w = np.max(np.abs(Hg[rows] - h_ref) / bound)
        worst["H"] = max(worst.get("H", 0), w)
        assert w <= 1.0, "expert %d gate/up stage: %.3f of bound" % (e, w)
        # down product from the GPU's own intermediate
        D_ref, BD = oracle.gemm(fmt, L.expert_blocks("down", e), H, I, res["dbg_H"][rows])
        w = util.assert_within_tol(Dg[rows], D_ref, BD, "expert %d down stage" % e)
        worst["D"] = max(worst.get("D", 0), w)
    # combine from the GPU's own expert outputs
    T = logits.shape[0]
    inv = np.empty(T * topk, dtype=np.int64)
    inv[perm_ref] = np.arange(T * topk)
    toks = np.arange(T) if tokens is None else np.asarray(tokens)
    for t in toks:
        rows = inv[t * topk:(t + 1) * topk]
        terms = p_ref[t][:, None] * Dg[rows]
        ref, B = terms.sum(axis=0), np.abs(terms).sum(axis=0)
        w = util.assert_within_tol(res["out"][t].astype(np.float64), ref, B, "combine token %d" % t)
        worst["out"] = max(worst.get("out", 0), w)
    return worst


def check_end_to_end(oracle, L, res, logits, X, topk, tokens):
    """The layer output against the all-fp64 layer (no intermediate rounding), within the bound composed
    from the per-product tolerance of every stage (util.moe_composed_bound)."""
    tokens = np.asarray(tokens)
    ref = oracle.moe_tokens(L.fmt, logits, X, L.gate, L.up, L.down, L.H, L.I, L.E, topk, tokens)
    ref2, bound = util.moe_composed_bound(oracle, L.fmt, logits, X, L.gate, L.up, L.down, L.H, L.I, L.E, topk, tokens)
    assert np.allclose(ref, ref2, rtol=1e-10, atol=1e-12)
    err = np.abs(res["out"][tokens].astype(np.float64) - ref)
    worst = float(np.max(err / bound))
    assert worst <= 1.0, "end to end: %.3f of the composed bound" % worst
    # The composed bound is a worst case over every stage (each product's tolerance is relative to
    # sum|w x|, ~10x the result when signs cancel); an error that large would still mean a broken
    # layer, so the output is also held to 2 % of the token's largest component.
    scale = np.maximum(np.abs(ref).max(axis=1, keepdims=True), 1e-3)
    assert np.all(err <= 2e-2 * scale + 1e-4)
    return worst


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("T,E,topk,H,I", [(1, 8, 2, 256, 256), (5, 8, 2, 256, 256), (4, 128, 8, 256, 256),
                                          (5, 128, 8, 512, 256), (37, 16, 4, 512, 256), (200, 8, 2, 256, 512),
                                          (64, 32, 8, 256, 256), (400, 4, 2, 256, 256)])
def test_moe_small_layers_every_row(qmm, oracle, fmt, T, E, topk, H, I):
    L = Layer(qmm, fmt, 500 + T + E, E, H, I)
    X = synth.activations(501, T, T, H)
    logits = synth.logits(502, T + E, T, E)
    if T >= 5:
        logits[3, 1] = logits[3, 0]                      # a tie inside one token's logits
    res = run_layer(qmm, L, logits, X, topk)
    check_stages(oracle, L, res, logits, X, topk, experts=range(E))
    check_end_to_end(oracle, L, res, logits, X, topk, tokens=range(min(T, 6)))


def test_moe_expert_without_tokens_and_skewed_load(qmm, oracle):
    T, E, topk, H, I = 96, 16, 2, 256, 256
    L = Layer(qmm, Q4, 611, E, H, I)
    X = synth.activations(612, 0, T, H)
    logits = synth.logits(613, 0, T, E)
    logits[:, 5] = -50.0                                 # expert 5 never selected
    logits[:, 2] += 6.0                                  # expert 2 selected by (almost) every token
    res = run_layer(qmm, L, logits, X, topk)
    assert res["expert_offsets"][6] == res["expert_offsets"][5]
    check_stages(oracle, L, res, logits, X, topk, experts=range(E))


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("T", [3, 120])
def test_moe_negative_and_zero_scales(qmm, oracle, fmt, T):
    """Expert weights with arbitrary codes and one block in 16 carrying a negative, zero or -0 scale,
    through the decode-sized path (T = 3: GEMVs) and the grouped tensor-core products (T = 120), at the
    stage-wise tolerances."""
    E, topk, H, I = 8, 2, 256, 512
    mk = lambda seed, rows, cols: util.random_blocks(synth, fmt, rows, cols, seed=seed, special_scales="no_subnormal",
                                                     scale_bits=(0x1000, 0x2400))[0]      # 2^-11 .. 2^-6
    L = Layer(qmm, fmt, 0, E, H, I, blocks=(mk(640 + fmt, E * I, H), mk(641 + fmt, E * I, H), mk(642 + fmt, E * H, I)))
    X = synth.activations(643, T, T, H)
    logits = synth.logits(644, T, T, E)
    res = run_layer(qmm, L, logits, X, topk)
    assert np.all(np.isfinite(res["out"].astype(np.float64)))
    check_stages(oracle, L, res, logits, X, topk, experts=range(E))
    check_end_to_end(oracle, L, res, logits, X, topk, tokens=range(min(T, 4)))


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("T,E,topk,H,I", [(1, 128, 8, 2048, 768), (4, 128, 8, 512, 256), (3, 16, 5, 256, 512), (32, 8, 1, 256, 256),
                                          (2, 256, 7, 256, 256), (1, 128, 8, 256, 1024)])
def test_moe_decode_two_launches_match_the_four_launch_form(qmm, oracle, fmt, T, E, topk, H, I):
    """Decode-sized layers run as two launches (routing inside the gate/up launch, down product and
    combine in one cluster kernel).  Forcing the separate route / gate-up / down / combine launches must
    give the same routing, the same Hm and D, and the same output bits: both forms do the same
    arithmetic in the same order."""
    L = Layer(qmm, fmt, 650 + T + E + topk, E, H, I)
    X = synth.activations(651, T + topk, T, H)
    logits = synth.logits(652, T + E, T, E)
    fused = run_layer(qmm, L, logits, X, topk)
    check_stages(oracle, L, fused, logits, X, topk, experts=sorted(set(fused["topk_idx"].reshape(-1).tolist())))
    check_end_to_end(oracle, L, fused, logits, X, topk, tokens=range(min(T, 3)))
    qmm.debug_config("moe_no_fuse", "1")
    plain = run_layer(qmm, L, logits, X, topk)
    for k in ("topk_idx", "topk_w", "perm", "expert_offsets", "dbg_H", "dbg_D", "out"):
        assert np.array_equal(fused[k], plain[k]), k
    qmm.debug_config(None)
    routed = run_layer(qmm, L, logits, X, topk, route_only=True)
    for k in ("topk_idx", "topk_w", "perm", "expert_offsets"):
        assert np.array_equal(fused[k], routed[k]), k
    assert np.all(routed["out"] == 3.0)


@pytest.mark.parametrize("fmt", [Q4, Q8])
@pytest.mark.parametrize("T", [1, 4])
def test_moe_decode_with_the_router_product_inside(qmm, oracle, fmt, T):
    """The library computes the router logits itself (X times the packed [E, H] router matrix, fp32
    outputs) ahead of the routing.  The exported logits are held to the product tolerance against the
    oracle; everything downstream is then checked against the oracle fed with those very logits, so the
    routing stays a bit-exact comparison."""
    E, topk, H, I = 128, 8, 512, 256
    L = Layer(qmm, fmt, 660 + T, E, H, I)
    X = synth.activations(661, T, T, H)
    wr = synth.quantize(fmt, synth.weights(662, fmt, E, H, std=0.05))
    out = torch.full((T, H), 3.0, dtype=torch.float16, device="cuda")
    o = dict(topk_idx=torch.full((T, topk), -1, dtype=torch.int32, device="cuda"),
             topk_w=torch.zeros((T, topk), dtype=torch.float32, device="cuda"),
             perm=torch.full((T * topk,), -1, dtype=torch.int32, device="cuda"),
             expert_offsets=torch.full((E + 1,), -1, dtype=torch.int32, device="cuda"),
             dbg_H=torch.zeros((T * topk, I), dtype=torch.float16, device="cuda"),
             dbg_D=torch.zeros((T * topk, H), dtype=torch.float16, device="cuda"))
    lg = torch.zeros((T, E), dtype=torch.float32, device="cuda")
    args = qmm.moe_args(fmt, T, H, I, E, topk, None, util.dev(X), L.p_gate, L.p_up, L.p_down, out,
                        w_router=qmm.pack(fmt, util.dev(wr), E, H), router_logits=lg, **o)
    ws = torch.zeros(qmm.moe_workspace_bytes(args), dtype=torch.uint8, device="cuda")
    qmm.moe(args, ws)
    qmm.status_check(ws)
    logits = lg.cpu().numpy()
    ref, B = oracle.gemm(fmt, wr, E, H, X)
    util.assert_within_tol(logits.astype(np.float64), ref, B, "router logits")
    res = {k: v.cpu().numpy() for k, v in o.items()}
    res["out"] = out.cpu().numpy()
    check_stages(oracle, L, res, logits, X, topk, experts=sorted(set(res["topk_idx"].reshape(-1).tolist())))
    check_end_to_end(oracle, L, res, logits, X, topk, tokens=range(T))
    # without an export buffer the logits live in the workspace: same output
    out2 = torch.empty_like(out)
    args2 = qmm.moe_args(fmt, T, H, I, E, topk, None, util.dev(X), L.p_gate, L.p_up, L.p_down, out2,
                         w_router=qmm.pack(fmt, util.dev(wr), E, H))
    ws2 = torch.zeros(qmm.moe_workspace_bytes(args2), dtype=torch.uint8, device="cuda")
    qmm.moe(args2, ws2)
    assert torch.equal(out, out2)
    # prefill-sized layers take caller logits only
    big = qmm.moe_args(fmt, 64, H, I, E, topk, None, util.dev(synth.activations(1, 1, 64, H)), L.p_gate, L.p_up, L.p_down,
                       torch.empty((64, H), dtype=torch.float16, device="cuda"), w_router=qmm.pack(fmt, util.dev(wr), E, H))
    assert qmm.lib().qmm_moe(big, ws.data_ptr(), ws.numel(), None) == 5


def test_moe_route_only_and_determinism(qmm, oracle):
    T, E, topk, H, I = 300, 128, 8, 256, 256
    L = Layer(qmm, Q4, 621, 1, H, I)                     # weights unused by the routing call
    L.E = E
    logits = synth.logits(622, 0, T, E)
    X = synth.activations(623, 0, T, H)
    first = run_layer(qmm, L, logits, X, topk, route_only=True)
    check_routing(oracle, first, logits, topk, E)
    assert np.all(first["out"] == 3.0)                   # the routing call writes no layer output
    for _ in range(3):
        again = run_layer(qmm, L, logits, X, topk, route_only=True)
        for k in ("topk_idx", "perm", "expert_offsets", "topk_w"):
            assert np.array_equal(first[k], again[k])


@pytest.fixture(scope="module")
def cfg4_layer(qmm):
    c = synth.CFG4
    return Layer(qmm, c["fmt"], c["seed"], c["E"], c["H"], c["I"])


@pytest.mark.parametrize("T", synth.CFG4["Ts"])
def test_cfg4_full_size_sampled(qmm, oracle, cfg4_layer, T):
    c = synth.CFG4
    L = cfg4_layer
    X = synth.activations(c["seed"], 100 + T, T, c["H"])
    logits = synth.logits(c["seed"], 200 + T, T, c["E"])
    res = run_layer(qmm, L, logits, X, c["topk"])
    counts = np.diff(res["expert_offsets"])
    experts = sorted({int(np.argmax(counts)), int(np.argmin(np.where(counts > 0, counts, 1 << 30))), 0, c["E"] - 1, 77})
    rng = np.random.default_rng(T)
    tokens = np.unique(np.concatenate([[0, T - 1], rng.integers(0, T, size=6)]))
    check_stages(oracle, L, res, logits, X, c["topk"], experts=experts, rows_per_expert=6, tokens=tokens)
    check_end_to_end(oracle, L, res, logits, X, c["topk"], tokens=tokens[:3])
