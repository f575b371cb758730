#!/usr/bin/env python
"""Benchmark of the block-quantised dequantise-and-multiply path on B200.

`python bench.py --gpus N --steps K --warmup W` prints ONE JSON line.

Headline (`value`): effective HBM GB/s of the decode GEMV stack -- a 16-layer,
1B-class transformer's linear layers at M = 1, in Q4 and in Q8 (the second
benchmark configuration): quantised-weight bytes read per step / step time.
One step = one pass over both stacks (every q/k/v/o/gate/up/down product of all
16 layers, once in Q4 and once in Q8).  Extra sections in the same line time
the other parts of the path on their own workloads: the Q8 LM-head GEMV, the
Q4 prefill GEMM (tensor cores) and the Q4 mixture-of-experts layer.

`--impl reference` times the CPU oracle (a deliberately plain program) on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_00501_b200 import synth  # noqa: E402

METRIC = "decode GEMV effective HBM bandwidth on quantised-weight bytes (Q4+Q8 16-layer stack)"
UNIT = "GB/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of gemv_batch_kernel on this workload: a RECORDED
# figure from one ncu capture per format of `bench.py --case gemv_batch_q4|q8` (algorithmic bytes:
# 547 356 672 / 1 033 895 936).  It is reported beside the live timings, never used in a computation, and
# does not change when the kernel does -- re-capture after changing gemv_batch_kernel.
NCU_DRAM_TRAFFIC = {synth.Q4: 552_050_000, synth.Q8: 1_038_200_000}
NCU_DRAM_TRAFFIC_SOURCE = "recorded from an ncu capture of --case gemv_batch_q4 / gemv_batch_q8; not measured in this run"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# fused launches per layer: (name, constituent matrices, N, K, activation)
FUSED = (("qkv", ("q", "k", "v"), 3072, 2048, "x_attn"), ("o", ("o",), 2048, 2048, "x_o"),
         ("gate_up", ("gate", "up"), 16384, 2048, "x_ffn"), ("down", ("down",), 2048, 8192, "x_down"))


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# --------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while a timed region runs (read-only queries).
    Every sample carries nvidia-smi's own timestamp, so that one sampler can serve several regions:
    stop() summarises all samples, window(t0, t1) those taken between two time.time() values."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, gpu_index: int, interval_ms: int = 100):
        self.gpu = gpu_index
        self.interval_ms = interval_ms
        self.proc = None
        self.path = None
        self.rows = []                  # (unix time, sm MHz, max sm MHz, power W, active reasons)

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", str(self.interval_ms)],
                                         stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def summarise(rows):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if rows:
            reasons = sorted({r for row in rows for r in row[4]})
            out.update(sm_mhz=float(np.median([r[1] for r in rows])), sm_max_mhz=rows[-1][2], reasons=reasons,
                       samples=len(rows), power_w_max=max(r[3] for r in rows))
        return out

    def stop(self):
        if self.proc is None:
            return self.summarise([])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        import datetime
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    row = (ts, float(f[1]), float(f[2]), float(f[3]),
                           [n for n, v in zip(self.REASONS, f[5:9]) if v.lower().startswith("active")])
                except ValueError:
                    continue
                self.rows.append(row)
            os.unlink(self.path)
        except Exception:
            pass
        return self.summarise(self.rows)

    def window(self, t0: float, t1: float):
        """Summary of the samples taken between two time.time() values (call after stop())."""
        return self.summarise([r for r in self.rows if t0 <= r[0] <= t1])


# --------------------------------------------------------------------------
# workload construction
# --------------------------------------------------------------------------

def build_stack_host(layers: int, fmts, threads: int = 8):
    """Canonical blocks of the decode stack: {fmt: [ {name: blocks} per layer ]} and activations per layer."""
    def one(layer):
        out = {f: {} for f in fmts}
        for name, N, K, act, w in synth.cfg1_layer_weights(layer):
            for f in fmts:
                out[f][name] = synth.quantize(f, w)
        return out, synth.cfg1_layer_acts(layer)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        res = list(ex.map(one, range(layers)))
    return {f: [r[0][f] for r in res] for f in fmts}, [r[1] for r in res]


def stack_bytes(fmt):
    return sum(synth.canonical_bytes(fmt, N, K) for _, N, K, _ in synth.CFG1_LAYER) * synth.CFG1["layers"]


# --------------------------------------------------------------------------
# multi-rank plumbing (weak scaling: every rank decodes its own tokens)
# --------------------------------------------------------------------------

def rank_activations(rank: int, host_acts):
    """Rank 0 keeps the workload's activations; every other rank draws its own (same shapes,
    its own seed) -- each rank stands for an independent decode request on the same weights."""
    if rank == 0:
        return host_acts
    return [{k: synth.activations(synth.CFG1["seed"] + 1000 * rank, 17 * l + i, v.size)
             for i, (k, v) in enumerate(a.items())} for l, a in enumerate(host_acts)]


def max_over_ranks(dist, values, device):
    """Element-wise maximum over all ranks (the job is as slow as its slowest rank)."""
    import torch
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(world: int, bytes_per_rank_step: int, ms_per_step: float) -> float:
    """GB/s over all ranks: every rank moves bytes_per_rank_step per step."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


# --------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------

def run_ours(args):
    import torch
    from paper_2607_00501_b200 import qmm

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod
    qmm.lib()
    pk = peaks()
    layers = synth.CFG1["layers"]
    fmts = synth.CFG1["fmts"]

    t_gen = time.time()
    host_blocks, host_acts = build_stack_host(layers, fmts)
    host_acts = rank_activations(rank, host_acts)
    gen_s = time.time() - t_gen

    # ---- device residency: packed weights (fused per launch), activations, outputs
    def dev_u8(a):
        return torch.from_numpy(a).cuda()

    ops = {f: [] for f in fmts}                          # (N, K, packed, x, y, ws)
    rows_of = {n: NN for n, NN, _, _ in synth.CFG1_LAYER}
    # all activation vectors live in one device buffer (one H2D copy per step in the e2e leg)
    x_host_all = np.concatenate([a[k] for a in host_acts for k, _ in synth.CFG1_ACTS])
    x_all = torch.from_numpy(x_host_all).cuda()
    x_dev, off = [], 0
    for a in host_acts:
        d = {}
        for k, n in synth.CFG1_ACTS:
            d[k] = x_all[off:off + n]
            off += n
        x_dev.append(d)
    need_fused = args.mode == "streams" or not args.no_sections     # fused per-matrix launches: streams mode, chained sections
    for f in (fmts if need_fused else ()):
        for l in range(layers):
            for name, parts, N, K, act in FUSED:
                packed = torch.cat([qmm.pack(f, dev_u8(host_blocks[f][l][p]), rows_of[p], K) for p in parts])
                y = torch.empty(N, dtype=torch.float16, device="cuda")
                need = qmm.gemv_workspace_bytes(f, N, K)
                ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
                ops[f].append((N, K, packed, x_dev[l][act], y, ws))
    # the same stack as one batched launch per format: every matrix its own problem (no fusion needed)
    batch = {}
    rows_per_stack = sum(N for _, N, _, _ in synth.CFG1_LAYER) * layers
    y_all = torch.empty(rows_per_stack * len(fmts), dtype=torch.float16, device="cuda")   # one D2H copy per step
    # a second set of activation / output buffers (same weights) so that the end-to-end leg can copy
    # step i+1 in and step i-1 out while step i computes
    x_all2, y_all2, batch2 = torch.empty_like(x_all), torch.empty_like(y_all), {}
    off = 0
    for f in fmts:
        probs, probs2 = [], []
        for l in range(layers):
            for name, N, K, act in synth.CFG1_LAYER:
                w = qmm.pack(f, dev_u8(host_blocks[f][l][name]), N, K)
                x = x_dev[l][act]
                x2 = x_all2[x.storage_offset():x.storage_offset() + x.numel()]
                probs.append((w, N, K, x, y_all[off:off + N]))
                probs2.append((w, N, K, x2, y_all2[off:off + N]))
                off += N
        batch[f] = qmm.gemv_batch_problems(probs)
        batch2[f] = qmm.gemv_batch_problems(probs2)
    torch.cuda.synchronize()
    bytes_step = sum(stack_bytes(f) for f in fmts)
    launches_per_step = len(fmts) if args.mode == "batch" else sum(len(v) for v in ops.values())

    nstreams = args.streams
    main = torch.cuda.Stream()
    side = [torch.cuda.Stream() for _ in range(nstreams)]

    def issue_all():
        """Every GEMV of both stacks.  The products are independent (each has its own seeded
        activation vector).  mode 'batch': one qmm_gemv_batch launch per format (112 problems each).
        mode 'streams': one qmm_gemv launch per fused matrix, spread over `nstreams` streams; within
        a stream consecutive launches are chained with programmatic dependent launch."""
        if args.mode == "batch":
            for f in fmts:
                qmm.gemv_batch(f, batch[f])
            return
        flat = [(f,) + op for f in fmts for op in ops[f]]
        if nstreams <= 1:
            for f, N, K, w, x, y, ws in flat:
                qmm.gemv(f, w, N, K, x, y=y, ws=ws)
            return
        ev = torch.cuda.Event()
        ev.record(torch.cuda.current_stream())
        for i, (f, N, K, w, x, y, ws) in enumerate(flat):
            st = side[i % nstreams]
            if i < nstreams:
                st.wait_event(ev)
            with torch.cuda.stream(st):
                qmm.gemv(f, w, N, K, x, y=y, ws=ws)
        for st in side:
            e = torch.cuda.Event()
            e.record(st)
            torch.cuda.current_stream().wait_event(e)

    with torch.cuda.stream(main):
        issue_all()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=main):
            issue_all()
        graph2 = None
        if args.mode == "batch":
            for f in fmts:
                qmm.gemv_batch(f, batch2[f])
            torch.cuda.synchronize()
            graph2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph2, stream=main):
                for f in fmts:
                    qmm.gemv_batch(f, batch2[f])

        def barrier():
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()

        for _ in range(max(args.warmup, 3)):
            graph.replay()
        barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        evs[0].record()
        for i in range(args.steps):
            graph.replay()
            evs[i + 1].record()
        barrier()
        step_ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]
        total_ms = evs[0].elapsed_time(evs[-1])
        # the two kernels of the step timed one by one (same launches, one format at a time)
        per_kernel = {}
        if args.mode == "batch":
            for f in fmts:
                for _ in range(3):
                    qmm.gemv_batch(f, batch[f])
                k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                k0.record()
                for _ in range(args.steps):
                    qmm.gemv_batch(f, batch[f])
                k1.record()
                torch.cuda.synchronize()
                us = k0.elapsed_time(k1) * 1e3 / args.steps
                per_kernel["gemv_batch_kernel<Q%d>" % f] = {
                    "avg_launch_us": round(us, 2), "algorithmic_bytes": stack_bytes(f),
                    "achieved_GBps": round(stack_bytes(f) / us / 1e3, 1),
                    "frac": round(stack_bytes(f) / us / 1e3 / pk["hbm_gbs"], 4),
                    "ncu_dram_traffic_bytes": NCU_DRAM_TRAFFIC[f]}
        # keep the GPU busy a little longer so that the clock sampler sees load even for short runs
        t_end = time.time() + 1.0
        while time.time() < t_end:
            graph.replay()
        torch.cuda.synchronize()
        clocks = sampler.stop() if rank == 0 else None

        # ---- end to end through the C ABI with host buffers: H2D activations, D2H outputs, per step
        pin_x = torch.from_numpy(x_host_all).pin_memory()
        ys = [y_all] if args.mode == "batch" else [op[4] for f in fmts for op in ops[f]]
        pin_y = [torch.empty(y.shape, dtype=y.dtype).pin_memory() for y in ys]
        h2d = pin_x.numel() * 2
        d2h = sum(y.numel() * 2 for y in ys)

        if args.mode == "batch":
            # two buffer sets, three streams: step i's activations come from the host while step i-1
            # computes and step i-2's outputs go back; every step still moves its own h2d + d2h bytes
            pin_y2 = torch.empty(y_all2.shape, dtype=y_all2.dtype).pin_memory()
            sets = [(x_all, y_all, graph, pin_y[0]), (x_all2, y_all2, graph2, pin_y2)]
            cin, cout = torch.cuda.Stream(), torch.cuda.Stream()
            in_done = [torch.cuda.Event() for _ in range(2)]
            comp_done = [torch.cuda.Event() for _ in range(2)]
            out_done = [torch.cuda.Event() for _ in range(2)]
            step_no = [0]

            def e2e_step():
                b = step_no[0] % 2
                step_no[0] += 1
                xb, yb, gb, pb = sets[b]
                with torch.cuda.stream(cin):
                    cin.wait_event(comp_done[b])           # the step that last read this buffer set
                    xb.copy_(pin_x, non_blocking=True)
                    in_done[b].record(cin)
                main.wait_event(in_done[b])
                main.wait_event(out_done[b])               # its outputs have left the device
                gb.replay()
                comp_done[b].record(main)
                with torch.cuda.stream(cout):
                    cout.wait_event(comp_done[b])
                    pb.copy_(yb, non_blocking=True)
                    out_done[b].record(cout)

            def e2e_drain():
                for b in range(2):
                    main.wait_event(out_done[b])
        else:
            def e2e_step():
                x_all.copy_(pin_x, non_blocking=True)
                graph.replay()
                for src, dst in zip(ys, pin_y):
                    dst.copy_(src, non_blocking=True)

            def e2e_drain():
                pass

        for _ in range(4):
            e2e_step()
        e2e_drain()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            e2e_step()
        e2e_drain()
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        if args.mode == "batch":                           # the copies did arrive: same outputs in both sets
            assert torch.equal(pin_y[0], pin_y2)

    total_ms, e2e_ms = max_over_ranks(dist, [total_ms, e2e_ms], "cuda")
    ms_per_step = total_ms / args.steps
    value = whole_job_value(world, bytes_step, ms_per_step)
    e2e_value = whole_job_value(world, bytes_step, e2e_ms / args.steps)

    # N > 1 only: strong scaling of ONE matrix -- the Q8 LM head with its rows spread over the ranks and
    # an all-gather of the fp16 outputs (every rank ends with the whole vector in its own memory)
    sharded_section = None
    if world > 1 and not args.no_sections:
        try:
            from paper_2607_00501_b200 import sharded
            c = synth.CFG2
            r0, r1 = sharded.shard_rows(c["N"], world, rank)
            full = synth.weights(c["seed"], 0, c["N"], c["K"])
            per_row = (c["K"] // 32) * synth.BLOCK_BYTES[c["fmt"]]
            blocks = np.zeros(c["N"] * per_row, dtype=np.uint8)          # only this rank's rows are quantised
            blocks.reshape(c["N"], per_row)[r0:r1] = synth.quantize(c["fmt"], full[r0:r1]).reshape(r1 - r0, per_row)
            del full
            op = sharded.RowShardedGemv(c["fmt"], blocks, c["N"], c["K"], device="cuda")
            xs = torch.from_numpy(synth.activations(c["seed"], 1, c["K"])).cuda()
            for _ in range(3):
                op(xs)
            torch.cuda.synchronize()
            dist.barrier()
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record()
            for _ in range(args.steps):
                op(xs)
            s1.record()
            torch.cuda.synchronize()
            ms, = max_over_ranks(dist, [s0.elapsed_time(s1) / args.steps], "cuda")
            nbytes = synth.canonical_bytes(c["fmt"], c["N"], c["K"])
            sharded_section = {"ms": round(ms, 4), "GBps_whole_matrix": round(nbytes / ms / 1e6, 1), "ranks": world,
                               "scaling": "strong", "exchange": "all_gather of %d fp16 outputs" % c["N"]}
        except Exception as ex:                                          # never lose the headline line to this section
            sharded_section = {"error": repr(ex)[:300]}

    sections = {}
    cpu = None
    if rank == 0 and not args.no_sections:
        sections = extra_sections(args, qmm, torch, pk, ops, fmts, batch, gpu_index=local)
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(host_blocks, host_acts, fmts, budget_s=args.cpu_seconds)

    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16 x int4/int8 -> f32 accumulate", "data": "synthetic",
        "config": {"workload": "cfg1: Q4+Q8 decode linear stack, 16 layers x 7 matrices, M=1",
                   "mode": args.mode, "launches_per_step": launches_per_step,
                   "streams": nstreams if args.mode == "streams" else 1,
                   "bytes_per_step": bytes_step, "l2": "inputs larger than L2 (1.58 GB of weights per step)",
                   "e2e": ("two buffer sets: a step's H2D / D2H copies overlap the neighbouring steps' kernels"
                           if args.mode == "batch" else "copies and kernels in sequence"),
                   "input_generation_s": round(gen_s, 1)},
        "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": round(value / world, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": round(value / world / pk["hbm_gbs"], 4),
                     "traffic": sum(NCU_DRAM_TRAFFIC[f] for f in fmts) if args.mode == "batch" else None,
                     "traffic_source": NCU_DRAM_TRAFFIC_SOURCE if args.mode == "batch" else None,
                     "frac_of_nominal_8000": round(value / world / NOMINAL_HBM_GBS, 4),
                     "algorithmic_bytes": bytes_step, "per_kernel": per_kernel,
                     "kernel": "gemv_batch_kernel (both launches of the step)" if args.mode == "batch" else "gemv_kernel (all launches of the step)", "peak_source": pk["source"],
                     "step_ms_min": round(min(step_ms), 5), "step_ms_max": round(max(step_ms), 5)},
        "cpu_baseline": cpu,
        "sections": dict(sections, **({"lm_head_q8_row_sharded": sharded_section} if sharded_section else {})),
    }
    print(json.dumps(line))


def time_op(torch, fn, iters, flush=None):
    """Median and best device time (ms) of fn() over iters runs, L2 flushed before each run."""
    times = []
    for _ in range(iters):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    return float(np.median(times)), float(min(times))


def measure(torch, fn, flush, iters=10, sustain_s=0.12):
    """One workload: cold (L2 flushed before every run: median and best of `iters`), then back to back
    without flushing for ~sustain_s (the L2-warm, sustained figure; the clock sampler's samples of this
    window are attached by attach_clocks)."""
    fn()
    med, best = time_op(torch, fn, iters, flush)
    n = max(10, int(sustain_s * 1e3 / max(med, 1e-3)))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.time()
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    return {"ms": round(med, 4), "ms_best": round(best, 4), "ms_warm": round(e0.elapsed_time(e1) / n, 4), "_win": (t0, t1)}


def attach_clocks(node, sampler):
    """Replace every "_win" left by measure() with the SM clock seen in that window."""
    if isinstance(node, dict):
        if "_win" in node:
            w = sampler.window(*node.pop("_win"))
            node["sm_mhz_warm_run"] = w["sm_mhz"]
            if w["reasons"]:
                node["clock_reasons"] = w["reasons"]
        for v in node.values():
            attach_clocks(v, sampler)


def tensor_fracs(tf, pk):
    """TFLOP/s against the three tensor denominators: measured burst, measured sustained, nominal."""
    return {"TFLOPs": round(tf, 1), "frac_tensor_measured": round(tf / pk["bf16_tflops"], 4),
            "frac_tensor_sustained": round(tf / pk["bf16_tflops_sustained"], 4),
            "frac_tensor_nominal": round(tf / NOMINAL_BF16_TFLOPS, 4)}


def hbm_fracs(nbytes, ms, pk):
    gbs = nbytes / ms / 1e6
    return {"GBps": round(gbs, 1), "frac_hbm": round(gbs / pk["hbm_gbs"], 4), "frac_hbm_nominal": round(gbs / NOMINAL_HBM_GBS, 4)}


def extra_sections(args, qmm, torch, pk, ops, fmts, batch, gpu_index=0):
    """The rest of the path on its own workloads.  Every entry: `ms` = median device time with L2 flushed
    before each run, `ms_warm` = back to back without flushing (with the SM clock seen during that run)."""
    out = {}
    want = set(args.sections.split(",")) if args.sections else None
    on = lambda name: want is None or name in want
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    sampler = ClockSampler(gpu_index, interval_ms=20)
    sampler.start()

    # the decode stack as ONE launch (qmm_chain): with the real dependencies of a decoder -- q/k/v, then o
    # on the first 2048 of its outputs, then gate/up with SiLU*mul, then down, whose output is the next
    # layer's input: 64 dependent stages -- and, for comparison, the same 112 matrices as independent products
    for f in (fmts if on("chain") else ()):
        layers = len(ops[f]) // 4
        stages = []
        for l in range(layers):
            qkv, o, gu, down = ops[f][4 * l:4 * l + 4]                 # (N, K, packed, x, y, ws)
            base = 4 * l
            half = gu[2].numel() // 2
            stages.append(dict(op=qmm.CHAIN_LINEAR, N=3072, K=2048, packed=qkv[2],
                               **({"x": qkv[3]} if l == 0 else {"x_stage": base - 1, "x_offset": 0})))
            stages.append(dict(op=qmm.CHAIN_LINEAR, N=2048, K=2048, packed=o[2], x_stage=base, x_offset=0))
            stages.append(dict(op=qmm.CHAIN_GATE_UP_SILU, N=8192, K=2048, packed=gu[2][:half], packed_up=gu[2][half:],
                               x_stage=base + 1, x_offset=0))
            stages.append(dict(op=qmm.CHAIN_LINEAR, N=2048, K=8192, packed=down[2], x_stage=base + 2, x_offset=0,
                               **({"y": down[4]} if l == layers - 1 else {})))
        for name, st in (("dependent", stages),
                         ("independent", [dict(op=qmm.CHAIN_LINEAR, N=N, K=K, packed=w, x=x, y=y) for (w, N, K, x, y) in batch[f]._keep])):
            chain = qmm.Chain(f, st)
            chain.run()
            qmm.status_check(chain.ws)
            g, sg = torch.cuda.CUDAGraph(), torch.cuda.Stream()
            fn = chain.run
            try:
                with torch.cuda.stream(sg):
                    with torch.cuda.graph(g, stream=sg):
                        chain.run()
                fn = g.replay
            except Exception:
                pass                                                   # (timed as plain launches then)
            med, best = time_op(torch, fn, 20)
            qmm.status_check(chain.ws)
            b = stack_bytes(f)
            out["decode_stack_q%d_one_launch_%s" % (f, name)] = dict(
                {"ms": round(med, 4), "ms_best": round(best, 4), "stages": len(st), "launches": 1,
                 "as_graph": fn is not chain.run}, **hbm_fracs(b, med, pk))
            del chain, g

    # per-format decode stacks, one qmm_gemv launch per fused matrix, chained on one stream with
    # programmatic dependent launch (a dependency between consecutive launches, as in a real decoder)
    for f in (fmts if on("chained") else ()):
        g = torch.cuda.CUDAGraph()
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for N, K, w, x, y, ws in ops[f][:4]:
                qmm.gemv(f, w, N, K, x, y=y, ws=ws)
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=s):
                for N, K, w, x, y, ws in ops[f]:
                    qmm.gemv(f, w, N, K, x, y=y, ws=ws)
            med, best = time_op(torch, g.replay, 10)
        b = stack_bytes(f)
        out["decode_stack_q%d_chained" % f] = dict({"ms": round(med, 4), "launches": len(ops[f])}, **hbm_fracs(b, med, pk))
        # the same chain for a decode batch of 2 / 8 sequences: qmm_gemm with M = 2 (the single-token kernel
        # with the second token in the idle half of its MMAs) / M = 8 (few-token kernel) per fused matrix;
        # the weights are streamed once for all tokens, so the bytes are the same
        for Mb in (2, 8):
            gm = torch.cuda.CUDAGraph()
            with torch.cuda.stream(s):
                opsm = []
                for N, K, w, x, y, ws in ops[f]:
                    Xm = x.reshape(1, K).repeat(Mb, 1).contiguous()
                    Ym = torch.empty((Mb, N), dtype=torch.float16, device="cuda")
                    wsm = torch.zeros(max(qmm.gemm_workspace_bytes(f, Mb, N, K), 256), dtype=torch.uint8, device="cuda")
                    opsm.append((N, K, w, Xm, Ym, wsm))
                for N, K, w, Xm, Ym, wsm in opsm[:4]:
                    qmm.gemm(f, w, N, K, Xm, Y=Ym, ws=wsm)
                torch.cuda.synchronize()
                with torch.cuda.graph(gm, stream=s):
                    for N, K, w, Xm, Ym, wsm in opsm:
                        qmm.gemm(f, w, N, K, Xm, Y=Ym, ws=wsm)
                medm, _ = time_op(torch, gm.replay, 10)
                # for comparison: the same tokens through the tensor-core prefill kernel
                qmm.debug_config("gemm_no_small", "1")
                gt = torch.cuda.CUDAGraph()
                for N, K, w, Xm, Ym, wsm in opsm[:4]:
                    qmm.gemm(f, w, N, K, Xm, Y=Ym, ws=wsm)
                torch.cuda.synchronize()
                with torch.cuda.graph(gt, stream=s):
                    for N, K, w, Xm, Ym, wsm in opsm:
                        qmm.gemm(f, w, N, K, Xm, Y=Ym, ws=wsm)
                qmm.debug_config("gemm_no_small", "0")
                medt, _ = time_op(torch, gt.replay, 10)
            out["decode_stack_q%d_chained_batch%d" % (f, Mb)] = dict({"ms": round(medm, 4), "launches": len(opsm), "tokens": Mb,
                                                                      "ms_over_single_token": round(medm / med, 3),
                                                                      "ms_tensor_core_kernel": round(medt, 4)}, **hbm_fracs(b, medm, pk))
            del gm, gt, opsm

    # the whole decode stack for a batch of 2 / 8 sequences as ONE launch per format (qmm_gemm_batch: the 112
    # matrices as independent problems, X [M, K] each): the weights are streamed once for all tokens, so the
    # algorithmic bytes are those of the single-token step.  Two sequences ride in the single-token kernel's
    # MMAs (the half of the B operand it leaves zero); eight run on the few-token ring kernel.
    for f in (fmts if on("batch8") else ()):
        for Mb in (2, 8):
            probs_m = []
            for w, N, K, x, y in batch[f]._keep:
                probs_m.append((w, N, K, x.reshape(1, K).repeat(Mb, 1).contiguous(), torch.empty((Mb, N), dtype=torch.float16, device="cuda")))
            arr_m = qmm.gemm_batch_problems(probs_m)
            g = torch.cuda.CUDAGraph()
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                qmm.gemm_batch(f, arr_m)
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=s):
                    qmm.gemm_batch(f, arr_m)
                m = measure(torch, g.replay, flush)
            out["decode_stack_q%d_batch%d_one_launch" % (f, Mb)] = dict(m, tokens=Mb, problems=len(probs_m), **hbm_fracs(stack_bytes(f), m["ms"], pk))
            del g, arr_m, probs_m

    # cfg0: one small Q4 GEMV (1.77 MB of weights: 0.27 us of HBM traffic, far below a launch).  Steady
    # state = 300 distinct packed copies (531 MB, larger than L2) so that every product streams from HBM:
    # as 300 chained launches in one graph, and as qmm_gemv_batch launches over the same 300 problems.
    if not on("cfg0"):
        return finish_sections(out, sampler) if not any(on(n) for n in ("lm_head", "ffn", "gemm", "formats", "moe")) else \
            rest_of_sections(args, qmm, torch, pk, fmts, out, flush, dev, sampler, on)
    c = synth.CFG0
    copies = 300
    blocks = synth.quantize(c["fmt"], synth.weights(c["seed"], 0, c["N"], c["K"]))
    one = qmm.pack(c["fmt"], dev(blocks), c["N"], c["K"])
    many = one.repeat(copies).reshape(copies, -1)
    x0 = dev(synth.activations(c["seed"], 1, c["K"]))
    y0 = torch.empty((copies, c["N"]), dtype=torch.float16, device="cuda")
    nb = blocks.nbytes

    def graph_of(fn_i):
        g, st = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        with torch.cuda.stream(st):
            fn_i(0)
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=st):
                for i in range(copies):
                    fn_i(i)
        return g

    g_cold = graph_of(lambda i: qmm.gemv(c["fmt"], many[i], c["N"], c["K"], x0, y=y0[i]))
    g_warm = graph_of(lambda i: qmm.gemv(c["fmt"], many[0], c["N"], c["K"], x0, y=y0[i]))
    arr = qmm.gemv_batch_problems([(many[i], c["N"], c["K"], x0, y0[i]) for i in range(copies)])
    cfg0 = {"bytes_per_gemv": nb, "copies": copies}
    med, _ = time_op(torch, g_cold.replay, 10)
    cfg0["chained_launches_hbm_cold"] = dict({"us_per_gemv": round(med * 1e3 / copies, 3)}, **hbm_fracs(nb * copies, med, pk))
    med, _ = time_op(torch, g_warm.replay, 10)
    cfg0["chained_launches_l2_warm"] = {"us_per_gemv": round(med * 1e3 / copies, 3), "GBps_from_l2": round(nb * copies / med / 1e6, 1)}
    med, _ = time_op(torch, lambda: qmm.gemv_batch(c["fmt"], arr), 10)
    cfg0["batched_hbm_cold"] = dict({"us_per_gemv": round(med * 1e3 / copies, 3), "launches": (copies + 127) // 128},
                                    **hbm_fracs(nb * copies, med, pk))
    med, best = time_op(torch, lambda: qmm.gemv(c["fmt"], many[7], c["N"], c["K"], x0, y=y0[7]), 20, flush)
    cfg0["isolated_launch_cold"] = dict({"us": round(med * 1e3, 3), "us_best": round(best * 1e3, 3)}, **hbm_fracs(nb, med, pk))
    out["cfg0_q4_gemv"] = cfg0
    del many, y0, g_cold, g_warm, arr
    return rest_of_sections(args, qmm, torch, pk, fmts, out, flush, dev, sampler, on)


def finish_sections(out, sampler):
    sampler.stop()
    attach_clocks(out, sampler)
    return out


def rest_of_sections(args, qmm, torch, pk, fmts, out, flush, dev, sampler, on):
    if not on("lm_head"):
        return sections_ffn_on(args, qmm, torch, pk, fmts, out, flush, dev, sampler, on)
    # cfg2: Q8 LM head GEMV
    c = synth.CFG2
    blocks = synth.quantize(c["fmt"], synth.weights(c["seed"], 0, c["N"], c["K"]))
    packed = qmm.pack(c["fmt"], dev(blocks), c["N"], c["K"])
    x = dev(synth.activations(c["seed"], 1, c["K"]))
    y = torch.empty(c["N"], dtype=torch.float16, device="cuda")
    m = measure(torch, lambda: qmm.gemv(c["fmt"], packed, c["N"], c["K"], x, y=y), flush, iters=20)
    out["lm_head_q8_gemv"] = dict(m, **hbm_fracs(blocks.nbytes, m["ms"], pk))
    del packed, blocks
    return sections_ffn_on(args, qmm, torch, pk, fmts, out, flush, dev, sampler, on)


def sections_ffn_on(args, qmm, torch, pk, fmts, out, flush, dev, sampler, on):
    # one cfg1 layer's feed-forward front half as a single launch: h = silu(Wgate x) * (Wup x)
    for f in (fmts if on("ffn") else ()):
        wts = {name: (N, K, w) for name, N, K, act, w in synth.cfg1_layer_weights(0) if name in ("gate", "up")}
        N, K, _ = wts["gate"]
        pgate = qmm.pack(f, dev(synth.quantize(f, wts["gate"][2])), N, K)
        pup = qmm.pack(f, dev(synth.quantize(f, wts["up"][2])), N, K)
        xf = dev(synth.cfg1_layer_acts(0)["x_ffn"])
        hf = torch.empty(N, dtype=torch.float16, device="cuda")
        fn = lambda: qmm.gemv_gate_up(f, pgate, pup, N, K, xf, hf)
        fn()
        med, best = time_op(torch, fn, 10, flush)
        b = 2 * synth.canonical_bytes(f, N, K)
        out["ffn_gate_up_silu_q%d_gemv" % f] = dict({"ms": round(med, 4)}, **hbm_fracs(b, med, pk))

    # cfg3: prefill GEMM sweep (Q4 as the config says, plus the small-batch sizes below one token tile:
    # M <= 8 runs on the few-token kernel, whose bound is the HBM stream of W; Q8 = the same kernels with
    # the byte expander, measured at M = 4 and the two largest M)
    c = synth.CFG3
    for f, Ms in (((c["fmt"], (2, 4, 8, 16, 32, 64) + tuple(c["Ms"])), (synth.Q8, (4,) + tuple(c["Ms"][-2:]))) if on("gemm") else ()):
        gemm = {}
        for name, N, K in c["shapes"]:
            blocks = synth.quantize(f, synth.weights(c["seed"], 0 if name == "gate_up" else 1, N, K))
            packed = qmm.pack(f, dev(blocks), N, K)
            for M in Ms:
                X = dev(synth.activations(c["seed"], 10 + M, M, K))
                Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
                ws = torch.zeros(qmm.gemm_workspace_bytes(f, M, N, K), dtype=torch.uint8, device="cuda")
                m = measure(torch, lambda: qmm.gemm(f, packed, N, K, X, Y=Y, ws=ws), flush)
                tf = 2.0 * M * N * K / m["ms"] / 1e9
                floor_ms = max(2.0 * M * N * K / pk["bf16_tflops"] / 1e9, (blocks.nbytes + 2 * M * (N + K)) / pk["hbm_gbs"] / 1e6)
                gemm["%s_M%d" % (name, M)] = dict(m, roofline_floor_ms=round(floor_ms, 4), frac_of_floor=round(floor_ms / m["ms"], 4),
                                                  **(hbm_fracs(blocks.nbytes, m["ms"], pk) if M <= 8 else tensor_fracs(tf, pk)))
                qmm.status_check(ws)
        out["prefill_gemm_q%d" % f] = gemm
    if on("gemm"):
        # not configs: two shapes the tile plan was never tuned on (its cycle estimates come from the cfg3 shapes)
        other = {}
        for N, K in ((4096, 4096), (14336, 4096)):
            blocks = synth.quantize(synth.Q4, synth.weights(33, N, N, K))
            packed = qmm.pack(synth.Q4, dev(blocks), N, K)
            for M in (512, 2048):
                X = dev(synth.activations(33, M, M, K))
                Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
                ws = torch.zeros(qmm.gemm_workspace_bytes(synth.Q4, M, N, K), dtype=torch.uint8, device="cuda")
                m = measure(torch, lambda: qmm.gemm(synth.Q4, packed, N, K, X, Y=Y, ws=ws), flush)
                qmm.status_check(ws)
                other["N%d_K%d_M%d" % (N, K, M)] = dict(m, **tensor_fracs(2.0 * M * N * K / m["ms"] / 1e9, pk))
        out["prefill_gemm_q4_other_shapes"] = other

    # not configs: the 5-bit and 6-bit formats through the same two kernel families (one decode-sized
    # GEMV on the LM-head shape, one prefill GEMM on the gate/up shape at M = 2048)
    for f in ((synth.Q5, synth.Q6) if on("formats") else ()):
        e = {}
        N, K = synth.CFG2["N"], synth.CFG2["K"]
        blocks = synth.quantize(f, synth.weights(synth.CFG2["seed"], 0, N, K))
        packed = qmm.pack(f, dev(blocks), N, K)
        x = dev(synth.activations(synth.CFG2["seed"], 1, K))
        y = torch.empty(N, dtype=torch.float16, device="cuda")
        m = measure(torch, lambda: qmm.gemv(f, packed, N, K, x, y=y), flush, iters=20)
        e["lm_head_gemv"] = dict(m, **hbm_fracs(blocks.nbytes, m["ms"], pk))
        _, N, K = synth.CFG3["shapes"][0]
        M = 2048
        blocks = synth.quantize(f, synth.weights(synth.CFG3["seed"], 0, N, K))
        packed = qmm.pack(f, dev(blocks), N, K)
        X = dev(synth.activations(synth.CFG3["seed"], 10 + M, M, K))
        Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        ws = torch.zeros(qmm.gemm_workspace_bytes(f, M, N, K), dtype=torch.uint8, device="cuda")
        m = measure(torch, lambda: qmm.gemm(f, packed, N, K, X, Y=Y, ws=ws), flush)
        qmm.status_check(ws)
        e["gemm_gate_up_M2048"] = dict(m, **tensor_fracs(2.0 * M * N * K / m["ms"] / 1e9, pk))
        out["format_q%d" % f] = e
        del packed, blocks

    # cfg4: MoE layer (Q4 as the config says; Q8 at the largest T)
    c = synth.CFG4

    def moe_entry(f, T, lg, pg, pu, pd, wbytes):
        X = dev(synth.activations(c["seed"], 100 + T, T, c["H"]))
        o = torch.empty((T, c["H"]), dtype=torch.float16, device="cuda")
        a = qmm.moe_args(f, T, c["H"], c["I"], c["E"], c["topk"], dev(lg), X, pg, pu, pd, o)
        ws = torch.zeros(qmm.moe_workspace_bytes(a), dtype=torch.uint8, device="cuda")
        m = measure(torch, lambda: qmm.moe(a, ws), flush)
        qmm.status_check(ws)
        fl = T * c["topk"] * 3 * 2.0 * c["H"] * c["I"]
        touched = min(1.0, T * c["topk"] / c["E"]) * wbytes + 4 * T * c["H"] + 4 * T * c["E"]
        floor_ms = max(fl / pk["bf16_tflops"] / 1e9, touched / pk["hbm_gbs"] / 1e6)
        return dict(m, hbm_floor_ms=round(touched / pk["hbm_gbs"] / 1e6, 4), roofline_floor_ms=round(floor_ms, 4),
                    frac_of_floor=round(floor_ms / m["ms"], 4), **tensor_fracs(fl / m["ms"] / 1e9, pk))

    for f, Ts in (((c["fmt"], c["Ts"]), (synth.Q8, c["Ts"][-1:])) if on("moe") else ()):
        gate, up, down = synth.moe_expert_weights(c["seed"], f, c["E"], c["H"], c["I"])
        pg = qmm.pack(f, dev(gate), c["E"] * c["I"], c["H"])
        pu = qmm.pack(f, dev(up), c["E"] * c["I"], c["H"])
        pd = qmm.pack(f, dev(down), c["E"] * c["H"], c["I"])
        wbytes = gate.nbytes + up.nbytes + down.nbytes
        moe = {}
        for T in Ts:
            moe["T%d" % T] = moe_entry(f, T, synth.logits(c["seed"], 200 + T, T, c["E"]), pg, pu, pd, wbytes)
        if f == c["fmt"]:
            # not a config: the same layer under an uneven expert load (a fixed N(0, 1.5^2) bias per
            # expert on the seeded logits; trained routers are skewed, the config's iid logits are not)
            T = c["Ts"][-1]
            bias = np.random.default_rng([c["seed"], 999]).standard_normal(c["E"]).astype(np.float32) * 1.5
            moe["T%d_skewed_load" % T] = moe_entry(f, T, synth.logits(c["seed"], 200 + T, T, c["E"]) + bias[None, :], pg, pu, pd, wbytes)
        out["moe_q%d" % f] = moe
        del pg, pu, pd, gate, up, down
    return finish_sections(out, sampler)


# --------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------

def cpu_baseline(host_blocks, host_acts, fmts, budget_s=12.0):
    """The oracle, as it stands, on the host cores: whole passes over the decode stack for ~budget_s."""
    import oracle
    shapes = {n: (N, K, a) for n, N, K, a in synth.CFG1_LAYER}
    t0 = time.time()
    done_bytes, done_layers = 0, 0
    while time.time() - t0 < budget_s:
        for l in range(len(host_acts)):
            for f in fmts:
                for name, (N, K, act) in shapes.items():
                    oracle.gemv(f, host_blocks[f][l][name], N, K, host_acts[l][act])
                    done_bytes += host_blocks[f][l][name].nbytes
            done_layers += 1
            if time.time() - t0 > budget_s:
                break
    dt = time.time() - t0
    return {"value": round(done_bytes / dt / 1e9, 3), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d layer passes (%.2f passes over the 16-layer Q4+Q8 decode stack, every GEMV), %.1f s" %
                      (done_layers, done_layers / len(host_acts), dt)}


def run_reference(args):
    """`--impl reference`: the CPU oracle on a bounded sample of the same workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    fmts = synth.CFG1["fmts"]
    layers = synth.CFG1["layers"]
    host_blocks, host_acts = build_stack_host(layers, fmts)
    shapes = {n: (N, K, a) for n, N, K, a in synth.CFG1_LAYER}
    nbytes = sum(host_blocks[f][l][n].nbytes for f in fmts for l in range(layers) for n in shapes)
    assert nbytes == sum(stack_bytes(f) for f in fmts)

    def step():
        for l in range(layers):
            for f in fmts:
                for name, (N, K, act) in shapes.items():
                    oracle.gemv(f, host_blocks[f][l][name], N, K, host_acts[l][act])

    for _ in range(max(args.warmup, 1)):
        step()
    t0 = time.time()
    for _ in range(args.steps):
        step()
    dt = time.time() - t0
    value = nbytes * args.steps / dt / 1e9
    sample = "the whole Q4+Q8 decode stack per step (all 16 layers, 224 GEMVs), host cores"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": max(args.warmup, 1),
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64 accumulate (CPU oracle)", "data": "synthetic",
        "config": {"workload": "cfg1: Q4+Q8 decode linear stack, 16 layers x 7 matrices, M=1", "sample": sample,
                   "bytes_per_step": nbytes},
        "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_case(args):
    """`--case NAME`: a few launches of one kernel on its benchmark workload and nothing else, so that a
    profiler can be pointed at it.  Prints no JSON.  Under ncu the flag `--clock-control none` is
    mandatory (without it ncu locks the GPU's clocks, and a killed ncu leaves them locked for the next
    user of a shared GPU); capture one kernel and a few launches:
    `ncu --clock-control none -k regex:gemm_kernel -s 2 -c 2 python bench.py --case gemm_q4_M2048`."""
    import torch
    from paper_2607_00501_b200 import qmm
    torch.cuda.set_device(0)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    name = args.case
    reps = 4
    if name in ("gemv_batch_q4", "gemv_batch_q8"):
        f = synth.Q4 if name.endswith("q4") else synth.Q8
        host_blocks, host_acts = build_stack_host(synth.CFG1["layers"], (f,))
        probs = []
        for l in range(synth.CFG1["layers"]):
            for mname, N, K, act in synth.CFG1_LAYER:
                probs.append((qmm.pack(f, dev(host_blocks[f][l][mname]), N, K), N, K, dev(host_acts[l][act]),
                              torch.empty(N, dtype=torch.float16, device="cuda")))
        arr = qmm.gemv_batch_problems(probs)
        for _ in range(reps):
            qmm.gemv_batch(f, arr)
    elif name in ("gemm_batch_q4_M8", "gemm_batch_q8_M8", "gemm_batch_q4_M2", "gemm_batch_q8_M2"):
        # the whole decode stack for a batch of 8 (or 2) sequences: 112 problems in one qmm_gemm_batch launch
        f = synth.Q4 if "_q4_" in name else synth.Q8
        Mb = int(name[-1])
        host_blocks, host_acts = build_stack_host(synth.CFG1["layers"], (f,))
        probs = []
        for l in range(synth.CFG1["layers"]):
            for mname, N, K, act in synth.CFG1_LAYER:
                probs.append((qmm.pack(f, dev(host_blocks[f][l][mname]), N, K), N, K,
                              dev(host_acts[l][act]).reshape(1, K).repeat(Mb, 1).contiguous(),
                              torch.empty((Mb, N), dtype=torch.float16, device="cuda")))
        arr = qmm.gemm_batch_problems(probs)
        for _ in range(reps):
            qmm.gemm_batch(f, arr)
    elif name in ("chain_q4_dependent", "chain_q4_independent", "chain_q8_dependent", "chain_q8_independent"):
        # four layers of the decode stack (137 / 258 MB of weights) through qmm_chain: as a dependent chain of
        # 16 stages, or as 28 independent products
        f = synth.Q4 if "_q4_" in name else synth.Q8
        layers = 4
        host_blocks, host_acts = build_stack_host(layers, (f,))
        rows_of = {n: NN for n, NN, _, _ in synth.CFG1_LAYER}
        stages = []
        if name.endswith("independent"):
            for l in range(layers):
                for mname, N, K, act in synth.CFG1_LAYER:
                    stages.append(dict(op=qmm.CHAIN_LINEAR, N=N, K=K, packed=qmm.pack(f, dev(host_blocks[f][l][mname]), N, K),
                                       x=dev(host_acts[l][act]), y=torch.empty(N, dtype=torch.float16, device="cuda")))
        else:
            for l in range(layers):
                pk_ = lambda parts, K: torch.cat([qmm.pack(f, dev(host_blocks[f][l][p]), rows_of[p], K) for p in parts])
                base = 4 * l
                stages.append(dict(op=qmm.CHAIN_LINEAR, N=3072, K=2048, packed=pk_(("q", "k", "v"), 2048),
                                   **({"x": dev(host_acts[0]["x_attn"])} if l == 0 else {"x_stage": base - 1, "x_offset": 0})))
                stages.append(dict(op=qmm.CHAIN_LINEAR, N=2048, K=2048, packed=pk_(("o",), 2048), x_stage=base, x_offset=0))
                stages.append(dict(op=qmm.CHAIN_GATE_UP_SILU, N=8192, K=2048, packed=pk_(("gate",), 2048), packed_up=pk_(("up",), 2048),
                                   x_stage=base + 1, x_offset=0))
                stages.append(dict(op=qmm.CHAIN_LINEAR, N=2048, K=8192, packed=pk_(("down",), 8192), x_stage=base + 2, x_offset=0,
                                   y=torch.empty(2048, dtype=torch.float16, device="cuda")))
        chain = qmm.Chain(f, stages)
        for _ in range(reps):
            chain.run()
        qmm.status_check(chain.ws)
    elif name == "gemv_lm_head_q8":
        c = synth.CFG2
        packed = qmm.pack(c["fmt"], dev(synth.quantize(c["fmt"], synth.weights(c["seed"], 0, c["N"], c["K"]))), c["N"], c["K"])
        x = dev(synth.activations(c["seed"], 1, c["K"]))
        y = torch.empty(c["N"], dtype=torch.float16, device="cuda")
        for _ in range(reps):
            qmm.gemv(c["fmt"], packed, c["N"], c["K"], x, y=y)
    elif name in ("gemv_kv_q4", "gemv_kv_q8"):
        # the k / v projection of the decode stack: 512 rows do not fill the SMs, so K is split over a
        # thread-block cluster.  64 distinct copies (37-70 MB) so that a few launches are not all L2 hits.
        f = synth.Q4 if name.endswith("q4") else synth.Q8
        N, K = 512, 2048
        one = qmm.pack(f, dev(synth.quantize(f, synth.weights(1, 1, N, K))), N, K)
        many = one.repeat(64).reshape(64, -1)
        x = dev(synth.activations(1, 1000, K))
        y = torch.empty(N, dtype=torch.float16, device="cuda")
        for i in range(8):
            qmm.gemv(f, many[i * 8], N, K, x, y=y)
    elif name.startswith("gemm_few_q") and "_M" in name:
        # gemm_few_q4_M8: the few-token kernel (M <= 8) on a [28672, 4096] matrix; three distinct copies
        # (198 MB in Q4, 374 MB in Q8) taken in turn, so that every launch streams from HBM
        f = synth.Q4 if name.startswith("gemm_few_q4") else synth.Q8
        M = int(name.split("_M")[1])
        N, K = 28672, 4096
        one = qmm.pack(f, dev(synth.quantize(f, synth.weights(9, 9, N, K))), N, K)
        copies = [one, one.clone(), one.clone()]
        X = dev(synth.activations(9, 10 + M, M, K))
        Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        ws = torch.zeros(max(qmm.gemm_workspace_bytes(f, M, N, K), 256), dtype=torch.uint8, device="cuda")
        for i in range(6):
            qmm.gemm(f, copies[i % 3], N, K, X, Y=Y, ws=ws)
        qmm.status_check(ws)
    elif name.startswith("gemm_q") and "_M" in name:
        # gemm_q4_M2048 (gate/up shape), gemm_q8_M1024, gemm_q4_down_M512 ...
        c = synth.CFG3
        f = synth.Q4 if name.startswith("gemm_q4") else synth.Q8
        M = int(name.split("_M")[1])
        which = 1 if "_down_" in name else 0
        _, N, K = c["shapes"][which]
        packed = qmm.pack(f, dev(synth.quantize(f, synth.weights(c["seed"], which, N, K))), N, K)
        X = dev(synth.activations(c["seed"], 10 + M, M, K))
        Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        ws = torch.zeros(qmm.gemm_workspace_bytes(f, M, N, K), dtype=torch.uint8, device="cuda")
        for _ in range(reps):
            qmm.gemm(f, packed, N, K, X, Y=Y, ws=ws)
        qmm.status_check(ws)
    elif name.startswith("moe_q") and "_T" in name:
        c = synth.CFG4
        f = synth.Q4 if name.startswith("moe_q4") else synth.Q8
        T = int(name.split("_T")[1])
        gate, up, down = synth.moe_expert_weights(c["seed"], f, c["E"], c["H"], c["I"])
        pg, pu = qmm.pack(f, dev(gate), c["E"] * c["I"], c["H"]), qmm.pack(f, dev(up), c["E"] * c["I"], c["H"])
        pd = qmm.pack(f, dev(down), c["E"] * c["H"], c["I"])
        X = dev(synth.activations(c["seed"], 100 + T, T, c["H"]))
        lg = dev(synth.logits(c["seed"], 200 + T, T, c["E"]))
        o = torch.empty((T, c["H"]), dtype=torch.float16, device="cuda")
        a = qmm.moe_args(f, T, c["H"], c["I"], c["E"], c["topk"], lg, X, pg, pu, pd, o)
        ws = torch.zeros(qmm.moe_workspace_bytes(a), dtype=torch.uint8, device="cuda")
        for _ in range(reps):
            qmm.moe(a, ws)
        qmm.status_check(ws)
    else:
        raise SystemExit("unknown --case %r (gemv_batch_q4|q8, gemm_batch_q4|q8_M2|M8, gemv_lm_head_q8, gemv_kv_q4|q8, gemm_q4|q8[_down]_M<M>, gemm_few_q4|q8_M<M>, "
                         "moe_q4|q8_T<T>, chain_q4|q8_dependent|independent)" % name)
    torch.cuda.synchronize()
    print("case %s: %d launches done" % (name, reps), file=sys.stderr)


def launch_ranks(n: int, argv) -> int:
    """`--gpus N` without a launcher: start N ranks of this script under torch.distributed.run on this
    node (one process per GPU, rendezvous on 127.0.0.1), exactly as an external launcher would."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_dry(args):
    """`--dry-run-cpu`: the multi-rank plumbing of the benchmark with no GPU and no kernels (gloo): every
    rank draws its own activations, pretends its step took (1 + rank) ms, the ranks agree on the maximum
    and rank 0 prints the whole-job line.  Exists so that the launcher and the N > 1 bookkeeping can be
    tested where there is no GPU; the line says "dry_run": true and carries no measurement."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    acts = rank_activations(rank, [synth.cfg1_layer_acts(0)])
    ms, = max_over_ranks(dist if world > 1 else None, [1.0 + rank], "cpu")
    value = whole_job_value(world, 1000, ms)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "gpus_arg": args.gpus, "ms_per_step": ms, "value": value,
                          "scaling": "weak", "x_attn_checksum": float(np.abs(acts[0]["x_attn"].astype(np.float64)).sum())}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--dry-run-cpu", action="store_true", help="test aid: multi-rank plumbing only, gloo, no GPU (see run_dry)")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="batch", choices=["batch", "streams"],
                    help="batch: one qmm_gemv_batch launch per format; streams: one qmm_gemv launch per matrix")
    ap.add_argument("--streams", type=int, default=8, help="streams for --mode streams")
    ap.add_argument("--no-sections", action="store_true", help="skip the LM-head / GEMM / MoE sections")
    ap.add_argument("--sections", default=None,
                    help="comma list of the sections to run (chain,chained,batch8,cfg0,lm_head,ffn,gemm,formats,moe); default: all")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--case", default=None, help="profiling aid: run a few launches of one kernel and exit (see run_case)")
    args = ap.parse_args()
    if args.case:
        run_case(args)
        return
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1:
        # not under a launcher: start the N ranks here (each re-enters main() with WORLD_SIZE set)
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if world_env is not None and int(world_env) != args.gpus and int(os.environ.get("RANK", "0")) == 0:
        print("bench.py: --gpus %d but the launcher started %s ranks; using the launcher's count" % (args.gpus, world_env),
              file=sys.stderr)
    if args.dry_run_cpu:
        run_dry(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
