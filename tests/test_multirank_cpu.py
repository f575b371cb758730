"""The N > 1 path of the benchmark on CPU: two gloo ranks (no GPU needed).

Covers what differs between ranks: each rank draws its own activations, the
step time is the maximum over ranks, the reported value is the whole-job sum,
and the reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2607_00501_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    base = [synth.cfg1_layer_acts(0)]
    mine = bench.rank_activations(rank, base)
    # rank r pretends its step took (1 + r) ms
    total_ms, = bench.max_over_ranks(dist, [1.0 + rank], "cpu")
    value = bench.whole_job_value(world, 1000, total_ms)
    dist.barrier()
    np.save(os.path.join(out_dir, "acts%d.npy" % rank), mine[0]["x_attn"])
    json.dump({"total_ms": total_ms, "value": value}, open(os.path.join(out_dir, "r%d.json" % rank), "w"))
    dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / ("r%d.json" % i))) for i in range(world)]
    assert r[0]["total_ms"] == r[1]["total_ms"] == 2.0           # the slowest rank sets the time
    assert r[0]["value"] == 2 * 1000 / 2e-3 / 1e9                # whole-job bytes over that time
    a0, a1 = np.load(tmp_path / "acts0.npy"), np.load(tmp_path / "acts1.npy")
    assert a0.shape == a1.shape and not np.array_equal(a0, a1)   # every rank decodes its own token


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_bench_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` outside any launcher starts two ranks under torch.distributed.run; the dry-run
    mode exercises that launcher and the N > 1 bookkeeping with gloo on CPU."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run-cpu"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                         # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["dry_run"] and d["n_gpus"] == 2 and d["gpus_arg"] == 2
    assert d["ms_per_step"] == 2.0 and d["value"] == 2 * 1000 / 2e-3 / 1e9


def _sharded_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import oracle
    from paper_2607_00501_b200 import sharded, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    res = {}
    for fmt, N, K in ((4, 384, 256), (8, 512, 512), (6, 256, 256)):       # 384 rows: 3 row blocks over 2 ranks (uneven)
        blocks = synth.quantize(fmt, synth.weights(77, fmt, N, K))
        x = synth.activations(77, 100 + fmt, K)
        # the local product on CPU: the oracle's fp64 result rounded to fp16 stands in for the GPU kernel
        prep = lambda f, b, n, k, dev: b
        prod = lambda f, b, n, k, xv: torch.from_numpy(oracle.gemv(f, b, n, k, xv.numpy())[0].astype(np.float16))
        op = sharded.RowShardedGemv(fmt, blocks, N, K, device="cpu", prepare=prep, product=prod)
        y = op(torch.from_numpy(x))
        res["%d_%d_%d" % (fmt, N, K)] = {"rows": [op.r0, op.r1], "y": y.numpy().view(np.uint16).tolist()}
    dist.barrier()
    json.dump(res, open(os.path.join(out_dir, "s%d.json" % rank), "w"))
    dist.destroy_process_group()


def test_row_sharded_gemv_two_ranks_equals_single_rank(tmp_path):
    """Two gloo ranks each hold half of W's rows, multiply and all-gather the fp16 outputs: every rank
    ends with the whole y, bit-identical to the unsharded product (rows are independent)."""
    import oracle
    from paper_2607_00501_b200 import sharded, synth
    world, port = 2, 31000 + os.getpid() % 2000
    mp.spawn(_sharded_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / ("s%d.json" % i))) for i in range(world)]
    for fmt, N, K in ((4, 384, 256), (8, 512, 512), (6, 256, 256)):
        key = "%d_%d_%d" % (fmt, N, K)
        blocks = synth.quantize(fmt, synth.weights(77, fmt, N, K))
        x = synth.activations(77, 100 + fmt, K)
        whole = oracle.gemv(fmt, blocks, N, K, x)[0].astype(np.float16).view(np.uint16).tolist()
        assert r[0][key]["y"] == whole and r[1][key]["y"] == whole
        assert r[0][key]["rows"][0] == 0 and r[0][key]["rows"][1] == r[1][key]["rows"][0] and r[1][key]["rows"][1] == N
    assert sharded.shard_rows(384, 2, 0) == (0, 256) and sharded.shard_rows(384, 2, 1) == (256, 384)
    assert sharded.shard_rows(128, 4, 3) == (128, 128)                     # more ranks than row blocks: an empty share
