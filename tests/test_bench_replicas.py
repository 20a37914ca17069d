"""The benchmark's multi-GPU mode is replicas only (no data-path collective): every rank runs the
same step on its own GPU, the timed region ends with the slowest rank, and the value is the bytes
all ranks processed over that time. Covered here on CPU with two gloo ranks; the reference arm must
print from rank 0 only."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, ms_by_rank, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    out = bench.replica_metrics(ms_by_rank[rank], step_bytes=1_000_000, steps=10, dist=dist, device="cpu")
    q.put((rank, out))
    dist.destroy_process_group()


def test_replica_metrics_take_the_slowest_rank_and_sum_the_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ms = [20.0, 50.0]   # rank 1 is slower
    procs = [ctx.Process(target=_worker, args=(r, 2, 29517, ms, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # both ranks agree; 2 replicas x 1 MB per step over 5 ms per step = 0.4 GB/s
    for r in range(2):
        ms_per_step, gbs, world = res[r]
        assert world == 2
        assert ms_per_step == pytest.approx(5.0)
        assert gbs == pytest.approx(2 * 1_000_000 / 5e-3 / 1e9)


def test_single_process_metrics():
    sys.path.insert(0, ROOT)
    import bench
    ms_per_step, gbs, world = bench.replica_metrics(30.0, step_bytes=3_000_000, steps=10)
    assert (world, ms_per_step) == (1, 3.0) and gbs == pytest.approx(1.0)


def test_reference_arm_prints_from_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "3", "--workload", "single_2048", "--sample-seconds", "0.05"]
    outs = []
    for rank in (0, 1):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29518")
        r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append([ln for ln in r.stdout.splitlines() if ln.strip()])
    assert outs[1] == []
    assert len(outs[0]) == 1
    line = json.loads(outs[0][0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
