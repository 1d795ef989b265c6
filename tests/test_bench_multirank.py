"""The N > 1 path of the benchmark on CPU: ranks are independent replicas (the path shards over sequences and KV heads
with no exchange), so all that crosses ranks is the slowest rank's time. Two gloo processes check that reduction, and a
two-rank launch of the reference arm checks that rank 0 alone works and prints the JSON line."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sec = bench.slowest_rank_seconds(1.0 + rank)            # rank 1 is the slow one
    value = bench.whole_job_value(1000.0, world, sec)
    out.put((rank, sec, value))
    dist.barrier()
    dist.destroy_process_group()


def test_slowest_rank_sets_the_whole_job_value():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29531, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, sec, value in got:
        assert sec == 2.0 and value == 2 * 1000.0 / 2.0


def test_single_process_is_its_own_slowest_rank():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank_seconds(0.25) == 0.25
    assert bench.whole_job_value(10.0, 1, 0.5) == 20.0


def test_reference_arm_under_a_two_rank_launch_prints_once():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", "29533", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "c2_llada"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
