"""N > 1: replicas only.  The aggregation bench.py applies (max of times, sum of tokens) with two
gloo ranks on the CPU, and the reference arm's rule that only rank 0 reports."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = [100.0, 130.0][rank]          # rank 1 is slower
    e2e = [110.0, 105.0][rank]
    out = bench.aggregate_replicas(ms, e2e, [50, 70][rank], [40, 45][rank], world, "cpu")
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, out))


def test_aggregation_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(2):
        assert got[r] == (130.0, 110.0, 120.0, 85.0)      # max, max, sum, sum on every rank


def test_single_replica_is_passed_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_replicas(1.0, 2.0, 3, 4, 1, "cpu") == (1.0, 2.0, 3, 4)


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "tiny-k2-ctx32", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "tiny-k2-ctx32", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=300)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
