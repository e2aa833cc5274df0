"""The N > 1 path on CPU (gloo, two processes): the benchmark's replicas share nothing but the timing reduction, and
the reference arm prints exactly one line under a multi-process launch."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # rank r measured (10 + 5 r) ms on device-resident inputs and (20 - 3 r) ms end to end
    got = bench.max_over_ranks([10.0 + 5.0 * rank, 20.0 - 3.0 * rank], dist, torch.device("cpu"))
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_times_are_the_maximum_over_ranks_and_throughput_is_the_whole_job():
    torch = pytest.importorskip("torch")
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    import bench
    world, port = 2, 29517
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        got = dict(out)
    assert got[0] == [15.0, 20.0] and got[1] == [15.0, 20.0]
    # two replicas of 2112-token steps, 4 steps each, slowest rank 15 ms: the job served 2 * 4 * 2112 tokens in 15 ms
    assert bench.aggregate_tokens_per_s(2, 2112, 4, 15.0) == pytest.approx(2 * 4 * 2112 / 0.015)
    assert bench.max_over_ranks([3.0, 4.0], None, None) == [3.0, 4.0]


def test_reference_arm_under_a_two_process_launch_prints_one_line():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29518", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0", "--workload", "cfg0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def test_self_launch_command_starts_one_rank_per_gpu():
    """`bench.py --gpus N` without a launcher around it starts N ranks itself; the command it builds is checked here
    with the CPU arm in place of the GPU arm (two gloo-free ranks, rank 0 prints the single line)."""
    import argparse
    sys.path.insert(0, ROOT)
    import bench
    args = argparse.Namespace(gpus=2, forward=["--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "cfg0",
                                               "--impl", "reference"])
    cmd = bench.replica_launch_command(args, 29519)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "2"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29519"
    assert os.path.basename(cmd[cmd.index("--master-port") + 2]) == "bench.py"
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
