"""Host-side logic of the multi-GPU benchmark, on CPU with gloo and two ranks: every rank draws its own
independent shard, the step time is the slowest rank's, the job throughput counts every shard, and only
rank 0 runs the reference arm."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np
    import torch
    import torch.distributed as dist
    import bench
    from paper_2605_07114_b200 import workloads as wl
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.make(bench.WORKLOAD, 256, seed=bench.shard_seed(rank))
    # shards are different draws of the same recipe
    sig = torch.tensor([float(w.alpha.sum()), float(w.c.sum())], dtype=torch.float64)
    sigs = [torch.zeros(2, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sigs, sig)
    assert not torch.equal(sigs[0], sigs[1])
    assert w.N == 256 and w.B == 24 * 256
    # the slowest rank sets the step time; throughput counts all shards
    local_ms = 2.0 + rank
    ms = bench.max_over_ranks(local_ms, world)
    assert ms == 3.0
    assert bench.job_throughput(w.N, world, ms) == 2 * 256 / 3e-3
    dist.barrier()
    dist.destroy_process_group()
    print("ok", rank)
""") % ROOT


def test_two_rank_sharding_and_timing_reduce(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(20000 + os.getpid() % 20000), str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2          # both ranks reached the end (their prints may interleave)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=120, env=env, cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_sample_size_is_bounded():
    sys.path.insert(0, ROOT)
    import bench
    N = 1 << 20
    for steps, warm in ((1, 0), (5, 2), (20, 5), (200, 10), (5000, 10)):
        n, why = bench.reference_sample_size(steps, warm, N)
        assert 1024 <= n <= N and n & (n - 1) == 0 and why
        # the whole run stays within the CPU time allowed for this arm (or sits at the floor of 1024 prompts)
        assert n * (steps + warm) * bench.ORACLE_US_PER_PROMPT * 1e-6 <= bench.REFERENCE_CPU_SECONDS or n == 1024
    # few enough steps: every step is the whole workload, the same one the repository's arm times
    assert bench.reference_sample_size(5, 2, N)[0] == N
