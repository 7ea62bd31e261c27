"""The N > 1 path is N independent replicas; what crosses ranks is the timing aggregation and the reference arm's
rank-0-only rule.  Both run here as two gloo processes on the CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2510_04476_b200.replicas import max_over_ranks, whole_job_rate
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = max_over_ranks(1.0 + rank, dist)                     # rank 1 is the slow one
    dist.barrier()
    q.put((rank, ms, whole_job_rate(32.0, ms, world)))
    dist.destroy_process_group()


def test_timing_is_the_max_over_ranks_and_the_rate_counts_every_replica():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [2.0, 2.0]
    assert all(abs(g[2] - 2 * 32.0 / 2e-3) < 1e-6 for g in got)


def test_single_process_needs_no_group():
    from paper_2510_04476_b200.replicas import max_over_ranks
    assert max_over_ranks(3.5) == 3.5


def test_reference_arm_under_two_ranks_prints_one_line():
    port = 31500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "cfg1_tiny"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
