"""The N > 1 control flow of bench.py on CPU: two gloo ranks reduce their device timings with MAX,
every rank draws its own batch, and under torch.distributed.run only rank 0 prints the reference
arm's JSON line."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2608_17336_b200 import synth
    times = [10.0 + rank, 5.0 - rank, 1.0]
    got = bench.max_over_ranks(times, torch.device("cpu"), world)
    w = bench.rank_workload(synth.WORKLOADS["cfg1_tiny"], rank)
    dist.barrier()
    q.put((rank, got, w.seed))
    dist.destroy_process_group()


def test_max_over_ranks_and_rank_seeds_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29571, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == [11.0, 5.0, 1.0]
    assert res[0][2] != res[1][2]


def test_job_value_is_whole_job_throughput():
    import bench
    assert bench.job_value(1e12, 1, 1000.0) == 1.0
    assert bench.job_value(1e12, 8, 1000.0) == 8.0          # weak scaling: N ranks, N batches


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29572", os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "cfg1_tiny"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
