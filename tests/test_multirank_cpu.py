"""World-size-2 checks of the benchmark's multi-rank host logic on CPU (gloo).

The path has no exchange step: every rank runs an independent replica of the workload, and the
only cross-rank traffic is the max-over-ranks of the measured times."""
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
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (10 + r, 5 - r) ms: the maximum is taken per entry, on every rank
    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], "cpu", world)
    q.put((rank, got, bench.replica_throughput(1000.0, got[0], world)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_replica_throughput_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, thr in res:
        assert got == [11.0, 5.0]                       # slowest rank per entry, same on both ranks
        assert abs(thr - 2 * 1000.0 / 11.0e-3) < 1e-6   # both replicas' units over the slowest time


def test_reference_arm_runs_on_rank0_only():
    """Under a multi-rank launch only rank 0 times the oracle; the others exit 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_single_rank_max_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 1.25], "cpu", 1) == [3.5, 1.25]
    assert json.dumps(bench.replica_throughput(4096, 2.0, 1)) == "2048000.0"
