"""The N > 1 path of the benchmark on CPU: world size 2 over gloo.  Rows are
independent, so ranks exchange nothing on the data path; what exists is the
timing aggregation (max over ranks, whole-job rate) and the rule that only rank
0 reports."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.rank_info() == (rank, rank, world)
    mine = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]
    got = bench.reduce_max(mine)
    dist.barrier()
    q.put((rank, got, bench.whole_job_rate(world, 4096, 10, got[0])))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, rate in results:
        assert got == [15.0, 3.0, 7.0]  # every rank sees the slowest rank's time
        assert rate == pytest.approx(2 * 4096 * 10 / 15e-3)


def test_single_process_reduce_is_identity():
    import bench

    assert bench.reduce_max([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_rate(1, 100, 2, 1000.0) == 200.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "tiny", "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    r0 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--workload", "tiny", "--steps", "2", "--warmup", "1"], env=env0, capture_output=True,
                        text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["value"] > 0 and line["e2e"]["value"] == line["value"] and line["config"]["workload"] == "tiny"
