"""Host-side logic of `bench.py --gpus N` (independent replicas, no collective on the data path):
two CPU processes over gloo check the max-over-ranks timing and the whole-job figure, and the
reference arm's rule that only rank 0 works."""
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        slowest = bench.max_over_ranks(mine, world, torch.device("cpu"))
        out.put((rank, slowest, bench.us_per_layer(slowest, 5, 32, world), bench.replica_seed(20778, rank)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_rank_and_the_whole_job_value():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]                      # both see the slowest rank's time
    assert got[0][2] == pytest.approx(15.0 / 5 * 1e3 / (32 * 2))    # two replicas did twice the layers
    assert got[0][3] != got[1][3]                                   # each replica has its own sequence


def test_single_process_needs_no_process_group():
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu")) == 7.5
    assert bench.us_per_layer(8.0, 10, 32, 1) == pytest.approx(25.0)


def test_reference_arm_runs_on_rank_0_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
