"""The benchmark's multi-rank bookkeeping (replicas, no data-path collective): slowest rank's time, whole-job
aggregate.  Runs as two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    out[rank] = (ms, bench.whole_job_gbs(3e9, ms, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1]
    ms, gbs = out[0]
    assert ms == 15.0
    assert abs(gbs - 2 * 3e9 / 15e-3 / 1e9) < 1e-9


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu")) == 7.5
    assert bench.whole_job_gbs(1e9, 1.0, 1) == 1000.0


def test_gpus_flag_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher re-executes itself under the launcher with two ranks (here: the
    CPU-only rank plumbing, gloo): rank 0 prints one line for a two-rank job with the slowest rank's time."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-ranks"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 11.0
    assert abs(lines[0]["value"] - 2 * 1e9 / 11e-3 / 1e9) < 1e-9
