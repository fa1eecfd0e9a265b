"""The N > 1 path of the benchmark on CPU: independent replicas, aggregated with gloo (world size 2).

The step has no exchange between GPUs, so `bench.py --gpus N` runs N replicas; the only cross-rank logic is the
aggregation of timings (slowest rank) and work (sum), which this test drives with two CPU processes, and the
launcher that starts the ranks when torchrun did not, which is run here with a stand-in rank on gloo.
"""
import json
import os
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parents[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, tokens = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 4096 * (rank + 1), world, "gloo")
    assert bench.dist_env()[0] == rank and bench.dist_env()[2] == world
    dist.barrier()
    out[rank] = (ms, tokens)
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_total_work():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29500 + os.getpid() % 1000, out), nprocs=world, join=True)
        assert dict(out) == {0: (15.0, 4096 * 3), 1: (15.0, 4096 * 3)}


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.aggregate_over_ranks(3.5, 100, 1, "gloo") == (3.5, 100)


def test_launcher_starts_the_ranks_with_a_torchrun_style_environment(tmp_path):
    """`bench.py --gpus 2` without torchrun: launch_replicas starts two processes that find each other."""
    sys.path.insert(0, str(ROOT))
    import bench
    out = tmp_path / "line.json"
    rc = bench.launch_replicas(2, [str(ROOT / "tests" / "replica_stub.py"), str(out)])
    assert rc == 0
    assert json.loads(out.read_text()) == {"n_gpus": 2, "ms": 3.0, "tokens": 3000}


def test_launcher_reports_a_failed_rank(tmp_path):
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.launch_replicas(2, ["-c", "import os, sys; sys.exit(3 if os.environ['RANK'] == '1' else 0)"]) == 3
