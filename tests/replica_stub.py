"""A stand-in rank for the launcher test: what one replica of bench.py does between its steps, without a GPU.

Started by bench.launch_replicas with the rank environment of a real run; joins a gloo group over that environment,
aggregates a made-up step time and token count the way the benchmark does, and rank 0 writes the result.
Usage: replica_stub.py OUT_FILE
"""
import json
import sys
from pathlib import Path

import torch.distributed as dist

sys.path.insert(0, str(Path(__file__).resolve().parents[1]))
import bench  # noqa: E402

rank, local_rank, world = bench.dist_env()
assert local_rank == rank
dist.init_process_group("gloo")                       # rendezvous from MASTER_ADDR / MASTER_PORT / RANK / WORLD_SIZE
ms, tokens = bench.aggregate_over_ranks(2.0 + rank, 1000 * (rank + 1), world, "gloo")
dist.barrier()
if rank == 0:
    Path(sys.argv[1]).write_text(json.dumps({"n_gpus": world, "ms": ms, "tokens": tokens}))
dist.destroy_process_group()
