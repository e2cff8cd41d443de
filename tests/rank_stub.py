"""A stand-in rank program for the launcher test: what bench.py's ranks do around their step, on CPU.
Every rank joins a gloo group from the environment the launcher gave it, the ranks reduce a time to its maximum,
and rank 0 prints one JSON line with the rank count."""
import json
import os
import sys

import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2403_11805_b200 import sharding  # noqa: E402

if __name__ == "__main__":
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert int(os.environ["LOCAL_RANK"]) == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
    dist.init_process_group("gloo")
    ms = sharding.max_over_ranks([10.0 + rank], dist)[0]
    dist.barrier()
    if len(sys.argv) > 1 and sys.argv[1] == "--fail" and rank == world - 1:
        sys.exit(3)
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ms_per_step": ms, "argv": sys.argv[1:]}))
    dist.destroy_process_group()
