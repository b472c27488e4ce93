"""Worker of tests/test_multiprocess.py::test_launcher_starts_replicas: what one replica of `bench.py --gpus N`
does around its measurement, with the measurement replaced by a fixed time per rank and gloo in place of NCCL.
Started by bench.spawn_replicas with the environment of a torchrun launch."""
import json
import os
import sys

import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert int(os.environ["LOCAL_RANK"]) == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
dist.init_process_group("gloo", rank=rank, world_size=world)
ms = bench.max_over_ranks([2.0 + rank])[0]          # the slowest replica sets the step time
if rank == 0:
    with open(sys.argv[1], "w") as f:
        json.dump({"n_gpus": world, "ms_per_step": ms, "value": bench.aggregate_value(4.0e9, ms, world)}, f)
dist.barrier()
dist.destroy_process_group()
