"""A stand-in replica for the launcher test: joins a gloo group from the environment the launcher set,
pretends to have moved some bytes in some time, and lets rank 0 print the aggregate as one JSON line."""
import json
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2601_20309_b200 import metrics as M  # noqa: E402

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert int(os.environ["LOCAL_RANK"]) == rank
dist.init_process_group("gloo")
nbytes, ms = 4.0e9 + rank * 2.0e9, 50.0 + 25.0 * rank
value = M.replicas_gbs(nbytes, ms, dist)
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "value": value}), flush=True)
else:
    print("noise from another rank")            # must not reach the launcher's output
dist.destroy_process_group()
if len(sys.argv) > 1 and sys.argv[1] == "--fail-rank" and rank == int(sys.argv[2]):
    sys.exit(3)
