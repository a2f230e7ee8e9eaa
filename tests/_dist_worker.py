"""Worker of the multi-process bench test: runs the rank plumbing bench.py uses for N > 1
(process-group setup, barrier, max over ranks, whole-job aggregation) on the gloo backend."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import torch

import bench

rank, world, local = bench._dist_setup(int(os.environ["WORLD_SIZE"]))
bench._barrier(world)
ms_local = 10.0 + 2.5 * rank                    # the slowest rank sets the step time
ms = bench._max_over_ranks(ms_local, world, torch.device("cpu"))
bench._barrier(world)
print(json.dumps({"rank": rank, "world": world, "local": local, "ms": ms,
                  "tokens_per_s": world * 8192 / (ms * 1e-3)}), flush=True)
import torch.distributed as dist
dist.destroy_process_group()
