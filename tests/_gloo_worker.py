"""Helper launched by tests/test_bench_host.py under torchrun (gloo, CPU): exercises the N > 1 host
logic of bench.py -- rank environment, max-over-ranks of the timing, whole-job aggregation."""
import json
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402

rank, world, local = bench.dist_env()
dist.init_process_group("gloo")
elapsed = 10.0 * (rank + 1)                       # rank r "took" 10 (r + 1) ms
slowest = bench.max_over_ranks(elapsed, world)
value = bench.aggregate(1000.0, slowest, world)   # every replica processed 1000 units
dist.barrier()
if rank == 0:
    print(json.dumps({"world": world, "slowest_ms": slowest, "value": value}), flush=True)
dist.destroy_process_group()
