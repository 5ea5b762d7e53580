"""Helper launched by tests/test_sharded_host.py under torchrun (gloo, CPU, 2 ranks): runs the group-per-rank
exchange of paper_1905_10395_b200.sharded through torch.distributed with the CPU stand-in engine and compares
this rank's rows, bit for bit, with the single-population oracle."""
import json
import os
import sys

import numpy as np
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
from oracle import lsgd_oracle as orc  # noqa: E402
from paper_1905_10395_b200 import inputs, sharded  # noqa: E402
from tests._shard_cpu_engine import CpuShardEngine  # noqa: E402

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
steps = 9
w = inputs.make_external(10, 5, 333, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=steps, loss_ring=5, config_id=140)
w.arrays["loss_ring"][1, :] = 0.5                       # an all-tie election: the lowest global index must win
eng = CpuShardEngine(w, rank, world)
leaders = []
for _ in range(steps):
    pull = eng.is_pull_step()
    sharded.distributed_step(eng)
    if pull:
        leaders.append(eng.global_leader_global)
o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                   w.lambda_g, w.tau)
o.run(steps)
same = bool(np.array_equal(eng.x_local().view(np.uint32), o.x[eng.shard.workers].view(np.uint32)))
want = [h["gl"] for h in o.history]
sys.stdout.write(json.dumps({"rank": rank, "world": world, "rows_equal": same, "leaders": leaders, "want": want,
                             "workers": eng.shard.workers.tolist()}) + "\n")
sys.stdout.flush()
dist.barrier()
dist.destroy_process_group()
