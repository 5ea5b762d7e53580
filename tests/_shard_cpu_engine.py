"""Test infrastructure: a CPU stand-in for one rank of paper_1905_10395_b200.sharded, built from the oracle's
election and update on the rank's rows plus the guest row (EXTERNAL objective).  It has the same four-piece
interface as the CUDA engine, so the exchange logic (who owns the global leader, which row travels where) can
be run on CPU tensors: in one process, or under torch.distributed with the gloo backend."""
import numpy as np
import torch

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200.sharded import Shard, argmin_by_rule


class CpuShardEngine:
    def __init__(self, w, rank, world):
        self.w, self.shard = w, Shard(w.group_of, w.G, rank, world)
        sh = self.shard
        self.x_np = sh.rows(w.x0, w.ld)
        self.x = torch.from_numpy(self.x_np)              # shares memory: collectives write straight into x_np
        self.g = sh.rows(w.arrays["g"], w.ld)
        self.ring = w.arrays["loss_ring"]
        self.t = 0
        self.n_elections = 0
        self.ll = None
        self.gl = -1
        self._best_local = -1
        self.global_leader_global = None
        self.local_leaders_global = None

    def is_pull_step(self):
        return self.t % self.w.tau == 0

    def phase_local(self):
        if not self.is_pull_step():
            return None
        sh = self.shard
        loss = self.ring[self.n_elections % self.ring.shape[0]][sh.workers]
        self.n_elections += 1
        full = np.concatenate([loss, np.array([np.nan], np.float32)]).astype(np.float32)
        self.ll, _ = orc.elect(full, sh.group_of_local, sh.G_local + 1)
        self.local_leaders_global = sh.workers[self.ll[: sh.G_local]]
        p = argmin_by_rule(loss, sh.workers)
        self._best_local = p
        return float(loss[p]), int(sh.workers[p])

    def leader_row(self):
        return self.x[self._best_local]

    def guest_row(self):
        return self.x[self.shard.guest]

    def phase_global(self, winner_rank, winner_index):
        self.gl = self._best_local if winner_rank == self.shard.rank else self.shard.guest
        self.global_leader_global = int(winner_index)
        self.finish_step()

    def finish_step(self):
        w, pull = self.w, self.is_pull_step()
        orc.update(self.x_np, self.g, self.shard.group_of_local, self.ll if pull else (), self.gl if pull else -1,
                   w.eta, w.lambda_l, w.lambda_g, pull)
        self.t += 1

    def x_local(self):
        return self.x_np[: self.shard.P_local].copy()
