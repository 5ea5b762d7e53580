"""Test infrastructure: a CPU stand-in for one rank of paper_1905_10395_b200.sharded, built from the oracle's
election and update on the rank's rows plus the guest row (EXTERNAL objective).  It has the same interface as the
CUDA engine, so the exchange logic (who owns the global leader, which row travels where) can be run on CPU
tensors: in one process, or under torch.distributed with the gloo backend.  The cross-rank election keys are
packed here independently of the CUDA library (same published format: orderable float bits, then the global
worker index), and ``argmin_by_rule`` is the plain restatement of the rule that the tests check both against."""
import numpy as np
import torch

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200.sharded import Shard


def _order_key(loss, index):
    """Sort key of the election's total order: NaN after +inf, -0 == +0, then the lower worker index."""
    v = float(np.float32(loss))
    if v != v:
        return (1, 0.0, int(index))
    return (0, v + 0.0, int(index))


def argmin_by_rule(loss, indices) -> int:
    """Position (into the given sequences) of the election winner among (loss, worker index) pairs."""
    keys = [_order_key(l, i) for l, i in zip(loss, indices)]
    return min(range(len(keys)), key=lambda p: keys[p])


def pack_key(loss, global_index) -> int:
    """(orderable(loss) << 32) | global index as an unsigned 64-bit integer: floats map monotonically to
    uint32 (negative: all bits flipped; non-negative: sign bit set), -0 counts as +0, NaN sorts last."""
    v = np.float32(loss)
    if v != v:
        o = 0xFFFFFFFF
    else:
        u = int((v + np.float32(0.0)).view(np.uint32))
        o = (~u) & 0xFFFFFFFF if u & 0x80000000 else u | 0x80000000
    return (o << 32) | int(global_index)


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
        self._key = torch.zeros(1, dtype=torch.int64)

    def is_pull_step(self):
        return self.t % self.w.tau == 0

    def begin_step(self):
        if not self.is_pull_step():
            return False
        sh = self.shard
        loss = self.ring[self.n_elections % self.ring.shape[0]][sh.workers]
        self.n_elections += 1
        full = np.concatenate([loss, np.array([np.nan], np.float32)]).astype(np.float32)
        self.ll, _ = orc.elect(full, sh.group_of_local, sh.G_local + 1)
        self.local_leaders_global = sh.workers[self.ll[: sh.G_local]]
        p = argmin_by_rule(loss, sh.workers)
        self._best_local = p
        self._key[0] = int(np.uint64(pack_key(loss[p], sh.workers[p])).astype(np.int64))
        return True

    def key(self):
        return self._key

    def new_keys(self, world):
        return torch.empty(world, dtype=torch.int64)

    def pick_global(self, keys, world):
        u = keys.numpy().astype(np.int64).view(np.uint64)
        winner = int(np.argmin(u))                        # first minimum: the lowest rank among equal keys
        self.gl = self._best_local if winner == self.shard.rank else self.shard.guest
        self.global_leader_global = int(u[winner] & np.uint64(0xFFFFFFFF))
        return winner, self.global_leader_global

    def leader_row(self):
        return self.x[self._best_local]

    def guest_row(self):
        return self.x[self.shard.guest]

    def finish_step(self):
        w, pull = self.w, self.is_pull_step()
        orc.update(self.x_np, self.g, self.shard.group_of_local, self.ll if pull else (), self.gl if pull else -1,
                   w.eta, w.lambda_l, w.lambda_g, pull)
        self.t += 1

    def x_local(self):
        return self.x_np[: self.shard.P_local].copy()
