"""Groups on several devices: the paper's own mapping (Section 2.2: a group of workers is a compute node, the
local leader is shared inside the node, the global leader across nodes, less often).

Each rank owns whole groups.  Everything inside a rank is the single-device path unchanged: the rank's handle
holds its workers plus one extra row, the *guest row*, in a group of its own.  On a pull step

  1. every rank evaluates its workers' election losses, elects its local leaders (``lsgd_elect``) and packs its
     best own worker into an 8-byte key on the device (``lsgd_shard_best_key``);
  2. ONE all-gather of those keys; each rank's ``lsgd_shard_pick_global`` takes their minimum on the device,
     points its global leader at its own winner or at the guest row, and hands the host the winning rank -- the
     one host synchronisation of the step;
  3. the rank that owns the global leader sends that worker's parameters (d floats) to the others, which receive
     them INTO THEIR OWN MEMORY (the guest row) -- the only bulk transfer, once per period, as in the paper;
  4. every rank takes the fused step; the update kernel reads nothing but local memory.

The result equals the single-device run bit for bit: the losses are per worker, the election rule is the same
total order (-inf < finite < +inf < NaN, -0 == +0, ties to the lowest GLOBAL worker index), and the update of a
row depends only on that row, its gradient and the two leader rows.

The exchange is written against ``torch.distributed`` (NCCL between GPUs, gloo in the CPU tests) and, for
emulating several ranks inside one process, as ``run_lockstep``.  Objectives: EXTERNAL and QUADRATIC."""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np


# ------------------------------------------------------------------------------------- host logic ----
def partition_groups(G: int, world: int) -> List[range]:
    """Contiguous, near-equal split of the G groups over the ranks (earlier ranks get the extra ones)."""
    if world < 1 or G < world:
        raise ValueError("need at least one group per rank")
    base, extra = divmod(G, world)
    out, lo = [], 0
    for r in range(world):
        n = base + (1 if r < extra else 0)
        out.append(range(lo, lo + n))
        lo += n
    return out


class Shard:
    """Which workers of the global population a rank holds.  Local worker order is global order."""

    def __init__(self, group_of: np.ndarray, G: int, rank: int, world: int):
        group_of = np.asarray(group_of, dtype=np.int32)
        self.rank, self.world = rank, world
        self.groups = partition_groups(G, world)[rank]
        self.workers = np.nonzero((group_of >= self.groups.start) & (group_of < self.groups.stop))[0].astype(np.int64)
        self.P_local = int(len(self.workers))
        self.G_local = len(self.groups)
        # the handle's population: the local workers, then the guest row in a group of its own
        self.group_of_local = np.concatenate([group_of[self.workers] - self.groups.start,
                                              np.array([self.G_local], dtype=np.int32)]).astype(np.int32)
        self.guest = self.P_local

    def rows(self, a: np.ndarray, ld: int) -> np.ndarray:
        """[P, ld] global array -> [P_local + 1, ld] local array with a zero guest row."""
        out = np.zeros((self.P_local + 1, ld), dtype=a.dtype)
        out[: self.P_local] = a[self.workers]
        return out


# ------------------------------------------------------------------------------------ CUDA engine ----
class CudaShardEngine:
    """One rank's part of a workload (``inputs.make_external`` / ``make_quadratic``) on one CUDA device."""

    def __init__(self, w, rank: int, world: int, device: str = "cuda:0", arithmetic: int = 0):
        import torch
        from . import api
        if w.objective not in ("external", "quadratic"):
            raise ValueError("the sharded driver covers the EXTERNAL and QUADRATIC objectives")
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU path)")
        self.w, self.shard = w, Shard(w.group_of, w.G, rank, world)
        sh = self.shard
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.x = torch.from_numpy(sh.rows(w.x0, w.ld)).to(self.dev)
        self.t = 0
        self.n_elections = 0
        A = w.arrays
        self.g = None
        self.batches: list = []
        desc = None
        if w.objective == "external":
            self.g = torch.from_numpy(sh.rows(A["g"], w.ld)).to(self.dev)
            ring = np.full((A["loss_ring"].shape[0], sh.P_local + 1), np.nan, dtype=np.float32)
            ring[:, : sh.P_local] = A["loss_ring"][:, sh.workers]
            self.loss_ring_host = ring
            self.loss_ring = torch.from_numpy(ring).to(self.dev)
            obj = api.OBJ_EXTERNAL
        else:
            self.a = torch.from_numpy(A["a"]).to(self.dev)
            self.b = torch.from_numpy(A["b"]).to(self.dev)
            desc = api.QuadraticDesc(self.a.data_ptr(), self.b.data_ptr(), float(w.meta["sigma"]))
            if A.get("noise") is not None:
                self.batches = [torch.from_numpy(sh.rows(n, w.ld)).to(self.dev) for n in A["noise"]]
            obj = api.OBJ_QUADRATIC
        cfg, keep = api.make_config(P=sh.P_local + 1, G=sh.G_local + 1, group_of=sh.group_of_local, d=w.d, ld=w.ld,
                                    eta=w.eta, lambda_l=w.lambda_l, lambda_g=w.lambda_g, tau=w.tau, objective=obj,
                                    x=self.x, g=self.g, desc=desc, arithmetic=arithmetic,
                                    stream=torch.cuda.current_stream(self.dev).cuda_stream)
        self.lsgd = api.Lsgd(cfg, keepalive=(keep, desc))
        self.global_leader_global: Optional[int] = None
        self._best_local = -1
        self.global_index = torch.from_numpy(sh.workers.astype(np.int32)).to(self.dev)
        self._key = torch.zeros(1, dtype=torch.int64, device=self.dev)

    # -- the pieces of a step
    def is_pull_step(self) -> bool:
        return self.t % self.w.tau == 0

    def _make_current(self) -> None:
        # the library refuses calls on a handle while another device is current (engines of several devices may
        # live in one process, as in run_lockstep)
        import torch
        if torch.cuda.current_device() != self.dev.index:
            torch.cuda.set_device(self.dev)

    def begin_step(self) -> bool:
        """Gradient; on a pull step also the local election and this rank's key.  True on a pull step."""
        self._make_current()
        batch = self.batches[self.t % len(self.batches)] if self.batches else None
        self.lsgd.grad(batch)
        if not self.is_pull_step():
            return False
        if self.w.objective == "external":
            self.lsgd.elect(self.loss_ring[self.n_elections % self.loss_ring.shape[0]])
        else:
            self.lsgd.elect(None)
        self.n_elections += 1
        self.lsgd.shard_best_key(self.shard.P_local, self.global_index, self._key)
        return True

    def key(self):
        """This rank's best own worker as an 8-byte election key (a one-element int64 tensor on the device)."""
        return self._key

    def new_keys(self, world: int):
        import torch
        return torch.empty(world, dtype=torch.int64, device=self.dev)

    def pick_global(self, keys, world: int):
        """From all ranks' keys: the winning rank and the winner's global worker index; sets this rank's global
        leader (own winner or guest row) on the device.  The one host synchronisation of a pull step."""
        self._make_current()
        winner, gidx, self._best_local = self.lsgd.shard_pick_global(keys, world, self.shard.rank, self.shard.guest)
        self.global_leader_global = gidx
        return winner, gidx

    @property
    def local_leaders_global(self) -> np.ndarray:
        """Global indices of this rank's local leaders (reads them back: for checks, not part of a step)."""
        ll, _ = self.lsgd.leaders()
        return self.shard.workers[ll[: self.shard.G_local]]

    def leader_row(self):
        """This rank's best worker's parameters (what it sends if it owns the global leader)."""
        return self.x[self._best_local]

    def guest_row(self):
        """Where a global leader owned by another rank is received."""
        return self.x[self.shard.guest]

    def finish_step(self) -> None:
        self._make_current()
        self.lsgd.step()
        self.t += 1

    def x_local(self) -> np.ndarray:
        import torch
        torch.cuda.synchronize(self.dev)
        return self.x[: self.shard.P_local].cpu().numpy()

    def close(self) -> None:
        self.lsgd.destroy()


# -------------------------------------------------------------------------------------- exchange ----
def distributed_step(engine, group=None) -> None:
    """One step of one rank under torch.distributed (one process per device).  The engine's rows and keys must
    live where the process group can send them (CUDA tensors for NCCL, CPU tensors for gloo).  A pull step costs
    one all-gather of 8 bytes per rank, one host synchronisation and the broadcast of the leader's row."""
    import torch.distributed as dist
    if not engine.begin_step():
        engine.finish_step()
        return
    world = dist.get_world_size(group)
    keys = engine.new_keys(world)
    dist.all_gather(list(keys.view(world, 1).unbind(0)), engine.key(), group=group)
    winner, _ = engine.pick_global(keys, world)
    # the winner's row goes into every other rank's own memory; the update kernel then reads local memory only
    buf = engine.leader_row() if winner == dist.get_rank(group) else engine.guest_row()
    dist.broadcast(buf, src=dist.get_global_rank(group, winner) if group is not None else winner, group=group)
    engine.finish_step()


def run_lockstep(engines: Sequence, steps: int) -> None:
    """Several ranks inside one process (any engines whose rows can be copied with ``copy_``): the same
    protocol with the exchange done by hand.  No rank's kernels wait on another's, so this is also valid on a
    single device."""
    world = len(engines)
    for _ in range(steps):
        pulls = [e.begin_step() for e in engines]
        if not pulls[0]:
            for e in engines:
                e.finish_step()
            continue
        winners = []
        for e in engines:
            keys = e.new_keys(world)
            for r, other in enumerate(engines):
                keys[r:r + 1].copy_(other.key())
            winners.append(e.pick_global(keys, world)[0])
        winner = winners[0]
        assert all(v == winner for v in winners)
        src = engines[winner].leader_row()
        for r, e in enumerate(engines):
            if r != winner:
                e.guest_row().copy_(src)
        for e in engines:
            e.finish_step()
