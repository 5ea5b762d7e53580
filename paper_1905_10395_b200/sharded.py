"""Groups on several devices: the paper's own mapping (Section 2.2: a group of workers is a compute node, the
local leader is shared inside the node, the global leader across nodes, less often).

Each rank owns whole groups.  Everything inside a rank is the single-device path unchanged: the rank's handle
holds its workers plus one extra row, the *guest row*, in a group of its own.  On a pull step

  1. every rank evaluates its workers' election losses and elects its local leaders (``lsgd_elect``);
  2. the ranks exchange (best local loss, global index of that worker) -- a few bytes per rank;
  3. the rank that owns the global leader sends that worker's parameters (d floats) to the others, which receive
     them INTO THEIR OWN MEMORY (the guest row) -- the only bulk transfer, once per period, as in the paper;
  4. every rank points its global leader at the local winner or at the guest row (``lsgd_set_leaders``) and
     takes the fused step; the update kernel reads nothing but local memory.

The result equals the single-device run bit for bit: the losses are per worker, the election rule is the same
total order (-inf < finite < +inf < NaN, -0 == +0, ties to the lowest GLOBAL worker index), and the update of a
row depends only on that row, its gradient and the two leader rows.

The exchange is written against ``torch.distributed`` (NCCL between GPUs, gloo in the CPU tests) and, for
emulating several ranks inside one process, as ``run_lockstep``.  Objectives: EXTERNAL and QUADRATIC."""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

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


def _order_key(loss: float, index: int) -> Tuple[int, float, int]:
    """Sort key of the election's total order: NaN after +inf, -0 == +0, then the lower worker index."""
    v = float(np.float32(loss))
    if v != v:
        return (1, 0.0, int(index))
    return (0, v + 0.0, int(index))


def argmin_by_rule(loss: Sequence[float], indices: Sequence[int]) -> int:
    """Position (into the given sequences) of the election winner among (loss, worker index) pairs."""
    keys = [_order_key(l, i) for l, i in zip(loss, indices)]
    return min(range(len(keys)), key=lambda p: keys[p])


def pick_global_leader(best_loss: Sequence[float], best_index: Sequence[int]) -> int:
    """Given every rank's best (loss, GLOBAL worker index), the rank that owns the global leader."""
    return argmin_by_rule(best_loss, best_index)


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
        self.local_leaders_global: Optional[np.ndarray] = None
        self.global_leader_global: Optional[int] = None
        self._best_local = -1

    # -- the four pieces of a step
    def is_pull_step(self) -> bool:
        return self.t % self.w.tau == 0

    def phase_local(self) -> Optional[Tuple[float, int]]:
        """Gradient; on a pull step also the local election.  Returns this rank's best (loss, global index)."""
        sh = self.shard
        batch = self.batches[self.t % len(self.batches)] if self.batches else None
        self.lsgd.grad(batch)
        if not self.is_pull_step():
            return None
        if self.w.objective == "external":
            slot = self.n_elections % self.loss_ring.shape[0]
            self.lsgd.elect(self.loss_ring[slot])
            loss = self.loss_ring_host[slot, : sh.P_local]
        else:
            self.lsgd.elect(None)
            loss = self.lsgd.loss()[: sh.P_local]
        self.n_elections += 1
        ll, _ = self.lsgd.leaders()
        self.local_leaders_global = sh.workers[ll[: sh.G_local]]
        p = argmin_by_rule(loss, sh.workers)
        self._best_local = p
        return float(loss[p]), int(sh.workers[p])

    def leader_row(self):
        """This rank's best worker's parameters (what it sends if it owns the global leader)."""
        return self.x[self._best_local]

    def guest_row(self):
        """Where a global leader owned by another rank is received."""
        return self.x[self.shard.guest]

    def phase_global(self, winner_rank: int, winner_index: int) -> None:
        """Point the global leader at the local winner or at the guest row, then take the step."""
        mine = winner_rank == self.shard.rank
        self.lsgd.set_leaders(None, self._best_local if mine else self.shard.guest)
        self.global_leader_global = int(winner_index)
        self.finish_step()

    def finish_step(self) -> None:
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
    """One step of one rank under torch.distributed (one process per device).  The engine's rows must live where
    the process group can send them (CUDA tensors for NCCL, CPU tensors for gloo)."""
    import torch
    import torch.distributed as dist
    best = engine.phase_local()
    if best is None:
        engine.finish_step()
        return
    world = dist.get_world_size(group)
    row = engine.leader_row()
    mine = torch.tensor([best[0]], dtype=torch.float32, device=row.device)
    idx = torch.tensor([best[1]], dtype=torch.int64, device=row.device)
    losses = [torch.empty_like(mine) for _ in range(world)]
    indices = [torch.empty_like(idx) for _ in range(world)]
    dist.all_gather(losses, mine, group=group)
    dist.all_gather(indices, idx, group=group)
    best_loss = [float(t.item()) for t in losses]
    best_index = [int(t.item()) for t in indices]
    winner = pick_global_leader(best_loss, best_index)
    # the winner's row goes into every other rank's own memory; the update kernel then reads local memory only
    buf = row if winner == dist.get_rank(group) else engine.guest_row()
    dist.broadcast(buf, src=dist.get_global_rank(group, winner) if group is not None else winner, group=group)
    engine.phase_global(winner, best_index[winner])


def run_lockstep(engines: Sequence, steps: int) -> None:
    """Several ranks inside one process (any engines whose rows can be copied with ``copy_``): the same
    protocol with the exchange done by hand.  No rank's kernels wait on another's, so this is also valid on a
    single device."""
    for _ in range(steps):
        bests = [e.phase_local() for e in engines]
        if bests[0] is None:
            for e in engines:
                e.finish_step()
            continue
        winner = pick_global_leader([b[0] for b in bests], [b[1] for b in bests])
        src = engines[winner].leader_row()
        for r, e in enumerate(engines):
            if r != winner:
                e.guest_row().copy_(src)
        for e in engines:
            e.phase_global(winner, bests[winner][1])
