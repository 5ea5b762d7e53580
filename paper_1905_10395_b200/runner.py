"""Drives the C ABI over a `inputs.Workload`: uploads the arrays with torch, creates the handle and
issues grad / elect / step in the order of one synchronous LSGD step.  Marshalling only."""
from __future__ import annotations

import ctypes as C
from typing import List, Optional

import numpy as np
import torch

from . import api
from .inputs import Workload


class Population:
    def __init__(self, w: Workload, *, fused_quadratic: bool = False, arithmetic: int = api.ARITH_FP64,
                 device: str = "cuda:0", x: Optional[torch.Tensor] = None, g: Optional[torch.Tensor] = None,
                 upload_noise: bool = True, flags: int = 0, algorithm1: Optional[dict] = None,
                 stream: Optional["torch.cuda.Stream"] = None, momentum: Optional[float] = None,
                 weight_decay: float = 0.0, eagd: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU path)")
        self.w = w
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.dev)
        dev = self.dev
        self.x = x if x is not None else torch.from_numpy(w.x0).to(dev)
        self.g = g
        self.batches: List[Optional[torch.Tensor]] = []
        self.loss_ring: Optional[torch.Tensor] = None
        self._keep = []
        desc = None
        A = w.arrays
        if w.objective == "external":
            obj = api.OBJ_EXTERNAL
            if self.g is None:
                self.g = torch.from_numpy(A["g"]).to(dev)
            self.loss_ring = torch.from_numpy(A["loss_ring"]).to(dev)
        elif w.objective == "quadratic":
            obj = api.OBJ_QUADRATIC
            self.a = torch.from_numpy(A["a"]).to(dev)
            self.b = torch.from_numpy(A["b"]).to(dev)
            desc = api.QuadraticDesc(self.a.data_ptr(), self.b.data_ptr(), float(w.meta["sigma"]))
            if upload_noise and A.get("noise") is not None:
                self.batches = [torch.from_numpy(n).to(dev) for n in A["noise"]]
            if not fused_quadratic and self.g is None:
                self.g = torch.empty_like(self.x)
        elif w.objective == "matcomp":
            obj = api.OBJ_MATCOMP
            m = w.meta
            self.obs_r = torch.from_numpy(A["obs_r"]).to(dev)
            self.obs_c = torch.from_numpy(A["obs_c"]).to(dev)
            self.obs_v = torch.from_numpy(A["obs_v"]).to(dev)
            self.held = torch.from_numpy(A["heldout_pos"]).to(dev)
            # the gradient accumulator is the caller's, like every large buffer
            self.scratch = torch.empty(api.matcomp_scratch_bytes(w.P, w.ld), dtype=torch.uint8, device=dev)
            desc = api.MatcompDesc(m["n_rows"], m["n_cols"], m["rank"], len(A["obs_r"]), self.obs_r.data_ptr(),
                                   self.obs_c.data_ptr(), self.obs_v.data_ptr(), m["batch"], len(A["heldout_pos"]),
                                   self.held.data_ptr(), self.scratch.data_ptr(), self.scratch.numel())
            self.batches = [torch.from_numpy(np.ascontiguousarray(p)).to(dev) for p in A["batch_pos"]]
            if self.g is None:
                self.g = torch.empty_like(self.x)
        elif w.objective == "psd":
            obj = api.OBJ_PSD_COMPLETION
            self.M = torch.from_numpy(A["M"]).to(dev)
            nbytes = api.psd_scratch_bytes(w.meta["r"], w.P, w.ld)
            self.scratch = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=dev)
            desc = api.PsdDesc(w.meta["n"], w.meta["r"], self.M.data_ptr(), self.scratch.data_ptr() if nbytes else None, nbytes)
            if self.g is None:
                self.g = torch.empty_like(self.x)
        elif w.objective == "mlp":
            obj = api.OBJ_MLP
            m = w.meta
            self.pool_x = torch.from_numpy(A["pool_x"]).to(dev)
            self.pool_y = torch.from_numpy(A["pool_y"]).to(dev)
            self.held_x = torch.from_numpy(A["held_x"]).to(dev)
            self.held_y = torch.from_numpy(A["held_y"]).to(dev)
            nbytes = api.mlp_scratch_bytes(m["dims"], w.P, m["batch"], len(A["held_y"]))
            self.scratch = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
            sp = (self.scratch.data_ptr() + 1023) // 1024 * 1024
            desc = api.MlpDesc((C.c_int32 * 4)(*m["dims"]), m["batch"], len(A["pool_y"]), self.pool_x.data_ptr(),
                               self.pool_y.data_ptr(), len(A["held_y"]), self.held_x.data_ptr(),
                               self.held_y.data_ptr(), sp, nbytes, int(m.get("loss_window", 0)))
            self.batches = [torch.from_numpy(np.ascontiguousarray(p)).to(dev) for p in A["batch_idx"]]
            if self.g is None:
                self.g = torch.empty_like(self.x)
        else:
            raise ValueError(w.objective)
        extra = {}
        self.alg1 = algorithm1
        if algorithm1 is not None:
            # the paper's Algorithm 1 schedule: dict(gamma_l=, gamma_g=, tau_g=)
            self.leader_copies = torch.zeros((w.G + 1, w.ld), dtype=torch.float32, device=dev)
            flags |= api.FLAG_ALGORITHM1
            extra = dict(gamma_l=algorithm1["gamma_l"], gamma_g=algorithm1["gamma_g"], tau_g=algorithm1["tau_g"],
                         leader_copies=self.leader_copies)
        self.eagd = bool(eagd)
        if self.eagd:
            # elastic averaging instead of leaders: row G of the copies buffer is the center variable
            self.leader_copies = torch.zeros((w.G + 1, w.ld), dtype=torch.float32, device=dev)
            flags |= api.FLAG_EAGD
            extra = dict(leader_copies=self.leader_copies)
        self.v = None
        if momentum is not None:
            # Section 4.1 optimiser: Nesterov momentum + weight decay; the buffers start at zero
            self.v = torch.zeros_like(self.x)
            extra.update(v=self.v, momentum=momentum, weight_decay=weight_decay)
        cfg, keep = api.make_config(P=w.P, G=w.G, group_of=w.group_of, d=w.d, ld=w.ld, eta=w.eta,
                                    lambda_l=w.lambda_l, lambda_g=w.lambda_g, tau=w.tau, objective=obj, desc=desc,
                                    x=self.x, g=self.g, stream=self.stream.cuda_stream, arithmetic=arithmetic,
                                    flags=flags, **extra)
        self._keep.append(keep)
        torch.cuda.synchronize(self.dev)          # uploads were made on torch's current stream
        self.lsgd = api.Lsgd(cfg, keep)
        self.t = 0
        self.n_elections = 0
        self.history: List[dict] = []

    # one synchronous step, in the order gradient -> (election loss, election) -> update
    def _elect(self, forced_loss, record):
        if forced_loss is not None:
            self.lsgd.elect(forced_loss)
        elif self.loss_ring is not None:
            self.lsgd.elect(self.loss_ring[self.n_elections % self.loss_ring.shape[0]])
        else:
            self.lsgd.elect(None)
        self.n_elections += 1
        if record:
            ll, gl = self.lsgd.leaders()
            self.history.append({"t": self.t, "ll": ll, "gl": gl, "loss": self.lsgd.loss()})

    def _step_algorithm1(self, forced_loss, record):
        # initialise the leaders at x_0; then: gradient + step (small pulls), and the communication when due
        if self.t == 0 and self.n_elections == 0:
            self._elect(None, record)
        batch = self.batches[self.t % len(self.batches)] if self.batches else None
        self.lsgd.grad(batch)
        self.lsgd.step()
        self.t += 1
        if self.t % self.w.tau == 0 or self.t % self.alg1["tau_g"] == 0:
            self._elect(forced_loss, record)

    def step(self, forced_loss: Optional[torch.Tensor] = None, record: bool = False) -> None:
        if self.alg1 is not None:
            return self._step_algorithm1(forced_loss, record)
        w = self.w
        if self.eagd:
            self.lsgd.grad(self.batches[self.t % len(self.batches)] if self.batches else None)
            self.lsgd.step()
            self.t += 1
            return
        batch = self.batches[self.t % len(self.batches)] if self.batches else None
        self.lsgd.grad(batch)
        if self.t % w.tau == 0:
            if forced_loss is not None:
                self.lsgd.elect(forced_loss)
            elif self.loss_ring is not None:
                self.lsgd.elect(self.loss_ring[self.n_elections % self.loss_ring.shape[0]])
            else:
                self.lsgd.elect(None)
            self.n_elections += 1
            if record:
                ll, gl = self.lsgd.leaders()
                self.history.append({"t": self.t, "ll": ll, "gl": gl, "loss": self.lsgd.loss()})
        self.lsgd.step()
        self.t += 1

    def run(self, steps: int, record: bool = False) -> None:
        for _ in range(steps):
            self.step(record=record)

    # ---- CUDA graphs: capture n whole steps once, replay them without per-launch host work
    def capture(self, n_steps: int):
        """Captures the next ``n_steps`` steps (a whole number of communication periods, starting at a
        period boundary, and a whole number of passes over the batch ring) into a CUDA graph.  The captured
        steps are not executed; ``replay`` runs them."""
        if self.alg1 is not None:
            raise ValueError("capture() drives the fused schedule only")
        if self.t % self.w.tau or n_steps % self.w.tau:
            raise ValueError("capture whole communication periods starting at t % tau == 0")
        if self.batches and n_steps % len(self.batches):
            raise ValueError("capture a whole number of passes over the batch ring")
        if self.loss_ring is not None and (n_steps // self.w.tau) % self.loss_ring.shape[0]:
            raise ValueError("capture a whole number of passes over the loss ring")
        if self.stream.cuda_stream == 0:
            raise ValueError("create the Population with stream=torch.cuda.Stream(): the default stream cannot be captured")
        t0, e0 = self.t, self.n_elections
        graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize(self.dev)
        # the library enqueues on the stream it was created with: capture on that very stream
        with torch.cuda.graph(graph, stream=self.stream):
            for _ in range(n_steps):
                self.step()
        # nothing ran yet; the library has counted the captured steps as enqueued (see replay)
        self._graph, self._graph_steps = graph, n_steps
        self.t, self.n_elections = t0, e0
        self._graph_lib_ahead = n_steps
        return graph

    def replay(self) -> None:
        self._graph.replay()
        if self._graph_lib_ahead:
            self._graph_lib_ahead = 0       # the capture already advanced the library's counter once
        else:
            self.lsgd.advance_step(self._graph_steps)
        self.t += self._graph_steps
        self.n_elections += self._graph_steps // self.w.tau

    def center_host(self) -> np.ndarray:
        """EAGD: the center variable."""
        torch.cuda.synchronize(self.dev)
        return self.leader_copies[self.w.G].cpu().numpy()

    def x_host(self) -> np.ndarray:
        torch.cuda.synchronize(self.dev)
        return self.x.cpu().numpy()

    def close(self) -> None:
        self.lsgd.destroy()
