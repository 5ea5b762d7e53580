#!/usr/bin/env python
"""Benchmark of the LSGD step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c1] [--tau T]
    python bench.py --impl reference ...        # the CPU oracle, timed on the host cores

Default workload: the large fused-update stress (P = 16 workers in G = 4 groups, d = 2^26 fp32
parameters per worker, supplied gradients and election losses, tau = 1).  One step = election +
fused update over the whole population.  Prints ONE JSON line (rank 0).

With N > 1 (torchrun, one process per GPU) every rank runs an independent replica of the workload:
the method keeps the whole population on one device and has no exchange step, so there is no
collective on the data path -- only the barrier and the max-over-ranks of the timing.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "lsgd_step_worker_params_per_s"
UNIT = "worker-params/s"


# ------------------------------------------------------------------------------------ helpers ----
def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def read_tensor_peak():
    """Dense bf16 tensor throughput for a kernel timed inside a long step (the sustained figure)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        if "bf16_tflops_sustained" in p:
            return float(p["bf16_tflops_sustained"]), "measured (sustained)"
    return 1400.0, "fallback (sustained)"


def mlp_algorithmic_bytes(dims):
    """Bytes ONE worker's fused gradient + SGD step cannot avoid moving, whatever the batch: the bf16 weights read
    by the forward products (2 B per parameter), W2 and W3 read again by the back-propagation products, the fp32
    master parameters read and rewritten by the step (4 + 4 B) and their new bf16 copy (2 B).  Activations, the
    batch and the deltas are left out (they are small and can stay on chip).  24.5 MB for 784-1024-1024-10."""
    d0, d1, d2, d3 = [int(v) for v in dims]
    n_w = d0 * d1 + d1 + d1 * d2 + d2 + d2 * d3 + d3
    return float(12 * n_w + 2 * (d1 * d2 + d2 * d3))


def mlp_step_bytes_flops(dims, batch):
    """Traffic model and tensor-core flops of ONE worker's fused gradient + SGD step as the kernels are split.

    Every operand is counted once per kernel that must read or write it: bf16 activations and shadow weights
    (2 B), the fp32 master weights read and rewritten by the step (4 + 4 B) plus their new bf16 shadow (2 B),
    the fp32 pool rows gathered into the bf16 batch.  The 10-wide head is counted with its fp32 weights."""
    d0, d1, d2, d3 = [int(v) for v in dims]
    B = int(batch)
    by = B * d0 * (4 + 2)                                    # gather
    by += d0 * d1 * 2 + B * (d0 + d1) * 2                    # H1 = relu(X W1^T + b1)
    by += d1 * d2 * 2 + B * (d1 + d2) * 2                    # H2
    by += d2 * d3 * 4 + B * d2 * 2                           # head forward
    by += d2 * d3 * (4 + 4 + 2) + 2 * B * d2 * 2             # head backward: dH2 out, H2 in, W3 stepped
    by += d1 * d2 * 2 + B * (d2 + 2 * d1) * 2 + B * d1 * 2   # dH1 = (dH2 W2) masked by H1
    by += B * (d1 + d2) * 2 + d1 * d2 * (4 + 4 + 2)          # dW2 with the step in its epilogue
    by += B * (d1 + d2) * 2                                  # bias gradients (column sums)
    by += B * (d0 + d1) * 2 + d0 * d1 * (4 + 4 + 2)          # dW1 with the step in its epilogue
    fl = 2.0 * B * (2 * d0 * d1 + 3 * d1 * d2 + 2 * d2 * d3)
    return float(by), fl


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, device_index: int):
        self.proc = None
        self.lines = []
        self.idx = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        inside = [l for (ts, l) in self.lines if t0 - 0.05 <= ts <= t1 + 0.15] or [l for (_, l) in self.lines]
        for l in inside:
            f = [c.strip() for c in l.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except Exception:
                continue
            for name, v in zip(self.NAMES, f[3:7]):
                if v == "Active":
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def host_cores() -> int:
    """Cores this process may run on (the affinity mask where the platform has one, else the core count)."""
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def _threads_used() -> int:
    """Threads the oracle's NumPy can use: 1 for its element-wise loops; BLAS threads for matmuls."""
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def aggregate(per_rank_units: float, elapsed_ms_max: float, world: int) -> float:
    """Whole-job throughput: the units all ranks processed over the slowest rank's time."""
    return per_rank_units * world / (elapsed_ms_max * 1e-3)


def max_over_ranks(value: float, world: int, device=None) -> float:
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# --------------------------------------------------------------------------------- workloads ----
def workload_spec(args):
    wl = args.workload
    if wl == "c4":
        return dict(kind="external", cfg=4, P=16, G=4, d=args.d or (1 << 26), eta=0.01, lambda_l=0.1, lambda_g=0.05,
                    tau=args.tau or 1, name="C4 fused-update stress: P=16 G=4 d=2^26 fp32, supplied g and losses",
                    launches=(2, 1), momentum=getattr(args, "momentum", None),
                    weight_decay=getattr(args, "weight_decay", 0.0))
    if wl == "c1":
        return dict(kind="quadratic", cfg=1, P=64, G=8, d=1 << 20, eta=0.05, lambda_l=0.1, lambda_g=0.05,
                    tau=args.tau or 4, name="C1 multi-leader quadratic: P=64 G=8 d=2^20 fp32, noise sigma=0.01, "
                    "gradient fused into the update", launches=(3, 1))
    if wl == "c0":
        return dict(kind="quadratic", cfg=0, P=4, G=1, d=1024, eta=0.1, lambda_l=0.1, lambda_g=0.0, tau=args.tau or 1,
                    name="C0 single-leader quadratic: P=4 G=1 d=1024", launches=(3, 1))
    if wl == "c2":
        return dict(kind="matcomp", cfg=2, P=16, G=4, d=200000, eta=0.01, lambda_l=0.1, lambda_g=0.05,
                    tau=args.tau or 8, name="C2 matrix completion: P=16 G=4, 10000x10000 rank 10, batch 4096",
                    launches=(5, 3 if args.mlp_unfused_step else 2))
    if wl == "c3":
        return dict(kind="mlp", cfg=3, P=32, G=4, d=1863712, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=args.tau or 4,
                    name="C3 MLP population: P=32 G=4, 784-1024-1024-10, batch 128, bf16 GEMM fp32 accumulate",
                    launches=(15, 9 if args.mlp_unfused_step else 8))
    if wl == "psd":
        r = args.rank
        return dict(kind="psd", cfg=5, P=8, G=1, d=1000 * r, n=1000, r=r, eta=5e-4, lambda_l=0.2, lambda_g=0.0,
                    tau=args.tau or 1, name=f"PSD completion (the paper's experiment): 8 workers, n=1000, rank {r}, "
                    "eta 5e-4, lambda 1/5, tau 1",
                    # gradient (+ the combine of the two partial gradients up to rank 32), election, update
                    launches=(4, 3) if r <= 32 else (3, 2), eagd=bool(getattr(args, "eagd", False)))
    raise SystemExit("unknown workload")


# DRAM bytes per worker-parameter that the update kernels of the default workload moved in a one-pass
# hardware-counter capture of the full-size launch (dram read + write bytes divided by P * d = 2^30): reads are the
# algorithmic 8 B exactly (8.59 GB); writes 4.24-4.25 GB of the algorithmic 4.29 GB, the rest being lines still
# dirty in the 126 MB L2 when the kernel ends.  Quoted for that workload only (d = 2^26).
MEASURED_TRAFFIC_PER_WORKER_PARAM = {"pull": 11.95, "plain": 11.96}
NOMINAL_HBM_GBS = 7700.0     # the part's data-sheet HBM3e bandwidth, for context beside the measured copy bandwidth


def bytes_per_worker_param(spec):
    # update kernel: read x + read g (or noise) + write x; the fused quadratic adds a, b once per column;
    # the MLP update also writes the bf16 copy of the weights
    if spec["kind"] == "quadratic":
        return 12.0 + 8.0 / spec["P"]
    if spec["kind"] == "mlp":
        return 14.0
    return 12.0


# ------------------------------------------------------------------------------ CPU oracle leg ----
def oracle_sample_run(spec, steps, warmup, sample_cols, min_seconds=0.0):
    """Times the oracle, as it stands, on a bounded sample of the workload: a column sample for the
    element-wise objectives (same P, G, tau), the full problem for matrix completion, 4 of the
    workers for the MLP population.  With ``min_seconds`` the step count is raised (once, from a first
    timing) so that the timed work lasts about that long.  Returns (worker-params/s, seconds, description,
    steps timed)."""
    v, dt, what = _oracle_sample_once(spec, steps, warmup, sample_cols)
    if min_seconds > 0.0 and dt < 0.8 * min_seconds:
        steps = int(min(max(steps * min_seconds / max(dt, 1e-4), steps + 1), 20000))
        v, dt, what = _oracle_sample_once(spec, steps, warmup, sample_cols)
    return v, dt, what, steps


def _oracle_sample_once(spec, steps, warmup, sample_cols):
    from oracle import lsgd_oracle as orc
    from paper_1905_10395_b200 import inputs
    P = spec["P"]
    if spec["kind"] == "external":
        w = inputs.make_external(P, spec["G"], sample_cols, eta=spec["eta"], lambda_l=spec["lambda_l"],
                                 lambda_g=spec["lambda_g"], tau=spec["tau"], steps=steps, config_id=4)
        obj = orc.External(w.arrays["g"], w.arrays["loss_ring"])
        what = f"{P} workers x {sample_cols} of {spec['d']} columns"
    elif spec["kind"] == "quadratic":
        cols = min(sample_cols, spec["d"])
        w = inputs.make_quadratic(P, spec["G"], cols, eta=spec["eta"], lambda_l=spec["lambda_l"],
                                  lambda_g=spec["lambda_g"], tau=spec["tau"], steps=steps, sigma=0.01,
                                  noise_ring=2, config_id=1)
        obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.01, w.arrays["noise"])
        what = f"{P} workers x {cols} of {spec['d']} columns"
    elif spec["kind"] == "matcomp":
        w = inputs.config(2, steps=steps + warmup, tau=spec["tau"])
        m, A = w.meta, w.arrays
        obj = orc.MatComp(m["n_rows"], m["n_cols"], m["rank"], A["obs_r"], A["obs_c"], A["obs_v"], A["batch_pos"],
                          A["heldout_pos"])
        what = "the full workload"
    elif spec["kind"] == "psd":
        w = inputs.make_psd(P=P, n=spec["n"], r=spec["r"], steps=steps + warmup)
        obj = orc.PsdCompletion(spec["n"], spec["r"], w.arrays["M"])
        what = "the full workload"
    else:
        P = 4
        w = inputs.config(3, P=P, G=1, steps=steps + warmup, tau=spec["tau"], pool=8192)
        A = w.arrays
        segs, _ = inputs.mlp_layout(w.meta["dims"])
        obj = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="bf16emu")
        what = f"{P} of {spec['P']} workers (one group)"
    mom = spec.get("momentum") if spec["kind"] == "external" else None
    if spec.get("eagd"):
        o = orc.EagdOracle(w.x0, obj, w.eta, w.lambda_l, tau=w.tau)
    else:
        o = orc.LsgdOracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau, momentum=mom,
                           weight_decay=spec.get("weight_decay", 0.0))
    for _ in range(warmup):
        o.step()
    t0 = time.perf_counter()
    for _ in range(steps):
        o.step()
    dt = time.perf_counter() - t0
    return P * w.d * steps / dt, dt, what


def _all_cores_worker(spec, steps, sample_cols, slot, barrier, out):
    """One process of the all-cores leg: the oracle, as it stands, on this process's own column sample."""
    try:
        from oracle import lsgd_oracle as orc
        from paper_1905_10395_b200 import inputs
        P = spec["P"]
        kw = dict(eta=spec["eta"], lambda_l=spec["lambda_l"], lambda_g=spec["lambda_g"], tau=spec["tau"], steps=steps)
        if spec["kind"] == "external":
            w = inputs.make_external(P, spec["G"], sample_cols, config_id=400 + slot, **kw)
            obj = orc.External(w.arrays["g"], w.arrays["loss_ring"])
        else:
            w = inputs.make_quadratic(P, spec["G"], sample_cols, sigma=0.01, noise_ring=2, config_id=100 + slot, **kw)
            obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.01, w.arrays["noise"])
        o = orc.LsgdOracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)
        o.step()
        barrier.wait(timeout=600)
        t0 = time.perf_counter()
        for _ in range(steps):
            o.step()
        out.put((slot, P * w.d * steps, time.perf_counter() - t0))
    except Exception as exc:                                # the parent must not wait for a result that never comes
        out.put((slot, 0.0, float("nan"), repr(exc)))


def oracle_all_cores(spec, steps, sample_cols, n_proc=None):
    """The element-wise workloads on every host core: columns are independent once the leaders are known, so each
    of ``n_proc`` processes (spawned: no CUDA state is inherited) times the unchanged oracle on its own column
    sample, all starting together; the throughputs add up over the slowest process's time.  Returns
    (worker-params/s, seconds, processes) or None for the other workloads."""
    if spec["kind"] not in ("external", "quadratic"):
        return None
    import multiprocessing as mp
    n_proc = n_proc or host_cores()
    ctx = mp.get_context("spawn")
    barrier, out = ctx.Barrier(n_proc), ctx.Queue()
    cols = int(min(sample_cols, spec["d"]))
    procs = [ctx.Process(target=_all_cores_worker, args=(spec, steps, cols, k, barrier, out)) for k in range(n_proc)]
    for p in procs:
        p.start()
    got, deadline = [], time.time() + 1200
    while len(got) < n_proc:
        try:
            got.append(out.get(timeout=2))
        except Exception:
            # a child that died before it could report (import failure, out of memory) must not stall the bench
            if any(p.exitcode not in (None, 0) for p in procs) or time.time() > deadline:
                for p in procs:
                    if p.is_alive():
                        p.terminate()
                raise RuntimeError("all-cores oracle leg: a worker process ended without a result")
    for p in procs:
        p.join(timeout=60)
    bad = [g for g in got if len(g) > 3]
    if bad:
        raise RuntimeError(f"all-cores oracle leg failed: {bad[0][3]}")
    units, slowest = sum(g[1] for g in got), max(g[2] for g in got)
    return units / slowest, slowest, n_proc


def cpu_baseline_record(spec, value, cores, sample, all_cores=None):
    """The ``cpu_baseline`` object: the single-process figure and, for the element-wise workloads, the figure on
    all host cores; ``value`` / ``cores`` are the larger configuration's."""
    rec = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    if all_cores is not None:
        v, dt, n = all_cores
        rec = {"value": v, "unit": UNIT, "cores": n, "kind": "oracle",
               "sample": f"{n} processes, each: {sample.split(', ')[0]}; {dt:.1f} s",
               "single_core": {"value": value, "cores": cores, "sample": sample},
               "host_cores": host_cores()}
    return rec


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    spec = workload_spec(args)
    steps, warmup = args.steps, args.warmup
    sample = args.sample_cols or (1 << 20)      # about a quarter of a second of oracle work per C4 step
    value, dt, what, _ = oracle_sample_run(spec, steps, warmup, sample)
    cores = _threads_used() if spec["kind"] in ("mlp", "psd") else 1
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec["name"], "tau": spec["tau"],
                   "sample": f"each step covers {what}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{steps} steps x {what}", "host_cores": host_cores()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------- GPU arm ----
def run_ours(args):
    import torch
    from paper_1905_10395_b200 import api, inputs
    from paper_1905_10395_b200.runner import Population

    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local if world > 1 else 0)
    torch.cuda.set_device(dev)
    api.lib()                                       # fail loudly if the CUDA library is missing
    spec = workload_spec(args)
    P, G, d = spec["P"], spec["G"], spec["d"]
    steps, warmup = args.steps, max(args.warmup, 3)

    # --graph: everything runs on a side stream so that whole periods can be captured into a CUDA graph
    gstream = None
    if args.graph:
        import contextlib
        gstream = torch.cuda.Stream(dev)
        _stack = contextlib.ExitStack()
        _stack.enter_context(torch.cuda.stream(gstream))
    # ---- inputs: generated on the host from the seed (C4: into pinned memory, also used by the e2e leg)
    hx = hg = None
    if spec["kind"] == "external":
        pin = world == 1                      # pinned only where the end-to-end leg will copy from them
        hx = torch.empty((P, d), dtype=torch.float32, pin_memory=pin)
        hg = torch.empty((P, d), dtype=torch.float32, pin_memory=pin)
        w = inputs.make_external(P, G, d, eta=spec["eta"], lambda_l=spec["lambda_l"], lambda_g=spec["lambda_g"],
                                 tau=spec["tau"], steps=steps, config_id=4, x_out=hx.numpy(), g_out=hg.numpy())
        x = hx.to(dev, non_blocking=True)
        g = hg.to(dev, non_blocking=True)
        alg1 = dict(gamma_l=0.1, gamma_g=0.05, tau_g=4 * spec["tau"]) if args.schedule == "algorithm1" else None
        pop = Population(w, device=str(dev), x=x, g=g, arithmetic=args.arith, algorithm1=alg1,
                         momentum=args.momentum, weight_decay=args.weight_decay)
    elif spec["kind"] == "psd":
        w = inputs.make_psd(P=P, n=spec["n"], r=spec["r"], steps=steps)
        pop = Population(w, device=str(dev), arithmetic=args.arith, stream=gstream, eagd=args.eagd)
    else:
        w = inputs.config(spec["cfg"], tau=spec["tau"])
        pop = Population(w, device=str(dev), fused_quadratic=True, arithmetic=args.arith, stream=gstream,
                         flags=0 if args.mlp_unfused_step else (api.FLAG_MLP_FUSED_STEP | api.FLAG_MATCOMP_FUSED_STEP))
    launches_per_step = lambda t: spec["launches"][0] if t % spec["tau"] == 0 else spec["launches"][1]
    torch.cuda.synchronize(dev)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    alg1_mode = getattr(pop, "alg1", None) is not None
    # ---- device-resident timing
    for _ in range(warmup):
        pop.step()
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    g_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier()
    torch.cuda.synchronize(dev)
    wall0 = time.time()
    ev0.record()
    n_launch = 0
    pull_flags = []
    e_ev = []                                    # MLP: events around the held-out election
    for s in range(steps):
        t = pop.t
        batch = pop.batches[t % len(pop.batches)] if pop.batches else None
        if spec["kind"] in ("psd", "mlp"):
            g_ev[s][0].record()
        pop.lsgd.grad(batch)
        if spec["kind"] in ("psd", "mlp"):
            g_ev[s][1].record()
        if alg1_mode:
            # Algorithm 1: step with small pulls towards the leader copies, then the communication when due
            k_ev[s][0].record()
            pop.lsgd.step()
            k_ev[s][1].record()
            pop.t += 1
            n_launch += 1
            pull_flags.append(True)
            loc, glo = pop.t % spec["tau"] == 0, pop.t % pop.alg1["tau_g"] == 0
            if loc or glo:
                pop._elect(None, False)
                n_launch += 1 + 2 * (int(loc) + int(glo))
            continue
        if t % spec["tau"] == 0 and not getattr(pop, "eagd", False):
            if spec["kind"] == "mlp":
                e_ev.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
                e_ev[-1][0].record()
            pop.lsgd.elect(pop.loss_ring[pop.n_elections % pop.loss_ring.shape[0]] if pop.loss_ring is not None else None)
            if spec["kind"] == "mlp":
                e_ev[-1][1].record()
            pop.n_elections += 1
        k_ev[s][0].record()
        pop.lsgd.step()
        k_ev[s][1].record()
        pop.t += 1
        n_launch += launches_per_step(t)
        pull_flags.append(t % spec["tau"] == 0)
    ev1.record()
    torch.cuda.synchronize(dev)
    wall1 = time.time()
    barrier()
    clocks = sampler.stop(wall0, wall1)
    elapsed_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    value = aggregate(P * d * steps, elapsed_ms, world)
    k_ms = [a.elapsed_time(b) for a, b in k_ev]
    upd_ms = float(np.mean(k_ms))
    alg_bytes = bytes_per_worker_param(spec) * P * d
    with_momentum = spec["kind"] == "external" and args.momentum is not None
    if with_momentum:
        alg_bytes += 8.0 * P * d                # the momentum buffer is read and rewritten
    if alg1_mode:
        alg_bytes += 4.0 * (G + 1) * d          # the G + 1 leader copies are read once per step
    peak, peak_src = read_peaks()
    achieved = alg_bytes / (upd_ms * 1e-3) / 1e9
    traffic = None
    if spec["kind"] == "external" and args.arith == 0 and not alg1_mode and not with_momentum and d == (1 << 26):
        n_pull = sum(pull_flags)
        traffic = P * d * (n_pull * MEASURED_TRAFFIC_PER_WORKER_PARAM["pull"] +
                           (steps - n_pull) * MEASURED_TRAFFIC_PER_WORKER_PARAM["plain"]) / steps
    if pop.lsgd.check_device() != 0:
        raise SystemExit("device status word set during the bench")

    if with_momentum:
        k1_name = "momentum_update_kernel"
    elif spec["kind"] == "quadratic" or spec["P"] > 25:
        k1_name = "update_chunked_kernel"
    else:
        k1_name = "pull_update_staged_kernel / plain_update_kernel"
    roofline = {"bound": "hbm", "kernel": k1_name, "achieved": achieved,
                "peak": peak, "peak_source": peak_src + " copy bandwidth (1 read : 1 write; this kernel reads 2 : 1, so "
                "a fraction slightly above 1 is possible)", "unit": "GB/s", "frac": achieved / peak,
                "nominal_peak": NOMINAL_HBM_GBS, "frac_of_nominal": achieved / NOMINAL_HBM_GBS,
                "traffic": traffic, "ms_per_launch": upd_ms, "algorithmic_bytes_per_launch": alg_bytes,
                "pull_steps": int(sum(pull_flags)), "plain_steps": int(steps - sum(pull_flags)),
                "ms_pull": float(np.mean([m for m, f in zip(k_ms, pull_flags) if f])) if any(pull_flags) else None,
                "ms_plain": float(np.mean([m for m, f in zip(k_ms, pull_flags) if not f])) if not all(pull_flags) else None}
    if spec["kind"] == "psd":
        # the gradient kernel dominates and is bound by fp64 arithmetic: 148 SMs x 64 FMA/clk x 2 x 1.965 GHz
        g_ms = float(np.mean([a.elapsed_time(b) for a, b in g_ev]))
        flops = 4.0 * P * spec["n"] ** 2 * spec["r"]           # two passes of n^2 r fused multiply-adds per worker
        fp64_peak = 148 * 64 * 2 * 1.965e9 / 1e12
        roofline = {"bound": "alu", "kernel": "psd_grad_kernel", "achieved": flops / (g_ms * 1e-3) / 1e12,
                    "peak": fp64_peak, "peak_source": "148 SMs x 64 fp64 FMA/clk x 1.965 GHz", "unit": "TFLOP/s",
                    "frac": flops / (g_ms * 1e-3) / 1e12 / fp64_peak, "traffic": None, "ms_per_launch": g_ms,
                    "flops_per_launch": flops}
    if spec["kind"] == "mlp" and not args.mlp_unfused_step and not all(pull_flags):
        # plain steps: the gradient call holds every GEMM and, in their epilogues, the SGD step itself.  With a
        # batch of 128 rows per worker each weight is used 2 x 128 times per pass, so the weight streams bound it.
        g_ms = float(np.mean([a.elapsed_time(b) for (a, b), f in zip(g_ev, pull_flags) if not f]))
        mb, mflops = mlp_step_bytes_flops(w.meta["dims"], int(w.meta["batch"]))
        ab = mlp_algorithmic_bytes(w.meta["dims"])
        t_peak, t_src = read_tensor_peak()
        roofline = {"bound": "hbm", "kernel": "bgemm_bf16_kernel inside the fused gradient + step call (plain steps)",
                    "achieved": P * ab / (g_ms * 1e-3) / 1e9, "peak": peak, "peak_source": peak_src + " copy bandwidth",
                    "unit": "GB/s", "frac": P * ab / (g_ms * 1e-3) / 1e9 / peak, "nominal_peak": NOMINAL_HBM_GBS,
                    "frac_of_nominal": P * ab / (g_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS, "traffic": None,
                    "ms_per_launch": g_ms, "algorithmic_bytes_per_launch": P * ab,
                    "traffic_model": {"bytes_per_launch": P * mb, "frac": P * mb / (g_ms * 1e-3) / 1e9 / peak,
                                      "what": "every operand counted once per kernel that reads or writes it"},
                    "tensor_tflops": P * mflops / (g_ms * 1e-3) / 1e12,
                    "tensor_peak_tflops": t_peak, "tensor_peak_source": t_src,
                    "tensor_frac": P * mflops / (g_ms * 1e-3) / 1e12 / t_peak}
        if e_ev:
            # the held-out election: its two hidden-layer products (M = held-out batch per worker) are the
            # tensor-bound part of this workload; their flops over the whole election call
            d0, d1, d2, d3 = [int(v) for v in w.meta["dims"]]
            n_h = int(w.arrays["held_y"].shape[0])
            e_ms = float(np.mean([a.elapsed_time(b) for a, b in e_ev]))
            e_flops = 2.0 * P * n_h * (d0 * d1 + d1 * d2 + d2 * d3)
            roofline["election"] = {"bound": "tensor", "kernel": "bgemm_pair_kernel (two hidden-layer products) + logits + softmax + election",
                                    "ms_per_election": e_ms, "elections": len(e_ev), "flops_per_election": e_flops,
                                    "achieved": e_flops / (e_ms * 1e-3) / 1e12, "peak": t_peak, "peak_source": t_src,
                                    "unit": "TFLOP/s", "frac": e_flops / (e_ms * 1e-3) / 1e12 / t_peak}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": elapsed_ms / steps, "steps_per_s": steps * world / (elapsed_ms * 1e-3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {0: "f64", 1: "f64", 2: "f32"}[args.arith], "data": "synthetic",
        "config": {"workload": spec["name"], "tau": spec["tau"], "storage": "f32",
                   "arithmetic": ["fp64 unfused", "fp64 fma", "fp32 fma"][args.arith],
                   "l2": ("per-step inputs exceed the 126 MB L2; no flush between steps" if P * d * 8 > 3e8 else
                          "working set fits in L2; steps run back to back as in training (no flush)"),
                   "multi_gpu": "replicas only", "schedule": "eagd" if getattr(args, "eagd", False) else args.schedule,
                   **({"momentum": args.momentum, "weight_decay": args.weight_decay} if with_momentum else {}),
                   **({"mlp_fused_step": not args.mlp_unfused_step} if spec["kind"] == "mlp" else {})},
        "clocks": clocks,
        "roofline": roofline,
        "gpu_launches": n_launch,
    }

    # ---- the same steps replayed from a CUDA graph (whole periods and whole passes over the batch ring)
    if args.graph and spec["kind"] in ("quadratic", "matcomp", "mlp") and world == 1:
        import math
        cap = spec["tau"] * (len(pop.batches) if pop.batches else 1) // math.gcd(spec["tau"], len(pop.batches) if pop.batches else 1)
        while pop.t % cap:
            pop.step()
        pop.capture(cap)
        pop.replay()                                # warm replay
        reps = max(1, steps // cap)
        torch.cuda.synchronize(dev)
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record()
        for _ in range(reps):
            pop.replay()
        q1.record()
        torch.cuda.synchronize(dev)
        g_ms_step = q0.elapsed_time(q1) / (reps * cap)
        line["graph"] = {"ms_per_step": g_ms_step, "steps_per_s": 1e3 / g_ms_step, "value": P * d / (g_ms_step * 1e-3),
                         "steps": reps * cap, "steps_per_graph": cap}
        if pop.lsgd.check_device() != 0:
            raise SystemExit("device status word set during the graph replays")

    # ---- end to end through the C ABI with HOST buffers: H2D of the step's inputs, D2H of its result.
    # Two handles on two streams take the steps in turn, so one step's read-back crosses the bus while the next
    # step's inputs come in (the link is full duplex); every step still copies all of x and g in and all of x out.
    if rank == 0 and world == 1 and not args.no_e2e and hx is not None and not alg1_mode:
        e_steps = max(2, args.e2e_steps + (args.e2e_steps & 1))       # an even number: both streams do the same work
        pop.close()
        torch.cuda.synchronize(dev)
        loss_host = torch.from_numpy(w.arrays["loss_ring"]).pin_memory()
        lanes = []
        for k in range(2):
            st = torch.cuda.Stream(dev)
            xk = x if k == 0 else torch.empty_like(x)
            gk = g if k == 0 else torch.empty_like(g)
            with torch.cuda.stream(st):
                pk = Population(w, device=str(dev), x=xk, g=gk, arithmetic=args.arith, stream=st,
                                momentum=args.momentum, weight_decay=args.weight_decay)
            lanes.append(dict(stream=st, pop=pk, out=torch.empty((P, d), dtype=torch.float32, pin_memory=True),
                              dloss=torch.empty(P, dtype=torch.float32, device=dev)))
        torch.cuda.synchronize(dev)

        def e2e_step(it):
            ln = lanes[it & 1]
            with torch.cuda.stream(ln["stream"]):
                ln["pop"].x.copy_(hx, non_blocking=True)
                ln["pop"].g.copy_(hg, non_blocking=True)
                ln["dloss"].copy_(loss_host[it % loss_host.shape[0]], non_blocking=True)
                ln["pop"].lsgd.grad(None)
                ln["pop"].lsgd.elect(ln["dloss"])
                ln["pop"].lsgd.step()
                ln["out"].copy_(ln["pop"].x, non_blocking=True)

        for it in range(2):                                            # one untimed step per stream
            e2e_step(it)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sa, sb = lanes[0]["stream"], lanes[1]["stream"]
        e0.record(sa)
        sb.wait_event(e0)
        for it in range(e_steps):
            e2e_step(it)
        sa.wait_stream(sb)
        e1.record(sa)
        torch.cuda.synchronize(dev)
        e_ms = e0.elapsed_time(e1) / e_steps
        for ln in lanes:
            if ln["pop"].lsgd.check_device() != 0:
                raise SystemExit("device status word set during the end-to-end steps")
            ln["pop"].close()
        line["e2e"] = {"value": P * d / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(2 * P * d * 4 + P * 4),
                       "d2h_bytes_per_step": int(P * d * 4), "ms_per_step": e_ms, "steps": e_steps,
                       "note": "every step elects (a pull step) so tau does not apply; two handles on two streams "
                               "alternate so that read-back and upload overlap on the full-duplex link"}
        pop = None
    else:
        line["e2e"] = None
    if pop is not None:
        pop.close()

    # ---- CPU oracle beside it (rank 0, N = 1 only): one process, then every host core
    if rank == 0 and world == 1 and not args.no_cpu:
        sample = args.sample_cols or (1 << 22)
        osteps = {"external": 3, "quadratic": 3, "matcomp": 8, "mlp": 4, "psd": 4}[spec["kind"]]
        v, dt, what, osteps = oracle_sample_run(spec, osteps, 1, sample, min_seconds=10.0)
        cores = _threads_used() if spec["kind"] in ("mlp", "psd") else 1
        # fewer steps for the all-cores leg: the processes share the memory system and run about three times longer
        allc = oracle_all_cores(spec, max(2, osteps // 3), min(sample, 1 << 20) if host_cores() > 16 else sample)
        line["cpu_baseline"] = cpu_baseline_record(spec, v, cores, f"{osteps} steps x {what}, {dt:.1f} s", allc)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------- groups sharded over ranks (optional mode) ----
def run_sharded(args):
    """--sharded: the paper's own mapping, groups on ranks (paper_1905_10395_b200/sharded.py).  The C4 shape
    (P = 16, G = 4; d = 2^22 unless --d is given, since every rank generates the whole seeded population on its
    host) split by groups over the N ranks; per pull step the ranks exchange their best loss and the owner
    broadcasts the global leader's row over NCCL.  Total work is fixed ("strong").  Not the default: the
    default multi-GPU mode is independent replicas."""
    import torch
    from paper_1905_10395_b200 import api, inputs, sharded

    rank, world, local = dist_env()
    dev = torch.device("cuda", local if world > 1 else 0)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    api.lib()
    P, G, d = 16, 4, args.d or (1 << 22)
    tau = args.tau or 1
    steps, warmup = args.steps, max(args.warmup, 3)
    w = inputs.make_external(P, G, d, eta=0.01, lambda_l=0.1, lambda_g=0.05, tau=tau, steps=steps, config_id=4)
    eng = sharded.CudaShardEngine(w, rank, world, device=str(dev), arithmetic=args.arith)

    def one_step():
        if world > 1:
            sharded.distributed_step(eng)
        else:
            sharded.run_lockstep([eng], 1)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(warmup):
        one_step()
    sampler = ClockSampler(local if world > 1 else 0)
    sampler.start()
    barrier()
    torch.cuda.synchronize(dev)
    wall0 = time.time()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        one_step()
    ev1.record()
    torch.cuda.synchronize(dev)
    wall1 = time.time()
    barrier()
    clocks = sampler.stop(wall0, wall1)
    elapsed_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    if eng.lsgd.check_device() != 0:
        raise SystemExit("device status word set during the bench")
    if rank == 0:
        n_pull = len([t for t in range(warmup, warmup + steps) if t % tau == 0])
        line = {"metric": METRIC, "value": P * d * steps / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
                "warmup": warmup, "ms_per_step": elapsed_ms / steps, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "f64" if args.arith < 2 else "f32", "data": "synthetic",
                "config": {"workload": f"C4 shape sharded by groups: P=16 G=4 d={d} over {world} rank(s)", "tau": tau,
                           "multi_gpu": "groups on ranks; per pull step an all-gather of the ranks' best losses and a "
                                        "broadcast of the global leader's row into every rank's own memory",
                           "l2": "per-step inputs exceed the 126 MB L2" if P * d * 8 / world > 126e6 else "working set fits in L2"},
                "clocks": clocks, "roofline": None, "e2e": None,
                "gpu_launches": steps * 1 + n_pull * 1}
        print(json.dumps(line), flush=True)
    eng.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0,
                    help="timed steps (default: 100 for c4; 1000-4000 for the small workloads, so that the timed "
                         "region lasts a few tenths of a second and holds several clock samples)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=["c0", "c1", "c2", "c3", "c4", "psd"])
    ap.add_argument("--rank", type=int, default=10, help="psd workload: rank r")
    ap.add_argument("--tau", type=int, default=0)
    ap.add_argument("--arith", type=int, default=0, choices=[0, 1, 2])
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--sample-cols", type=int, default=0)
    ap.add_argument("--d", type=int, default=0, help="c4: parameters per worker (default 2^26); smaller values give a small case")
    ap.add_argument("--schedule", default="fused", choices=["fused", "algorithm1"],
                    help="c4 only: algorithm1 = the paper's Algorithm 1 schedule (gamma 0.1 / 0.05, tau_G = 4 tau)")
    ap.add_argument("--mlp-unfused-step", action="store_true",
                    help="c2, c3: do not set LSGD_FLAG_MATCOMP_FUSED_STEP / LSGD_FLAG_MLP_FUSED_STEP")
    ap.add_argument("--graph", action="store_true", help="c0-c3: also time the steps replayed from a CUDA graph")
    ap.add_argument("--momentum", type=float, default=None,
                    help="c4: Nesterov momentum of the Section 4.1 optimiser (adds the buffer v: 20 B per worker-param)")
    ap.add_argument("--weight-decay", type=float, default=0.0)
    ap.add_argument("--eagd", action="store_true",
                    help="psd: elastic averaging towards a center variable instead of leaders (the paper's comparison line)")
    ap.add_argument("--sharded", action="store_true",
                    help="groups sharded over the ranks with a leader broadcast per pull step (see run_sharded)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.steps <= 0:
        args.steps = 100 if args.impl == "reference" else \
            {"c4": 100, "c0": 4000, "c1": 2000, "c2": 4000, "c3": 1000, "psd": 2000}[args.workload]
    if args.eagd and args.workload != "psd":
        raise SystemExit("--eagd times the comparison line of the PSD completion experiment only")
    if args.impl == "reference":
        run_reference(args)
    elif args.sharded:
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
