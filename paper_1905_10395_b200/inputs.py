"""Seeded synthetic input generators for the Leader SGD workloads.

This module only draws random arrays (NumPy ``Philox`` streams) and lays them out.
It contains none of the method's arithmetic: no gradient, loss, election or update
is evaluated here.  Both the CPU oracle's tests and the CUDA path's tests / bench
consume exactly these arrays, so neither side ever produces an input for the other.

Conventions
-----------
* Worker parameters are a row-major ``float32[P, ld]`` matrix, ``ld >= d`` a multiple
  of 32 floats; columns ``d..ld`` are zero padding.
* A variance written ``N(0, v)`` in a workload description is a *variance*
  (``std = sqrt(v)``).
* ``group_of[i]`` is the group of worker ``i``; the presets use ``G`` contiguous
  equal groups (the paper's n groups of l workers, Section 2.2).
"""
from __future__ import annotations

import math
import threading
from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

SEED_BASE = 190510395

# MLP population geometry (784-1024-1024-10 ReLU classifier).
MLP_DIMS = (784, 1024, 1024, 10)


def rng(config_id: int, stream: int) -> np.random.Generator:
    """Independent Philox stream for (config, stream)."""
    return np.random.Generator(np.random.Philox(key=[SEED_BASE + int(config_id), int(stream)]))


def round_up(n: int, m: int) -> int:
    return (n + m - 1) // m * m


def contiguous_groups(P: int, G: int) -> np.ndarray:
    """Worker i belongs to group i // ceil(P/G) (equal contiguous groups when G | P)."""
    l = (P + G - 1) // G
    g = (np.arange(P) // l).astype(np.int32)
    assert g.max() == G - 1, "every group must be non-empty"
    return g


@dataclass
class Workload:
    """One synthetic problem instance: hyper-parameters plus every array either path reads."""
    name: str
    objective: str                      # "external" | "quadratic" | "matcomp" | "mlp"
    P: int
    G: int
    d: int
    ld: int
    group_of: np.ndarray
    eta: float
    lambda_l: float
    lambda_g: float
    tau: int
    steps: int
    x0: Optional[np.ndarray] = None     # float32 [P, ld]
    arrays: Dict[str, np.ndarray] = field(default_factory=dict)
    meta: Dict[str, object] = field(default_factory=dict)


def _normal_rows(out: np.ndarray, config_id: int, stream0: int, std: float = 1.0, threads: int = 8) -> None:
    """Fill the rows of ``out`` (float32 [R, n]) with N(0, std^2), one Philox stream per row."""
    R = out.shape[0]

    def work(lo: int, hi: int) -> None:
        for r in range(lo, hi):
            g = rng(config_id, stream0 + r)
            g.standard_normal(out=out[r], dtype=np.float32)
            if std != 1.0:
                out[r] *= np.float32(std)

    if R == 1 or out[0].size < (1 << 18):
        work(0, R)
        return
    nt = max(1, min(threads, R))
    bounds = [R * k // nt for k in range(nt + 1)]
    ts = [threading.Thread(target=work, args=(bounds[k], bounds[k + 1])) for k in range(nt)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()


def _padded(P: int, d: int, ld: int, config_id: int, stream0: int, std: float = 1.0,
            out: Optional[np.ndarray] = None) -> np.ndarray:
    """float32 [P, ld] with N(0, std^2) in columns < d and zeros in the padding."""
    if out is None:
        out = np.zeros((P, ld), dtype=np.float32)
    if ld == d:
        _normal_rows(out, config_id, stream0, std)
    else:
        tmp = np.empty((P, d), dtype=np.float32)
        _normal_rows(tmp, config_id, stream0, std)
        out[:, :d] = tmp
        out[:, d:] = 0.0
    return out


# --------------------------------------------------------------------------------------
# Quadratic: f(x) = 1/2 sum_k a_k (x_k - b_k)^2, a log-uniform in [0.01, 1], b ~ N(0,1)
# --------------------------------------------------------------------------------------
def make_quadratic(P: int, G: int, d: int, *, eta: float, lambda_l: float, lambda_g: float, tau: int,
                   steps: int, sigma: float = 0.01, noise_ring: int = 10, config_id: int = 0,
                   ld: Optional[int] = None, group_of: Optional[np.ndarray] = None,
                   name: str = "quadratic") -> Workload:
    ld = round_up(d, 32) if ld is None else ld
    r = rng(config_id, 0)
    a = np.zeros(ld, dtype=np.float32)
    b = np.zeros(ld, dtype=np.float32)
    a[:d] = np.power(10.0, r.uniform(-2.0, 0.0, size=d)).astype(np.float32)
    b[:d] = r.standard_normal(d).astype(np.float32)
    x0 = _padded(P, d, ld, config_id, 1000)
    noise = np.zeros((noise_ring, P, ld), dtype=np.float32)
    for s in range(noise_ring):
        _padded(P, d, ld, config_id, 100000 + 1000 * s, out=noise[s])
    go = contiguous_groups(P, G) if group_of is None else np.asarray(group_of, dtype=np.int32)
    return Workload(name=name, objective="quadratic", P=P, G=G, d=d, ld=ld, group_of=go, eta=eta,
                    lambda_l=lambda_l, lambda_g=lambda_g, tau=tau, steps=steps, x0=x0,
                    arrays={"a": a, "b": b, "noise": noise}, meta={"sigma": float(sigma)})


# --------------------------------------------------------------------------------------
# External objective: gradients and election losses are given (large fused-update stress)
# --------------------------------------------------------------------------------------
def make_external(P: int, G: int, d: int, *, eta: float, lambda_l: float, lambda_g: float, tau: int,
                  steps: int, loss_ring: int = 16, config_id: int = 4, ld: Optional[int] = None,
                  group_of: Optional[np.ndarray] = None, name: str = "external",
                  x_out: Optional[np.ndarray] = None, g_out: Optional[np.ndarray] = None) -> Workload:
    """x0 ~ N(0,1), one fixed gradient array g ~ N(0,1) reused every step, and a ring of
    ``loss_ring`` election-loss vectors ~ U[0,1), one consumed per election.
    ``x_out`` / ``g_out`` may be caller-provided (e.g. pinned) float32 [P, ld] buffers."""
    ld = round_up(d, 32) if ld is None else ld
    x0 = _padded(P, d, ld, config_id, 1000, out=x_out)
    g = _padded(P, d, ld, config_id, 5000, out=g_out)
    losses = rng(config_id, 7).random((loss_ring, P), dtype=np.float32)
    go = contiguous_groups(P, G) if group_of is None else np.asarray(group_of, dtype=np.int32)
    return Workload(name=name, objective="external", P=P, G=G, d=d, ld=ld, group_of=go, eta=eta,
                    lambda_l=lambda_l, lambda_g=lambda_g, tau=tau, steps=steps, x0=x0,
                    arrays={"g": g, "loss_ring": losses})


# --------------------------------------------------------------------------------------
# Matrix completion on observed entries of M = U V^T
# --------------------------------------------------------------------------------------
def _distinct_cells(r: np.random.Generator, n_cells: int, n_obs: int) -> np.ndarray:
    """``n_obs`` distinct linear cell indices in [0, n_cells), in draw order."""
    if n_obs > n_cells:
        raise ValueError("more observed cells than cells")
    if n_obs == n_cells:
        return r.permutation(n_cells).astype(np.int64)
    chosen = np.empty(0, dtype=np.int64)
    while chosen.size < n_obs:
        draw = r.integers(0, n_cells, size=int((n_obs - chosen.size) * 1.1) + 16, dtype=np.int64)
        cat = np.concatenate([chosen, draw])
        _, first = np.unique(cat, return_index=True)
        chosen = cat[np.sort(first)]
    return chosen[:n_obs]


def make_matcomp(P: int, G: int, *, n_rows: int = 10000, n_cols: int = 10000, rank: int = 10,
                 n_obs: int = 1_000_000, n_heldout: int = 65536, batch: int = 4096, eta: float = 0.01,
                 lambda_l: float = 0.1, lambda_g: float = 0.05, tau: int = 8, steps: int = 16,
                 config_id: int = 2, group_of: Optional[np.ndarray] = None,
                 name: str = "matcomp") -> Workload:
    """Ground truth M = U V^T, entries of U, V ~ N(0, 1/sqrt(rank)); ``n_obs`` distinct observed
    cells (noiseless values); per-worker factors [X | Y] ~ N(0, 0.01); per-step per-worker
    minibatches are positions into the observed list drawn with replacement; the held-out set is
    the first ``n_heldout`` entries of a seeded permutation of the observed list."""
    r = rng(config_id, 0)
    std_uv = (1.0 / math.sqrt(rank)) ** 0.5
    U = r.standard_normal((n_rows, rank)) * std_uv
    V = r.standard_normal((n_cols, rank)) * std_uv
    cells = _distinct_cells(r, n_rows * n_cols, n_obs)
    obs_r = (cells // n_cols).astype(np.int32)
    obs_c = (cells % n_cols).astype(np.int32)
    obs_v = np.einsum("ij,ij->i", U[obs_r], V[obs_c]).astype(np.float32)
    held = r.permutation(n_obs)[:n_heldout].astype(np.int32)
    d = (n_rows + n_cols) * rank
    ld = round_up(d, 32)
    x0 = _padded(P, d, ld, config_id, 1000, std=0.1)
    pos = rng(config_id, 9).integers(0, n_obs, size=(steps, P, batch), dtype=np.int32)
    go = contiguous_groups(P, G) if group_of is None else np.asarray(group_of, dtype=np.int32)
    return Workload(name=name, objective="matcomp", P=P, G=G, d=d, ld=ld, group_of=go, eta=eta,
                    lambda_l=lambda_l, lambda_g=lambda_g, tau=tau, steps=steps, x0=x0,
                    arrays={"obs_r": obs_r, "obs_c": obs_c, "obs_v": obs_v, "heldout_pos": held,
                            "batch_pos": pos},
                    meta={"n_rows": n_rows, "n_cols": n_cols, "rank": rank, "batch": batch})


# --------------------------------------------------------------------------------------
# Dense positive semi-definite completion (the paper's own experiment)
# --------------------------------------------------------------------------------------
def make_psd(P: int = 8, n: int = 1000, r: int = 10, *, eta: float = 5e-4, lambda_l: float = 0.2,
             lambda_g: float = 0.0, tau: int = 1, steps: int = 10, G: int = 1, config_id: int = 5,
             name: str = "psd") -> Workload:
    """M = U U^T with U in R^{n x r}, i.i.d. N(0,1) entries; every worker starts from its own X ~ N(0,1);
    defaults are the settings the paper lists for this experiment (eta 5e-4, lambda 1/5, 8 workers,
    tau 1, n 1000)."""
    U = rng(config_id, 0).standard_normal((n, r))
    M = (U @ U.T).astype(np.float32)
    d = n * r
    ld = round_up(d, 32)
    x0 = _padded(P, d, ld, config_id, 1000)
    return Workload(name=name, objective="psd", P=P, G=G, d=d, ld=ld, group_of=contiguous_groups(P, G), eta=eta,
                    lambda_l=lambda_l, lambda_g=lambda_g, tau=tau, steps=steps, x0=x0, arrays={"M": M},
                    meta={"n": n, "r": r})


# --------------------------------------------------------------------------------------
# MLP population on a synthetic Gaussian mixture
# --------------------------------------------------------------------------------------
def mlp_layout(dims=MLP_DIMS):
    """Offsets (in floats) of [W1 | b1 | W2 | b2 | W3 | b3] inside a parameter row.

    W_l is stored ``[out_l, in_l]`` row-major (input index contiguous).  Every segment starts
    on a multiple of 32 floats; padding between segments is zero and has zero gradient."""
    off = 0
    segs = []
    for l in range(len(dims) - 1):
        n_in, n_out = dims[l], dims[l + 1]
        w = off
        off = round_up(off + n_in * n_out, 32)
        b = off
        off = round_up(off + n_out, 32)
        segs.append({"w": w, "b": b, "n_in": n_in, "n_out": n_out})
    return segs, off


def make_mlp(P: int, G: int, *, dims=MLP_DIMS, pool: int = 65536, heldout: int = 1024, batch: int = 128,
             n_classes: int = 10, eta: float = 0.05, lambda_l: float = 0.1, lambda_g: float = 0.05,
             tau: int = 4, steps: int = 10, config_id: int = 3, group_of: Optional[np.ndarray] = None,
             name: str = "mlp") -> Workload:
    """Gaussian mixture: class means ~ N(0, I), sample = mean[label] + 2 N(0, I); labels are a
    seeded permutation of ``position mod n_classes`` (balanced).  He-normal weights
    (std sqrt(2 / fan_in)), zero biases, distinct stream per worker."""
    n_in = dims[0]
    r = rng(config_id, 0)
    means = r.standard_normal((n_classes, n_in)).astype(np.float32)

    def mixture(n: int, stream: int):
        rr = rng(config_id, stream)
        labels = rr.permutation(n).astype(np.int32) % n_classes
        pts = np.empty((n, n_in), dtype=np.float32)
        chunks = 8 if (n * n_in) % 8 == 0 and n * n_in >= (1 << 21) else 1
        _normal_rows(pts.reshape(chunks, -1), config_id, stream * 100 + 50)
        pts *= np.float32(2.0)
        pts += means[labels]
        return pts, labels.astype(np.int32)

    pool_x, pool_y = mixture(pool, 11)
    held_x, held_y = mixture(heldout, 12)
    segs, d = mlp_layout(dims)
    ld = d
    x0 = np.zeros((P, ld), dtype=np.float32)
    for i in range(P):
        rw = rng(config_id, 1000 + i)
        for s in segs:
            w = rw.standard_normal((s["n_out"], s["n_in"])).astype(np.float32)
            w *= np.float32(math.sqrt(2.0 / s["n_in"]))
            x0[i, s["w"]:s["w"] + w.size] = w.ravel()
    batch_idx = rng(config_id, 9).integers(0, pool, size=(steps, P, batch), dtype=np.int32)
    go = contiguous_groups(P, G) if group_of is None else np.asarray(group_of, dtype=np.int32)
    return Workload(name=name, objective="mlp", P=P, G=G, d=d, ld=ld, group_of=go, eta=eta,
                    lambda_l=lambda_l, lambda_g=lambda_g, tau=tau, steps=steps, x0=x0,
                    arrays={"pool_x": pool_x, "pool_y": pool_y, "held_x": held_x, "held_y": held_y,
                            "batch_idx": batch_idx},
                    meta={"dims": tuple(dims), "batch": batch, "n_classes": n_classes})


# --------------------------------------------------------------------------------------
# The five named configurations
# --------------------------------------------------------------------------------------
def config(k: int, **over) -> Workload:
    """C0..C4.  Keyword overrides shrink a configuration (tests) without changing its recipe."""
    if k == 0:
        kw = dict(P=4, G=1, d=1024, eta=0.1, lambda_l=0.1, lambda_g=0.0, tau=1, steps=10, sigma=0.01,
                  noise_ring=10, config_id=0, name="C0")
        kw.update(over)
        return make_quadratic(**kw)
    if k == 1:
        kw = dict(P=64, G=8, d=1 << 20, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=4, steps=100,
                  sigma=0.01, noise_ring=10, config_id=1, name="C1")
        kw.update(over)
        return make_quadratic(**kw)
    if k == 2:
        kw = dict(P=16, G=4, config_id=2, name="C2")
        kw.update(over)
        return make_matcomp(**kw)
    if k == 3:
        kw = dict(P=32, G=4, config_id=3, name="C3")
        kw.update(over)
        return make_mlp(**kw)
    if k == 4:
        kw = dict(P=16, G=4, d=1 << 26, eta=0.01, lambda_l=0.1, lambda_g=0.05, tau=1, steps=3,
                  config_id=4, name="C4")
        kw.update(over)
        return make_external(**kw)
    raise ValueError("config id must be 0..4")
