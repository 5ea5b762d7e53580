"""CPU oracle for the Leader (Stochastic) Gradient Descent step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct NumPy restatement of what one synchronous LSGD step computes,
written from the paper (Section 2.2, Eq. (1), Algorithm 1; Section 3.1.1 and the supplement's
"Definitions and Notation" for the eta-scaled form of the step and for communication periods;
the supplement's matrix-completion section for the written-out update).  Only the tests, the
smoke check and the CPU-baseline leg of the benchmark may import it; the product path never does,
and this file imports nothing from the CUDA package.

Arithmetic convention: worker parameters, gradients and losses are *stored* as float32.  Every
stored value is produced by evaluating its defining formula in float64 from the float32 inputs
and rounding once.  Reductions are float64.  There is no blocking, fusion or reordering beyond
what the formulas state.

Readings of the paper taken here (each is also exercised by a pin in tests/test_oracle_pins.py):
  * pulls are scaled by the learning rate: x+ = x - eta (g + lambda (x - z))  (Section 3.1.1,
    supplement "Definitions and Notation", and the written-out matrix-completion update
    X+ = (1 - eta lambda) X + eta lambda Z - eta grad F(X); Eq. (1) prints them unscaled).
  * gamma = gamma_G = 0 and tau_G = tau: leaders are re-elected and both pulls applied on steps
    t = 0, tau, 2 tau, ... (leaders change only at period boundaries: supplement, "Definitions and
    Notation"); all other steps are plain (S)GD steps.
  * on a pull step the gradient, both leaders and both pulls are all taken at x_t (Eq. (1): every
    right-hand term carries subscript t), i.e. a simultaneous (Jacobi) update of all workers.
  * argmin ties go to the lowest worker index; the order on losses is
    -inf < finite < +inf < NaN, and -0.0 == +0.0.
  * Nesterov momentum and weight decay (Section 4.1) act on the gradient step only; the pulls stay outside
    the momentum buffer (momentum_update).

Pins: see tests/test_oracle_pins.py, test_oracle_algorithm1.py, test_oracle_momentum.py, test_oracle_eagd.py.
Parity unpinned (self-consistent definitions only, no external fact fixes them): the placement of bf16
roundings in the backward pass of the MLP objective's "bf16emu" mode, and the 1/(2|B|) / 1/N constants of
the observed-entry matrix-completion objective.
"""
from __future__ import annotations

import math
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

F32 = np.float32
F64 = np.float64


# ----------------------------------------------------------------------------------------------
# Election (Section 2.2: local leader = argmin within the group, global leader = argmin over all)
# ----------------------------------------------------------------------------------------------
def _better(a: float, b: float) -> bool:
    """True iff loss a strictly precedes loss b in the order -inf < finite < +inf < NaN."""
    if math.isnan(a):
        return False
    if math.isnan(b):
        return True
    return a < b            # IEEE: -0.0 < +0.0 is False, so the two zeros tie


def elect(loss: np.ndarray, group_of: Sequence[int], G: int) -> Tuple[np.ndarray, int]:
    """Local leaders ll[j] = argmin_{i in group j} loss_i and global leader gl = argmin_i loss_i.

    One left-to-right scan; a later worker replaces the incumbent only if strictly better, so
    ties resolve to the lowest index."""
    P = len(loss)
    ll = [-1] * G
    gl = -1
    for i in range(P):
        li = float(loss[i])
        j = int(group_of[i])
        if ll[j] < 0 or _better(li, float(loss[ll[j]])):
            ll[j] = i
        if gl < 0 or _better(li, float(loss[gl])):
            gl = i
    return np.asarray(ll, dtype=np.int32), int(gl)


# ----------------------------------------------------------------------------------------------
# The update (Eq. (1), eta-scaled pulls; plain SGD form between communications)
# ----------------------------------------------------------------------------------------------
def update(x: np.ndarray, g: np.ndarray, group_of: Sequence[int], ll: Sequence[int], gl: int,
           eta: float, lambda_l: float, lambda_g: float, pull: bool) -> None:
    """In-place on x (float32 [P, ld]).

    pull:  x_i <- x_i - eta g_i - eta lambda_l (x_i - x_{ll[group(i)]}) - eta lambda_g (x_i - x_gl)
    else:  x_i <- x_i - eta g_i
    with every right-hand side taken from x at time t (leader rows are snapshotted first)."""
    eta = float(F32(eta))
    lambda_l = float(F32(lambda_l))
    lambda_g = float(F32(lambda_g))
    P = x.shape[0]
    if pull:
        snap_l = {int(r): x[int(r)].astype(F64) for r in set(int(v) for v in ll)}
        snap_g = x[int(gl)].astype(F64)
    for i in range(P):
        xi = x[i].astype(F64)
        new = xi - eta * g[i].astype(F64)
        if pull:
            zl = snap_l[int(ll[int(group_of[i])])]
            new = new - eta * lambda_l * (xi - zl) - eta * lambda_g * (xi - snap_g)
        x[i] = new.astype(F32)


def momentum_update(x: np.ndarray, v: np.ndarray, g: np.ndarray, group_of: Sequence[int], ll: Sequence[int],
                    gl: int, eta: float, lambda_l: float, lambda_g: float, pull: bool, mu: float,
                    wd: float) -> None:
    """The optimiser of the deep-network runs (Section 4.1: Nesterov momentum 0.9 and weight decay 1e-4 for
    every method), in place on x and on the momentum buffer v (both float32 [P, ld]):

        d  = g + wd x            weight decay enters as the gradient of (wd / 2) |x|^2
        v+ = mu v + d            momentum buffer, v_0 = 0
        u  = d + mu v+           Nesterov look-ahead direction
        x+ = x - eta u  [ - eta lambda_l (x - x_ll) - eta lambda_g (x - x_gl)  on a pull step ]

    The paper does not say how the pulls and the momentum buffer combine; the reading here keeps the pulls
    out of the buffer, so that with mu = wd = 0 the step is Eq. (1) again.  Every stored value is evaluated
    in float64 in the order written and rounded once; u uses the unrounded v+."""
    eta = float(F32(eta))
    lambda_l = float(F32(lambda_l))
    lambda_g = float(F32(lambda_g))
    mu = float(F32(mu))
    wd = float(F32(wd))
    P = x.shape[0]
    if pull:
        snap_l = {int(r): x[int(r)].astype(F64) for r in set(int(q) for q in ll)}
        snap_g = x[int(gl)].astype(F64)
    for i in range(P):
        xi = x[i].astype(F64)
        d = g[i].astype(F64) + wd * xi
        vn = mu * v[i].astype(F64) + d
        u = d + mu * vn
        new = xi - eta * u
        if pull:
            zl = snap_l[int(ll[int(group_of[i])])]
            new = new - eta * lambda_l * (xi - zl) - eta * lambda_g * (xi - snap_g)
        x[i] = new.astype(F32)
        v[i] = vn.astype(F32)


# ----------------------------------------------------------------------------------------------
# Objectives
# ----------------------------------------------------------------------------------------------
class Objective:
    """grad(x, t) -> float32 [P, ld] stochastic gradients at step t; loss(x, n) -> float32 [P]
    election losses for the n-th election."""

    def grad(self, x: np.ndarray, t: int) -> np.ndarray:
        raise NotImplementedError

    def loss(self, x: np.ndarray, n: int) -> np.ndarray:
        raise NotImplementedError


class External(Objective):
    """Gradients and election losses are supplied: one fixed g, a ring of loss vectors."""

    def __init__(self, g: np.ndarray, loss_ring: np.ndarray):
        self.g, self.loss_ring = g, loss_ring

    def grad(self, x, t):
        return self.g

    def loss(self, x, n):
        return self.loss_ring[n % len(self.loss_ring)]


class Quadratic(Objective):
    """f(x) = 1/2 sum_k a_k (x_k - b_k)^2  (the positive-definite quadratic model of Section 3.3
    with a diagonal Hessian);  g = a (x - b) + sigma eps;  election loss = f(x_i) exactly."""

    def __init__(self, a: np.ndarray, b: np.ndarray, sigma: float, noise: Optional[np.ndarray]):
        self.a, self.b = a.astype(F64), b.astype(F64)
        self.sigma = float(F32(sigma))
        self.noise = noise                              # float32 [ring, P, ld] or None (batch LGD)

    def grad(self, x, t):
        g = np.empty_like(x)
        for i in range(x.shape[0]):
            gi = self.a * (x[i].astype(F64) - self.b)
            if self.noise is not None:
                gi = gi + self.sigma * self.noise[t % len(self.noise)][i].astype(F64)
            g[i] = gi.astype(F32)
        return g

    def loss(self, x, n):
        out = np.empty(x.shape[0], dtype=F32)
        for i in range(x.shape[0]):
            r = x[i].astype(F64) - self.b
            out[i] = F32(0.5 * np.sum(self.a * r * r))
        return out


class MatComp(Objective):
    """Factorised completion on observed entries.  Parameter row = [X (n_rows x rank) | Y (n_cols x
    rank)], both row-major.  Minibatch loss (1/(2|B|)) sum_{(r,c,v) in B} (<X_r, Y_c> - v)^2, so
    dX_r += e Y_c / |B| and dY_c += e X_r / |B| with e = <X_r, Y_c> - v, accumulated over the
    batch in list order (duplicates add).  Election loss = mean squared residual over a fixed
    held-out list."""

    def __init__(self, n_rows, n_cols, rank, obs_r, obs_c, obs_v, batch_pos, heldout_pos):
        self.n_rows, self.n_cols, self.rank = n_rows, n_cols, rank
        self.obs_r, self.obs_c, self.obs_v = obs_r, obs_c, obs_v
        self.batch_pos, self.heldout_pos = batch_pos, heldout_pos

    def _factors(self, xi):
        nx = self.n_rows * self.rank
        X = xi[:nx].astype(F64).reshape(self.n_rows, self.rank)
        Y = xi[nx:nx + self.n_cols * self.rank].astype(F64).reshape(self.n_cols, self.rank)
        return X, Y

    def grad(self, x, t):
        g = np.zeros_like(x)
        nx = self.n_rows * self.rank
        for i in range(x.shape[0]):
            pos = self.batch_pos[t % len(self.batch_pos)][i]
            r, c, v = self.obs_r[pos], self.obs_c[pos], self.obs_v[pos].astype(F64)
            X, Y = self._factors(x[i])
            e = np.sum(X[r] * Y[c], axis=1) - v
            gX = np.zeros_like(X)
            gY = np.zeros_like(Y)
            np.add.at(gX, r, e[:, None] * Y[c] / len(pos))
            np.add.at(gY, c, e[:, None] * X[r] / len(pos))
            g[i, :nx] = gX.ravel().astype(F32)
            g[i, nx:nx + gY.size] = gY.ravel().astype(F32)
        return g

    def loss(self, x, n):
        pos = self.heldout_pos
        r, c, v = self.obs_r[pos], self.obs_c[pos], self.obs_v[pos].astype(F64)
        out = np.empty(x.shape[0], dtype=F32)
        for i in range(x.shape[0]):
            X, Y = self._factors(x[i])
            e = np.sum(X[r] * Y[c], axis=1) - v
            out[i] = F32(np.sum(e * e) / len(pos))
        return out


class PsdCompletion(Objective):
    """The paper's low-rank matrix completion experiment (Section 2.1 and the supplement):
    F(X) = 1/4 ||M - X X^T||_F^2 with X in R^{n x r} (the worker's parameter row, row-major),
    grad F(X) = (X X^T - M) X, exact (batch LGD); election loss F(X_i)."""

    def __init__(self, n: int, r: int, M: np.ndarray):
        self.n, self.r = int(n), int(r)
        self.M = np.asarray(M, dtype=F64).reshape(n, n)

    def _residual(self, xi):
        X = xi[: self.n * self.r].astype(F64).reshape(self.n, self.r)
        return X, X @ X.T - self.M

    def grad(self, x, t):
        g = np.zeros_like(x)
        for i in range(x.shape[0]):
            X, R = self._residual(x[i])
            g[i, : self.n * self.r] = (R @ X).ravel().astype(F32)
        return g

    def loss(self, x, n):
        out = np.empty(x.shape[0], dtype=F32)
        for i in range(x.shape[0]):
            _, R = self._residual(x[i])
            out[i] = F32(0.25 * np.sum(R * R))
        return out


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even), returned as float32 (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=F32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(F32).reshape(np.shape(a))


class Mlp(Objective):
    """Population of ReLU MLP classifiers with mean softmax cross-entropy.

    Parameter row = [W1 | b1 | W2 | b2 | ...], W_l stored [out, in] row-major at the float offsets
    given by ``segs`` (list of dicts with keys w, b, n_in, n_out).  Layer: z = h_prev W^T + b,
    h = relu(z) (no relu on the last layer).
    mode "fp32": everything float64-evaluated from float32 storage.
    mode "bf16emu": every matrix-product operand -- weights, the input batch, the stored hidden
    activations, and the back-propagated dz / dh -- is first rounded to bfloat16; products are
    accumulated in float64; bias gradients are column sums of the *rounded* dz / dh; the relu mask
    is taken from the stored (rounded) activation."""

    def __init__(self, segs, data_x, data_y, batch_idx, held_x, held_y, mode="bf16emu", loss_window=0):
        # loss_window K > 0: the election loss is the mean of the worker's minibatch losses over the last K
        # gradient evaluations (Section 4.1: "the average of the training loss computed over the last 10 ...
        # data batches"), kept in a ring of K slots and averaged in slot order
        self.loss_window = int(loss_window)
        self.ring = []
        self.n_grads = 0
        self.segs = segs
        self.data_x, self.data_y, self.batch_idx = data_x, data_y, batch_idx
        self.held_x, self.held_y = held_x, held_y
        self.rd = bf16_round if mode == "bf16emu" else (lambda a: np.asarray(a, dtype=F32))
        self.last_train_loss = None

    def _weights(self, xi):
        Ws, bs = [], []
        for s in self.segs:
            W = xi[s["w"]:s["w"] + s["n_in"] * s["n_out"]].reshape(s["n_out"], s["n_in"])
            Ws.append(self.rd(W).astype(F64))
            bs.append(xi[s["b"]:s["b"] + s["n_out"]].astype(F64))
        return Ws, bs

    def _forward(self, xi, inp):
        Ws, bs = self._weights(xi)
        hs = [self.rd(inp).astype(F64)]
        L = len(Ws)
        for l in range(L):
            z = hs[-1] @ Ws[l].T + bs[l]
            if l < L - 1:
                hs.append(self.rd(np.maximum(z, 0.0).astype(F32)).astype(F64))
        return Ws, hs, z

    @staticmethod
    def _softmax_ce(z, y):
        zs = z - z.max(axis=1, keepdims=True)
        lse = np.log(np.exp(zs).sum(axis=1, keepdims=True))
        logp = zs - lse
        n = z.shape[0]
        ce = -logp[np.arange(n), y].sum() / n
        return ce, np.exp(logp)

    def grad(self, x, t):
        g = np.zeros_like(x)
        losses = np.empty(x.shape[0], dtype=F32)
        for i in range(x.shape[0]):
            idx = self.batch_idx[t % len(self.batch_idx)][i]
            y = self.data_y[idx]
            Ws, hs, z = self._forward(x[i], self.data_x[idx])
            ce, p = self._softmax_ce(z, y)
            losses[i] = F32(ce)
            n = len(idx)
            dz = p.copy()
            dz[np.arange(n), y] -= 1.0
            dz /= n
            delta = self.rd(dz.astype(F32)).astype(F64)
            for l in range(len(Ws) - 1, -1, -1):
                s = self.segs[l]
                dW = delta.T @ hs[l]                               # [out, in]
                g[i, s["w"]:s["w"] + dW.size] = dW.ravel().astype(F32)
                g[i, s["b"]:s["b"] + s["n_out"]] = delta.sum(axis=0).astype(F32)
                if l > 0:
                    dh = (delta @ Ws[l]) * (hs[l] > 0.0)
                    delta = self.rd(dh.astype(F32)).astype(F64)
        self.last_train_loss = losses
        if self.loss_window > 0:
            slot = self.n_grads % self.loss_window
            if slot == len(self.ring):
                self.ring.append(losses.copy())
            else:
                self.ring[slot] = losses.copy()
            self.n_grads += 1
        return g

    def loss(self, x, n):
        if self.loss_window > 0:
            acc = np.zeros(x.shape[0], dtype=F64)
            for slot_losses in self.ring:
                acc = acc + slot_losses.astype(F64)
            return (acc / len(self.ring)).astype(F32)
        out = np.empty(x.shape[0], dtype=F32)
        for i in range(x.shape[0]):
            _, _, z = self._forward(x[i], self.held_x)
            out[i] = F32(self._softmax_ce(z, self.held_y)[0])
        return out


class FromCallables(Objective):
    """Any differentiable f: grad_fn(x_i) -> gradient, loss_fn(x_i) -> scalar (batch LGD)."""

    def __init__(self, grad_fn: Callable, loss_fn: Callable):
        self.grad_fn, self.loss_fn = grad_fn, loss_fn

    def grad(self, x, t):
        return np.stack([np.asarray(self.grad_fn(x[i].astype(F64)), dtype=F64).astype(F32)
                         for i in range(x.shape[0])])

    def loss(self, x, n):
        return np.asarray([F32(self.loss_fn(x[i].astype(F64))) for i in range(x.shape[0])], dtype=F32)


def center_variable(x: np.ndarray) -> np.ndarray:
    """The "center variable" reported at test time for LSGD (Section 4.1): the average of the parameters
    of all workers, accumulated in float64 in worker order and rounded once."""
    acc = np.zeros(x.shape[1], dtype=F64)
    for i in range(x.shape[0]):
        acc = acc + x[i].astype(F64)
    return (acc * (1.0 / x.shape[0])).astype(F32)


# ----------------------------------------------------------------------------------------------
# The loop
# ----------------------------------------------------------------------------------------------
class LsgdOracle:
    """State (x, t, ll, gl) and one synchronous step:

      1. g_i = stochastic gradient at x_i^t                                  (Eq. (1), Algorithm 1)
      2. if t mod tau == 0: election losses at x^t, then local / global argmin   (Section 2.2)
      3. fused update (pull form iff t mod tau == 0)                          (Eq. (1))
      4. t <- t + 1
    """

    def __init__(self, x0: np.ndarray, objective: Objective, group_of: Sequence[int], G: int,
                 eta: float, lambda_l: float, lambda_g: float, tau: int, momentum: Optional[float] = None,
                 weight_decay: float = 0.0):
        assert tau >= 1
        self.x = np.array(x0, dtype=F32, copy=True)
        # momentum is None: the step of Eq. (1); a number (0 included): the Section 4.1 optimiser
        self.mu, self.wd = momentum, weight_decay
        self.v = None if momentum is None else np.zeros_like(self.x)
        self.obj = objective
        self.group_of = np.asarray(group_of, dtype=np.int32)
        self.G = int(G)
        self.eta, self.lambda_l, self.lambda_g, self.tau = eta, lambda_l, lambda_g, int(tau)
        self.t = 0
        self.n_elections = 0
        self.ll: Optional[np.ndarray] = None
        self.gl: Optional[int] = None
        self.loss: Optional[np.ndarray] = None
        self.history: List[dict] = []           # one record per election

    def step(self, forced_loss: Optional[np.ndarray] = None) -> None:
        g = self.obj.grad(self.x, self.t)
        pull = (self.t % self.tau == 0)
        if pull:
            self.loss = np.asarray(self.obj.loss(self.x, self.n_elections) if forced_loss is None
                                   else forced_loss, dtype=F32)
            self.ll, self.gl = elect(self.loss, self.group_of, self.G)
            self.history.append({"t": self.t, "loss": self.loss.copy(), "ll": self.ll.copy(),
                                 "gl": self.gl})
            self.n_elections += 1
        if self.v is None:
            update(self.x, g, self.group_of, self.ll if pull else (), self.gl if pull else -1,
                   self.eta, self.lambda_l, self.lambda_g, pull)
        else:
            momentum_update(self.x, self.v, g, self.group_of, self.ll if pull else (), self.gl if pull else -1,
                            self.eta, self.lambda_l, self.lambda_g, pull, self.mu, self.wd)
        self.t += 1

    def run(self, steps: int) -> np.ndarray:
        for _ in range(steps):
            self.step()
        return self.x


# ----------------------------------------------------------------------------------------------
# Algorithm 1 (the paper's asynchronous LSGD listing), run synchronously
# ----------------------------------------------------------------------------------------------
class Algorithm1Oracle:
    """Algorithm 1 with all workers in lock-step (the sum of the workers' counters is then n l t, so
    "n l tau divides the sum" reads "tau divides t").  State: x, t, and the leaders' parameters
    x~^j (one per group) and x~ as COPIES taken when they are determined -- between communications
    they are stale, as in the paper's description of the modification.

      initialise:  x~^j, x~ <- parameters of the argmin workers at x_0
      repeat:      g_i at x_i
                   x_i <- x_i - eta g_i - eta (gamma/tau) (x_i - x~^{group(i)}) - eta (gamma_G/tau_G) (x_i - x~)
                   t <- t + 1
                   if tau   | t:  x~^j <- argmin inside each group (losses at the new x);  x_i <- x_i - eta lambda   (x_i - x~^j)
                   if tau_G | t:  x~   <- argmin over all workers;                         x_i <- x_i - eta lambda_G (x_i - x~)

    Readings: every pull is scaled by eta like the gradient (Section 3.1.1; the listing prints them
    unscaled -- pass coefficient / eta to obtain that form).  A communication follows the listing's order:
    the local argmin is taken on losses evaluated after the gradient step; when the global period fires as
    well, the global argmin is taken on losses evaluated AFTER the local pull has moved the workers (the
    listing's second "if" comes after the first one's pull).  A loss vector supplied from outside
    (``forced_loss``, or an objective whose losses do not depend on x) serves both elections."""

    def __init__(self, x0, objective, group_of, G, eta, lambda_l, lambda_g, gamma_l, gamma_g, tau, tau_g):
        assert tau >= 1 and tau_g >= 1
        self.x = np.array(x0, dtype=F32, copy=True)
        self.obj = objective
        self.group_of = np.asarray(group_of, dtype=np.int32)
        self.G = int(G)
        self.eta = float(F32(eta))
        self.lambda_l, self.lambda_g = float(F32(lambda_l)), float(F32(lambda_g))
        self.gamma_l, self.gamma_g = float(F32(gamma_l)), float(F32(gamma_g))
        self.tau, self.tau_g = int(tau), int(tau_g)
        self.t = 0
        self.n_elections = 0
        self.history: List[dict] = []
        loss = np.asarray(self.obj.loss(self.x, self.n_elections), dtype=F32)
        self.n_elections += 1
        self.ll, self.gl = elect(loss, self.group_of, self.G)
        self.z_l = [self.x[int(l)].copy() for l in self.ll]      # x~^j
        self.z_g = self.x[int(self.gl)].copy()                   # x~
        self.history.append({"t": 0, "loss": loss.copy(), "ll": self.ll.copy(), "gl": self.gl})

    def _pull(self, coef, target_of_worker):
        for i in range(self.x.shape[0]):
            xi = self.x[i].astype(F64)
            self.x[i] = (xi - coef * (xi - target_of_worker(i).astype(F64))).astype(F32)

    def step(self, forced_loss: Optional[np.ndarray] = None) -> None:
        g = self.obj.grad(self.x, self.t)
        cl = self.eta * (self.gamma_l / self.tau)
        cg = self.eta * (self.gamma_g / self.tau_g)
        for i in range(self.x.shape[0]):
            xi = self.x[i].astype(F64)
            new = xi - self.eta * g[i].astype(F64) - cl * (xi - self.z_l[int(self.group_of[i])].astype(F64)) \
                - cg * (xi - self.z_g.astype(F64))
            self.x[i] = new.astype(F32)
        self.t += 1
        local, glob = self.t % self.tau == 0, self.t % self.tau_g == 0
        if local or glob:
            n = self.n_elections                      # one communication = one election event
            self.n_elections += 1

            def losses():
                return np.asarray(self.obj.loss(self.x, n) if forced_loss is None else forced_loss, dtype=F32)

            loss = losses()
            loss_global = loss
            if local:
                self.ll, _ = elect(loss, self.group_of, self.G)
                self.z_l = [self.x[int(l)].copy() for l in self.ll]
                self._pull(self.eta * self.lambda_l, lambda i: self.z_l[int(self.group_of[i])])
            if glob:
                if local:
                    loss_global = losses()            # the local pull has moved the workers
                _, self.gl = elect(loss_global, self.group_of, self.G)
                self.z_g = self.x[int(self.gl)].copy()
                self._pull(self.eta * self.lambda_g, lambda i: self.z_g)
            self.history.append({"t": self.t, "loss": loss.copy(), "loss_global": loss_global.copy(),
                                 "ll": self.ll.copy(), "gl": self.gl, "local": local, "global": glob})

    def run(self, steps: int) -> np.ndarray:
        for _ in range(steps):
            self.step()
        return self.x


# ----------------------------------------------------------------------------------------------
# EAGD / EASGD, the elastic-averaging comparison line of the paper's matrix-completion experiment
# ----------------------------------------------------------------------------------------------
def eagd_center_update(center: np.ndarray, x: np.ndarray, eta: float, lam: float) -> np.ndarray:
    """X~+ = (1 - p eta lambda) X~ + p eta lambda (1/p sum_i X^i)  (supplement, "Low-Rank Matrix Completion
    Experiments"), p = number of workers.  Evaluated in float64 as printed -- k = (p eta) lambda, the mean as
    the worker-order sum times 1/p, then (1 - k) X~ + k mean -- and rounded once."""
    eta, lam = float(F32(eta)), float(F32(lam))
    p = x.shape[0]
    k = (p * eta) * lam
    acc = np.zeros(x.shape[1], dtype=F64)
    for i in range(p):
        acc = acc + x[i].astype(F64)
    mean = acc * (1.0 / p)
    return ((1.0 - k) * center.astype(F64) + k * mean).astype(F32)


class EagdOracle:
    """Elastic averaging (S)GD as the paper states it beside LGD: every worker takes the same step as in LGD,
    X+ = (1 - eta lambda) X + eta lambda Z - eta grad F(X), but towards Z = X~, a center variable that is itself
    updated by ``eagd_center_update``.  Communication every tau steps (the paper's experiment uses tau = 1);
    plain (S)GD steps in between, as for LSGD.

    Readings (the paper does not say): all right-hand sides of a communication step are taken at time t -- the
    workers move towards the old center while the center moves towards the old workers' mean; the center starts
    at the mean of the workers' starting points (with that start and 100 iterations the supplement's toy problem
    gives the printed EAGD value)."""

    def __init__(self, x0, objective, eta, lam, tau=1):
        self.x = np.array(x0, dtype=F32, copy=True)
        self.obj = objective
        self.eta, self.lam, self.tau = eta, lam, int(tau)
        self.t = 0
        self.center = center_variable(self.x)

    def step(self) -> None:
        g = self.obj.grad(self.x, self.t)
        P = self.x.shape[0]
        if self.t % self.tau == 0:
            new_center = eagd_center_update(self.center, self.x, self.eta, self.lam)
            # the workers' step is the pull form of Eq. (1) with the center as the only guide point: run it on the
            # population extended by the center as a row that is everybody's leader (its own step is x - eta 0)
            ext = np.concatenate([self.x, self.center[None, :]], axis=0)
            gext = np.concatenate([g, np.zeros_like(self.center)[None, :]], axis=0)
            update(ext, gext, [0] * (P + 1), [P], P, self.eta, 0.0, self.lam, True)
            self.x = ext[:P]
            self.center = new_center
        else:
            update(self.x, g, [0] * P, (), -1, self.eta, 0.0, 0.0, False)
        self.t += 1

    def run(self, steps: int) -> np.ndarray:
        for _ in range(steps):
            self.step()
        return self.x
