"""How ill-conditioned the free-running MLP trajectory of the 784-1024-1024-10 population is (CPU only).

The parity statement for this objective is "2e-2 relative on parameters and loss".  With eta = 0.05 on inputs of
norm ~60 the first steps overshoot (mean loss 5 -> 15 -> 20 -> ... -> 0.1), and a free-running trajectory
amplifies any difference in the order or precision of the accumulations step after step.  This file measures
that on the oracle alone: the oracle's own bf16-emulation definition (same operands, same roundings) is evaluated
twice, once accumulating every product in float64 (the oracle as it stands) and once in float32 (a library
sgemm), and the two runs are compared with the elementwise metric |x - ref| / max(|ref|, 1e-3).

What it fixes for the GPU tests: one step from a common state agrees to well below 2e-2 on every entry, but two
or more free-running steps do not -- for ANY implementation that accumulates in float32, as the tensor cores
do.  Hence the GPU parity of this workload is asserted entry by entry for every step taken from the oracle's
state, and in the bulk and norm-wise for the free-running run (tests/test_gpu_mlp.py)."""
import numpy as np

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

F32, F64 = np.float32, np.float64


class MlpFloat32Accumulation(orc.Mlp):
    """The oracle's definition with every matrix product accumulated in float32 instead of float64."""

    def _weights(self, xi):
        Ws, bs = super()._weights(xi)
        return [W.astype(F32) for W in Ws], [b.astype(F32) for b in bs]

    def _forward(self, xi, inp):
        Ws, bs = self._weights(xi)
        hs = [self.rd(inp).astype(F32)]
        for l in range(len(Ws)):
            z = hs[-1] @ Ws[l].T + bs[l]
            if l < len(Ws) - 1:
                hs.append(self.rd(np.maximum(z, 0.0).astype(F32)).astype(F32))
        return Ws, hs, z.astype(F64)

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
            delta = self.rd(dz.astype(F32)).astype(F32)
            for l in range(len(Ws) - 1, -1, -1):
                s = self.segs[l]
                dW = delta.T @ hs[l]
                g[i, s["w"]:s["w"] + dW.size] = dW.ravel().astype(F32)
                g[i, s["b"]:s["b"] + s["n_out"]] = delta.astype(F64).sum(axis=0).astype(F32)
                if l > 0:
                    delta = self.rd(((delta @ Ws[l]) * (hs[l] > 0.0)).astype(F32)).astype(F32)
        self.last_train_loss = losses
        return g


def _pair(w):
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    A = w.arrays

    def make(cls):
        obj = cls(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"])
        return orc.LsgdOracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)
    return make(orc.Mlp), make(MlpFloat32Accumulation)


def _a17(x, ref):
    return np.abs(x.astype(F64) - ref) / np.maximum(np.abs(ref.astype(F64)), 1e-3)


def test_free_running_trajectory_amplifies_accumulation_differences_beyond_the_elementwise_bound():
    w = inputs.config(3, P=2, G=1, steps=4)
    a, b = _pair(w)
    worst = []
    for t in range(4):
        a.step()
        b.step()
        worst.append(float(_a17(b.x, a.x).max()))
    assert worst[0] <= 2e-2                      # one step from a common state: every entry within the bound
    assert worst[-1] > 2e-2                      # a few free-running steps: not any more, on the CPU alone
    assert all(worst[k + 1] > worst[k] for k in range(2))
    # ... while the bulk stays within it
    assert float((_a17(b.x, a.x) > 2e-2).mean()) <= 2e-2


def test_every_step_from_a_common_state_stays_within_the_elementwise_bound():
    w = inputs.config(3, P=2, G=1, steps=4)
    a, b = _pair(w)
    for t in range(4):
        b.x[...] = a.x
        a.step()
        b.step()
        assert float(_a17(b.x, a.x).max()) <= 2e-2, t
        assert np.allclose(b.obj.last_train_loss, a.obj.last_train_loss, rtol=2e-2, atol=0)
