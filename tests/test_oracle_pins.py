"""Pins for the CPU oracle: facts the paper and the mathematics fix, none of them produced by the
oracle itself.  Each test names the passage it rests on.  No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

F32, F64 = np.float32, np.float64
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _small_quadratic(P=6, G=2, d=37, **kw):
    args = dict(eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=7, sigma=0.01, noise_ring=4,
                config_id=40)
    args.update(kw)
    return inputs.make_quadratic(P, G, d, **args)


def _oracle_for(w, noise=True, **over):
    obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"] if noise else None)
    hp = dict(eta=w.eta, lambda_l=w.lambda_l, lambda_g=w.lambda_g, tau=w.tau)
    hp.update(over)
    return orc.LsgdOracle(w.x0, obj, w.group_of, w.G, **hp)


# ---- P1: lambda = 0 reduces to P independent SGD runs (Eq. (1) with both pulls removed) ---------
def test_zero_pull_is_independent_sgd():
    w = _small_quadratic()
    o = _oracle_for(w, lambda_l=0.0, lambda_g=0.0)
    o.run(w.steps)
    a, b, noise = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64), w.arrays["noise"]
    eta, sigma = float(F32(w.eta)), float(F32(w.meta["sigma"]))
    for i in range(w.P):                                  # stand-alone SGD, one worker at a time
        xi = w.x0[i].copy()
        for t in range(w.steps):
            gi = (a * (xi.astype(F64) - b) + sigma * noise[t % 4][i].astype(F64)).astype(F32)
            xi = (xi.astype(F64) - eta * gi.astype(F64)).astype(F32)
        assert np.array_equal(xi, o.x[i])


# ---- P2: the leader's own step is a plain (S)GD step (supplement, "Definitions and Notation") ---
def test_leader_step_is_plain_sgd_step():
    w = _small_quadratic(tau=1)
    o = _oracle_for(w)
    for _ in range(4):
        x_before = o.x.copy()
        o.step()
        g = o.obj.grad(x_before, o.t - 1)
        gl = o.gl
        plain = (x_before[gl].astype(F64) - float(F32(w.eta)) * g[gl].astype(F64)).astype(F32)
        assert np.array_equal(o.x[gl], plain)            # global leader: both pulls vanish
        for j, l in enumerate(o.ll):                     # local leader: only the global pull acts
            if l == gl:
                continue
            xi = x_before[l].astype(F64)
            want = xi - float(F32(w.eta)) * g[l].astype(F64) \
                - float(F32(w.eta)) * float(F32(w.lambda_g)) * (xi - x_before[gl].astype(F64))
            assert np.array_equal(o.x[l], want.astype(F32))


# ---- P3: multiple leaders == one combined guide point (Section 3, first paragraph) -------------
def test_two_pulls_equal_one_combined_pull():
    w = _small_quadratic(P=8, G=2, d=64)
    rng = np.random.default_rng(5)
    g = rng.standard_normal(w.x0.shape).astype(F32)
    ll, gl = np.array([2, 5], dtype=np.int32), 5
    x = w.x0.copy()
    orc.update(x, g, w.group_of, ll, gl, w.eta, w.lambda_l, w.lambda_g, True)
    eta, l1, l2 = float(F32(w.eta)), float(F32(w.lambda_l)), float(F32(w.lambda_g))
    Lam = l1 + l2
    for i in range(w.P):
        xi = w.x0[i].astype(F64)
        z = (l1 * w.x0[ll[w.group_of[i]]].astype(F64) + l2 * w.x0[gl].astype(F64)) / Lam
        want = xi - eta * (g[i].astype(F64) + Lam * (xi - z))          # Section 3.1.1 iteration
        assert np.allclose(x[i], want, rtol=0, atol=2e-7 * (1 + np.abs(want).max()))


def test_single_group_is_single_leader_lsgd():
    # lambda_G term "disappears" in the single-leader setting; with G = 1 the two leaders coincide
    w = _small_quadratic(P=5, G=1, d=33, tau=1)
    o2 = _oracle_for(w)
    o1 = _oracle_for(w, lambda_l=float(F32(w.lambda_l)) + float(F32(w.lambda_g)), lambda_g=0.0)
    for _ in range(5):
        o1.step()
        o2.step()
        assert o2.gl == int(o2.ll[0])
    assert np.allclose(o1.x, o2.x, rtol=0, atol=1e-6)


# ---- written-out update of the matrix-completion section: X+ = (1-eta lam)X + eta lam Z - eta G --
def test_update_matches_written_out_form():
    rng = np.random.default_rng(11)
    P, d = 4, 50
    x0 = rng.standard_normal((P, d)).astype(F32)
    g = rng.standard_normal((P, d)).astype(F32)
    eta, lam = 5e-4, 0.2                                   # the section's own settings
    x = x0.copy()
    orc.update(x, g, np.zeros(P, np.int32), np.array([1], np.int32), 1, eta, lam, 0.0, True)
    e, l = float(F32(eta)), float(F32(lam))
    want = (1 - e * l) * x0.astype(F64) + e * l * x0[1].astype(F64) - e * g.astype(F64)
    assert np.allclose(x, want, rtol=0, atol=3e-7)
    # and it is NOT the unscaled form printed in Eq. (1):
    unscaled = x0.astype(F64) - e * g.astype(F64) - l * (x0.astype(F64) - x0[1].astype(F64))
    assert np.abs(x - unscaled).max() > 1e-2


# ---- P4: all workers at a stationary point is a fixed point (Section 3.2) -----------------------
@pytest.mark.parametrize("tau", [1, 3])
def test_coincident_stationary_point_is_fixed(tau):
    w = _small_quadratic(tau=tau)
    x0 = np.tile(w.arrays["b"], (w.P, 1)).astype(F32)
    obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.0, None)
    o = orc.LsgdOracle(x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, tau)
    o.run(6)
    assert np.array_equal(o.x, x0)


# ---- P5: closed-form linear recursion of batch LGD on the diagonal quadratic --------------------
def test_closed_form_single_leader_tau1():
    # C0's shape.  While worker w leads:  w_t - b = (1-eta a)^t (w_0 - b),
    # x_t - w_t = (1 - eta (a + lambda))^t (x_0 - w_0).
    wl = inputs.config(0)
    x0 = wl.x0.copy()
    x0[0] = wl.arrays["b"] + F32(0.01) * x0[0]            # worker 0 starts closest and stays leader
    obj = orc.Quadratic(wl.arrays["a"], wl.arrays["b"], 0.0, None)
    o = orc.LsgdOracle(x0, obj, wl.group_of, 1, wl.eta, wl.lambda_l, 0.0, 1)
    T = 10
    o.run(T)
    assert all(h["gl"] == 0 for h in o.history)
    a, b = wl.arrays["a"].astype(F64), wl.arrays["b"].astype(F64)
    eta, lam = float(F32(wl.eta)), float(F32(wl.lambda_l))
    w_t = b + (1 - eta * a) ** T * (x0[0].astype(F64) - b)
    assert np.allclose(o.x[0], w_t, rtol=0, atol=2e-6)
    for i in range(1, wl.P):
        x_t = w_t + (1 - eta * (a + lam)) ** T * (x0[i].astype(F64) - x0[0].astype(F64))
        assert np.allclose(o.x[i], x_t, rtol=0, atol=2e-6)


def test_closed_form_multi_leader_with_period():
    # global leader w, other groups' local leaders v, members x.  Per coordinate:
    #   pull step:  (w-b) *= 1-eta a ; (v-w) *= 1-eta(a+lam_g) ; (x-v) *= 1-eta(a+lam_l+lam_g)
    #   other step: every difference *= 1-eta a
    P, G, d, tau, T = 9, 3, 41, 3, 11
    wl = inputs.make_quadratic(P, G, d, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=tau, steps=T,
                               config_id=41)
    b32 = wl.arrays["b"]
    x0 = wl.x0.copy()
    x0[0] = b32 + F32(0.01) * x0[0]
    for lead in (3, 6):
        x0[lead] = b32 + F32(0.1) * x0[lead]
    obj = orc.Quadratic(wl.arrays["a"], b32, 0.0, None)
    o = orc.LsgdOracle(x0, obj, wl.group_of, G, wl.eta, wl.lambda_l, wl.lambda_g, tau)
    o.run(T)
    for h in o.history:
        assert h["gl"] == 0 and list(h["ll"]) == [0, 3, 6]
    a, b = wl.arrays["a"].astype(F64), b32.astype(F64)
    eta, ll_, lg_ = float(F32(wl.eta)), float(F32(wl.lambda_l)), float(F32(wl.lambda_g))
    n_pull = len([t for t in range(T) if t % tau == 0])
    n_plain = T - n_pull
    base = (1 - eta * a) ** n_plain
    cw = base * (1 - eta * a) ** n_pull
    cv = base * (1 - eta * (a + lg_)) ** n_pull
    cx = base * (1 - eta * (a + ll_ + lg_)) ** n_pull
    X0 = x0.astype(F64)
    w_t = b + cw * (X0[0] - b)
    for i in range(P):
        lead = [0, 3, 6][wl.group_of[i]]
        v_t = w_t + (cv * (X0[lead] - X0[0]) if lead != 0 else 0.0)
        x_t = v_t + (cx * (X0[i] - X0[lead]) if i != lead else 0.0)
        assert np.allclose(o.x[i], x_t[: wl.ld], rtol=0, atol=3e-6), i


# ---- P6: election == brute force on exhaustive tiny inputs; tie rule = lowest index --------------
def _key(v):
    v = float(v)
    return (1, 0.0) if math.isnan(v) else (0, v)           # tuple order: numbers < NaN; -0.0 == 0.0


def _brute_argmin(loss, members):
    for i in members:                                      # i wins iff nobody beats it and no
        if all(not (_key(loss[j]) < _key(loss[i])) and     # earlier member ties with it
               (j >= i or _key(loss[i]) < _key(loss[j])) for j in members):
            return i
    raise AssertionError("no argmin")


def _surjections(P, G):
    for m in itertools.product(range(G), repeat=P):
        if len(set(m)) == G:
            yield m


def test_election_matches_brute_force_exhaustively():
    vals = [-math.inf, -1.0, -0.0, 0.0, 1.0, math.inf, math.nan]
    for P in (1, 2, 3, 4):
        maps = [m for G in range(1, P + 1) for m in _surjections(P, G)]
        for combo in itertools.product(vals, repeat=P):
            loss = np.asarray(combo, dtype=F32)
            for m in maps:
                G = max(m) + 1
                ll, gl = orc.elect(loss, m, G)
                for j in range(G):
                    assert ll[j] == _brute_argmin(loss, [i for i in range(P) if m[i] == j])
                assert gl == _brute_argmin(loss, list(range(P)))


def _set_partitions(P):
    """Every grouping of P workers up to renaming the groups (restricted-growth strings)."""
    def rec(prefix, n_used):
        if len(prefix) == P:
            yield tuple(prefix)
            return
        for j in range(n_used + 1):
            yield from rec(prefix + [j], max(n_used, j + 1))
    yield from rec([], 0)


def _exhaustive_election(P):
    vals = [-1.0, -0.0, 0.0, 1.0, math.inf, math.nan]
    parts = [(m, max(m) + 1, [[i for i in range(P) if m[i] == j] for j in range(max(m) + 1)])
             for m in _set_partitions(P)]
    for combo in itertools.product(vals, repeat=P):
        loss = np.asarray(combo, dtype=F32)
        best = {}
        for m, G, members in parts:
            ll, gl = orc.elect(loss, m, G)
            for j in range(G):
                key = tuple(members[j])
                if key not in best:
                    best[key] = _brute_argmin(loss, members[j])
                assert ll[j] == best[key], (combo, m)
            key = tuple(range(P))
            if key not in best:
                best[key] = _brute_argmin(loss, list(range(P)))
            assert gl == best[key], (combo, m)


def test_election_matches_brute_force_five_workers_all_groupings():
    _exhaustive_election(5)                                # 6^5 loss vectors x 52 groupings


@pytest.mark.slow
def test_election_matches_brute_force_six_workers_all_groupings():
    _exhaustive_election(6)                                # 6^6 loss vectors x 203 groupings; run with --runslow


def test_election_tie_examples():
    ll, gl = orc.elect(np.asarray([0.5, 0.5, 0.25, 0.25], F32), [0, 0, 1, 1], 2)
    assert list(ll) == [0, 2] and gl == 2
    ll, gl = orc.elect(np.asarray([np.nan, np.inf, np.nan, np.nan], F32), [0, 0, 1, 1], 2)
    assert list(ll) == [1, 2] and gl == 1                  # +inf beats NaN; all-NaN group: lowest
    ll, gl = orc.elect(np.asarray([0.0, -0.0, -0.0], F32), [0, 0, 0], 1)
    assert list(ll) == [0] and gl == 0                     # signed zeros tie


# ---- P8: the global leader is the best of the local leaders (Section 2.2) -----------------------
def test_global_leader_is_a_local_leader():
    rng = np.random.default_rng(3)
    for _ in range(300):
        P = int(rng.integers(1, 20))
        G = int(rng.integers(1, P + 1))
        m = np.concatenate([np.arange(G), rng.integers(0, G, P - G)])
        rng.shuffle(m)
        loss = rng.integers(0, 4, P).astype(F32)           # many ties
        ll, gl = orc.elect(loss, m, G)
        assert all(m[ll[j]] == j for j in range(G))
        assert gl == ll[m[gl]]
        assert gl == min(ll, key=lambda i: (loss[i], i))


# ---- P7: the paper's toy problem (value printed in the supplement's table) ----------------------
def _read_toy():
    starts, kv = [], {}
    with open(os.path.join(GOLDEN, "toy_sinc.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            if k == "start":
                starts.append([float(t) for t in v])
            else:
                kv[k] = float(v[0])
    return np.asarray(starts), kv


def test_toy_sinc_reaches_printed_optimum():
    starts, kv = _read_toy()

    def L(p):
        r = math.pi * math.hypot(p[0], p[1])
        return math.sin(r) / r

    def dL(p):
        rho = math.hypot(p[0], p[1])
        r = math.pi * rho
        dr = (r * math.cos(r) - math.sin(r)) / (r * r)     # d/dr sinc
        return np.asarray([dr * math.pi * p[0] / rho, dr * math.pi * p[1] / rho])

    o = orc.LsgdOracle(starts.astype(F32), orc.FromCallables(dL, L), np.zeros(4, np.int32), 1,
                       kv["eta"], kv["lambda"], 0.0, int(kv["tau"]))
    o.run(3000)
    best = min(L(o.x[i].astype(F64)) for i in range(4))
    assert round(best, 4) == kv["lgd_optimum"]
    assert best > -0.21724                                  # global minimum of sinc is -0.217234


# ---- P9: leader descent lemma: noise-free LGD with eta < 2/M never worsens the leader -----------
@pytest.mark.parametrize("tau", [1, 4])
def test_leader_loss_is_monotone_without_noise(tau):
    w = _small_quadratic(P=8, G=2, d=128, tau=tau, eta=0.5)   # M = max a <= 1, so eta < 2/M
    o = _oracle_for(w, noise=False)
    o.run(40)
    best = [float(h["loss"].min()) for h in o.history]
    assert all(b1 <= b0 * (1 + 1e-6) for b0, b1 in zip(best, best[1:]))
    assert best[-1] < 0.2 * best[0]


# ---- P10: gradients against finite differences, autograd and the dense formula ------------------
def _fd(f, x, h=1e-6):
    g = np.zeros_like(x)
    for k in range(x.size):
        e = np.zeros_like(x)
        e[k] = h
        g[k] = (f(x + e) - f(x - e)) / (2 * h)
    return g


def test_quadratic_gradient_and_loss():
    w = _small_quadratic(P=2, G=1, d=9)
    a, b = w.arrays["a"].astype(F64)[:9], w.arrays["b"].astype(F64)[:9]
    obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.0, None)
    g = obj.grad(w.x0, 0)
    loss = obj.loss(w.x0, 0)
    for i in range(2):
        f = lambda v: 0.5 * sum(a[k] * (v[k] - b[k]) ** 2 for k in range(9))
        assert np.allclose(g[i, :9], _fd(f, w.x0[i, :9].astype(F64)), atol=1e-6)
        assert math.isclose(loss[i], f(w.x0[i, :9].astype(F64)), rel_tol=1e-6)
    # noise enters additively with weight sigma
    objn = orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.01, w.arrays["noise"])
    gn = objn.grad(w.x0, 1)
    assert np.allclose(gn - g, F32(0.01) * w.arrays["noise"][1], atol=1e-7)


def _tiny_matcomp(full=False):
    n_rows, n_cols, rank = 6, 5, 2
    n_obs = 30 if full else 17
    return inputs.make_matcomp(3, 1, n_rows=n_rows, n_cols=n_cols, rank=rank, n_obs=n_obs,
                               n_heldout=8, batch=n_obs if full else 12, steps=2, config_id=42)


def _matcomp_obj(w):
    m, A = w.meta, w.arrays
    return orc.MatComp(m["n_rows"], m["n_cols"], m["rank"], A["obs_r"], A["obs_c"], A["obs_v"],
                       A["batch_pos"], A["heldout_pos"])


def test_matcomp_gradient_finite_differences_with_duplicates():
    w = _tiny_matcomp()
    w.arrays["batch_pos"][0, 0, :4] = w.arrays["batch_pos"][0, 0, 4]     # force duplicates
    obj = _matcomp_obj(w)
    g = obj.grad(w.x0, 0)
    m, A = w.meta, w.arrays
    nx = m["n_rows"] * m["rank"]
    for i in range(w.P):
        pos = A["batch_pos"][0][i]

        def f(v):
            X = v[:nx].reshape(m["n_rows"], m["rank"])
            Y = v[nx:].reshape(m["n_cols"], m["rank"])
            tot = 0.0
            for p in pos:
                e = float(X[A["obs_r"][p]] @ Y[A["obs_c"][p]]) - float(A["obs_v"][p])
                tot += e * e
            return tot / (2 * len(pos))

        assert np.allclose(g[i, :w.d], _fd(f, w.x0[i, :w.d].astype(F64)), atol=2e-7)


def test_matcomp_all_cells_equals_dense_formula():
    w = _tiny_matcomp(full=True)
    A, m = w.arrays, w.meta
    A["batch_pos"][0, :, :] = np.arange(30, dtype=np.int32)             # every cell exactly once
    obj = _matcomp_obj(w)
    g = obj.grad(w.x0, 0)
    M = np.zeros((m["n_rows"], m["n_cols"]))
    M[A["obs_r"], A["obs_c"]] = A["obs_v"]
    nx = m["n_rows"] * m["rank"]
    for i in range(w.P):
        X = w.x0[i, :nx].astype(F64).reshape(m["n_rows"], m["rank"])
        Y = w.x0[i, nx:w.d].astype(F64).reshape(m["n_cols"], m["rank"])
        R = X @ Y.T - M
        assert np.allclose(g[i, :nx].reshape(X.shape), R @ Y / 30, atol=1e-7)
        assert np.allclose(g[i, nx:w.d].reshape(Y.shape), R.T @ X / 30, atol=1e-7)
    # held-out loss = plain mean of squared residuals
    loss = obj.loss(w.x0, 0)
    hp = A["heldout_pos"]
    X = w.x0[0, :nx].astype(F64).reshape(m["n_rows"], m["rank"])
    Y = w.x0[0, nx:w.d].astype(F64).reshape(m["n_cols"], m["rank"])
    e = [(X[A["obs_r"][p]] @ Y[A["obs_c"][p]]) - A["obs_v"][p] for p in hp]
    assert math.isclose(loss[0], np.mean(np.square(e)), rel_tol=1e-6)


def _tiny_mlp(mode):
    w = inputs.make_mlp(2, 1, dims=(5, 4, 4, 3), pool=40, heldout=16, batch=8, n_classes=3, steps=2,
                        config_id=43)
    rng = np.random.default_rng(0)
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    for s in segs:                                                     # non-zero biases for the check
        w.x0[:, s["b"]:s["b"] + s["n_out"]] = rng.standard_normal((2, s["n_out"])).astype(F32) * 0.1
    A = w.arrays
    obj = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode=mode)
    return w, segs, obj


def _torch_mlp_loss_and_grad(w, segs, xi, inp, y):
    import torch
    p = torch.tensor(xi.astype(F64), requires_grad=True)
    h = torch.tensor(inp.astype(F64))
    for l, s in enumerate(segs):
        W = p[s["w"]:s["w"] + s["n_in"] * s["n_out"]].reshape(s["n_out"], s["n_in"])
        h = h @ W.T + p[s["b"]:s["b"] + s["n_out"]]
        if l < len(segs) - 1:
            h = torch.relu(h)
    loss = torch.nn.functional.cross_entropy(h, torch.tensor(y.astype(np.int64)))
    loss.backward()
    return float(loss), p.grad.numpy()


def test_mlp_fp32_gradient_matches_autograd():
    w, segs, obj = _tiny_mlp("fp32")
    g = obj.grad(w.x0, 0)
    A = w.arrays
    for i in range(w.P):
        idx = A["batch_idx"][0][i]
        loss, gref = _torch_mlp_loss_and_grad(w, segs, w.x0[i], A["pool_x"][idx], A["pool_y"][idx])
        assert np.allclose(g[i], gref, atol=1e-6)
        assert math.isclose(obj.last_train_loss[i], loss, rel_tol=1e-6)
    held = obj.loss(w.x0, 0)
    loss, _ = _torch_mlp_loss_and_grad(w, segs, w.x0[0], A["held_x"], A["held_y"])
    assert math.isclose(held[0], loss, rel_tol=1e-6)


def test_mlp_full_width_gradient_matches_autograd():
    w = inputs.make_mlp(1, 1, pool=256, heldout=32, batch=16, steps=1, config_id=44)
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    A = w.arrays
    obj = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="fp32")
    g = obj.grad(w.x0, 0)
    idx = A["batch_idx"][0][0]
    _, gref = _torch_mlp_loss_and_grad(w, segs, w.x0[0], A["pool_x"][idx], A["pool_y"][idx])
    assert np.allclose(g[0], gref, atol=2e-6)


def test_mlp_bf16emu_is_close_to_fp32_and_rounding_matches_library():
    import torch
    v = np.random.default_rng(1).standard_normal(10000).astype(F32) * 3
    v[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]                  # exact ties -> even
    want = torch.tensor(v).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(orc.bf16_round(v), want)
    w, segs, o32 = _tiny_mlp("fp32")
    _, _, o16 = _tiny_mlp("bf16emu")
    g32, g16 = o32.grad(w.x0, 0), o16.grad(w.x0, 0)
    assert np.abs(g32 - g16).max() <= 2e-2 * np.abs(g32).max()
    assert not np.array_equal(g32, g16)


def test_mlp_bf16emu_rounds_operands_only():
    """Where every matrix-product operand is exactly representable in bfloat16 -- small integers for the data, the
    weights and hence the hidden activations -- rounding the operands changes nothing: the bf16-emulation mode must
    give the fp32 mode's losses bit for bit (forward pass and held-out loss), and its gradient of the last layer,
    whose operands are the representable activations and the rounded dZ, must be the fp32 mode's within the one
    rounding of dZ (2^-9 relative)."""
    w, segs, o32 = _tiny_mlp("fp32")
    rng = np.random.default_rng(4)
    A = w.arrays
    A["pool_x"][...] = rng.integers(-3, 4, A["pool_x"].shape).astype(F32)
    A["held_x"][...] = rng.integers(-3, 4, A["held_x"].shape).astype(F32)
    x0 = w.x0.copy()
    x0[...] = rng.integers(-2, 3, x0.shape).astype(F32)
    o16 = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="bf16emu")
    o32 = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="fp32")
    assert np.array_equal(o16.loss(x0, 0), o32.loss(x0, 0))
    g16, g32 = o16.grad(x0, 0), o32.grad(x0, 0)
    assert np.array_equal(o16.last_train_loss, o32.last_train_loss)
    s3 = segs[-1]
    a, b = g16[:, s3["w"]:s3["w"] + s3["n_in"] * s3["n_out"]], g32[:, s3["w"]:s3["w"] + s3["n_in"] * s3["n_out"]]
    assert np.abs(a - b).max() <= 2.0 ** -8 * np.abs(b).max() + 1e-12
    assert np.abs(b).max() > 0


# ---- center variable = plain average of the workers (Section 4.1) ---------------------------------
def test_center_variable_is_the_average():
    rng = np.random.default_rng(8)
    x = rng.standard_normal((7, 50)).astype(F32)
    c = orc.center_variable(x)
    assert np.allclose(c, x.astype(F64).mean(axis=0), rtol=0, atol=1e-7)
    assert np.array_equal(orc.center_variable(np.tile(x[:1], (5, 1))), x[0])     # identical workers


# ---- the paper's completion experiment: F = 1/4 ||M - X X^T||^2, grad = (X X^T - M) X ---------------
def test_psd_completion_gradient_and_monotone_descent():
    w = inputs.make_psd(P=3, n=7, r=2, steps=3, config_id=45)
    obj = orc.PsdCompletion(7, 2, w.arrays["M"])
    g = obj.grad(w.x0, 0)
    loss = obj.loss(w.x0, 0)
    M = w.arrays["M"].astype(F64)
    for i in range(w.P):
        f = lambda v: 0.25 * np.sum((M - v.reshape(7, 2) @ v.reshape(7, 2).T) ** 2)
        x = w.x0[i, :14].astype(F64)
        assert np.allclose(g[i, :14], _fd(f, x, h=1e-5), rtol=1e-6, atol=1e-6)
        assert math.isclose(loss[i], f(x), rel_tol=1e-6)
    # "a value was found for which both methods exhibited monotonic decrease": LGD at the paper's settings
    w = inputs.make_psd(P=8, n=120, r=10, steps=60, config_id=46)
    o = orc.LsgdOracle(w.x0, orc.PsdCompletion(120, 10, w.arrays["M"]), w.group_of, 1, w.eta, w.lambda_l, 0.0, 1)
    o.run(60)
    best = [float(h["loss"].min()) for h in o.history]
    assert all(b1 <= b0 for b0, b1 in zip(best, best[1:])) and best[-1] < 0.5 * best[0]


# ---- running-mean election loss of the deep-network runs (Section 4.1) ------------------------------
def test_mlp_running_mean_election_loss():
    w, segs, _ = _tiny_mlp("fp32")
    A = w.arrays
    obj = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="fp32", loss_window=3)
    seen = []
    for t in range(5):
        obj.grad(w.x0 * F32(1.0 + 0.1 * t), t)
        seen.append(obj.last_train_loss.astype(F64))
        want = np.mean(seen[-3:], axis=0)
        assert np.allclose(obj.loss(w.x0, 0), want, rtol=1e-6, atol=0)
