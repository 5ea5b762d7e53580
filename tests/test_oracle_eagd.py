"""Pins for the oracle's EAGD (elastic averaging) comparison line: supplement, "Low-Rank Matrix Completion
Experiments" (the update and the center rule) and "LGD versus EAGD: Illustrative Example" (the toy table)."""
import math
import os

import numpy as np

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

F32, F64 = np.float32, np.float64
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _toy():
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


def _sinc(p):
    u = math.pi * math.hypot(p[0], p[1])
    return math.sin(u) / u


def _sinc_grad(p):
    r = math.hypot(p[0], p[1])
    u = math.pi * r
    dldr = (math.cos(u) * u - math.sin(u)) / (u * u) * math.pi
    return np.asarray([dldr * p[0] / r, dldr * p[1] / r])


def test_toy_problem_reaches_the_value_the_paper_prints_for_eagd():
    """4 workers from the listed starts, learning rate 0.1, beta = p eta lambda = 0.43: EAGD settles on the second
    ring of the sinc surface, L = -0.0912 in the paper's table, while LGD reaches the global ring (-0.2172)."""
    starts, kv = _toy()
    eta, beta = kv["eta"], kv["eagd_beta"]
    lam = beta / (len(starts) * eta)
    o = orc.EagdOracle(starts, orc.FromCallables(_sinc_grad, _sinc), eta, lam, tau=int(kv["tau"]))
    o.run(100)
    assert abs(_sinc(o.center.astype(F64)) - kv["eagd_optimum"]) <= 1e-4
    o.run(900)
    ring2 = -0.0913252                                   # second local minimum of sin(pi r) / (pi r), r = 3.4709
    assert abs(_sinc(o.center.astype(F64)) - ring2) <= 1e-6
    assert all(abs(_sinc(o.x[i].astype(F64)) - ring2) <= 1e-6 for i in range(4))
    assert _sinc(o.center.astype(F64)) > kv["lgd_optimum"] + 0.1     # and not the global ring LGD finds


def test_center_rule_special_cases():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((8, 37)).astype(F32)
    c = rng.standard_normal(37).astype(F32)
    # p eta lambda = 1: the new center is the workers' mean, whatever the old center was
    assert np.array_equal(orc.eagd_center_update(c, x, 0.125, 1.0), orc.center_variable(x))
    # eta lambda = 0: the center does not move
    assert np.array_equal(orc.eagd_center_update(c, x, 0.125, 0.0), c)
    # all workers at the center, p eta lambda = 1/2: (1/2) c + (1/2) c = c exactly
    same = np.repeat(c[None, :], 8, axis=0)
    assert np.array_equal(orc.eagd_center_update(c, same, 0.0625, 1.0), c)
    # written out for one coordinate
    got = orc.eagd_center_update(c, x, 0.01, 0.2)
    k = 8 * float(F32(0.01)) * float(F32(0.2))
    want = (1 - k) * float(c[3]) + k * float(np.sum(x[:, 3].astype(F64)) / 8)
    assert abs(float(got[3]) - want) <= 1e-7 * max(1.0, abs(want))


def test_workers_at_the_center_at_a_stationary_point_do_not_move():
    w = inputs.make_quadratic(5, 1, 40, eta=0.05, lambda_l=0.3, lambda_g=0.0, tau=1, steps=3, config_id=130)
    b = w.arrays["b"]
    x0 = np.repeat(b[None, :], 5, axis=0)
    o = orc.EagdOracle(x0, orc.Quadratic(w.arrays["a"], b, 0.0, None), 0.05, 0.3)
    o.run(3)
    assert np.array_equal(o.x, x0) and np.array_equal(o.center, b)


def test_workers_pull_towards_the_old_center_and_zero_strength_is_plain_gd():
    w = inputs.make_quadratic(4, 1, 24, eta=0.05, lambda_l=0.0, lambda_g=0.0, tau=1, steps=3, sigma=0.0, config_id=131)
    a, b = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64)
    obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.0, None)
    o = orc.EagdOracle(w.x0, obj, 0.05, 0.0)
    o.run(2)
    x = w.x0.copy()
    for _ in range(2):
        x = (x.astype(F64) - float(F32(0.05)) * (a * (x.astype(F64) - b)).astype(F32).astype(F64)).astype(F32)
    assert np.array_equal(o.x, x)
    # with a pull: one step written out, X+ = (1 - eta lambda) X + eta lambda Z - eta grad F(X), Z the OLD center
    o = orc.EagdOracle(w.x0, obj, 0.05, 0.4)
    z = o.center.astype(F64)
    o.step()
    eta, lam = float(F32(0.05)), float(F32(0.4))
    g = (a * (w.x0.astype(F64) - b)).astype(F32).astype(F64)
    want = (1 - eta * lam) * w.x0.astype(F64) + eta * lam * z - eta * g
    assert np.allclose(o.x, want, rtol=0, atol=2e-7)


def test_closed_form_on_the_diagonal_quadratic():
    """Exact gradients on f = 1/2 sum a (x - b)^2: per coordinate the workers' mean m and the center c follow
    the 2 x 2 recursion  m+ = (1 - eta a - eta lam) m + eta lam c + eta a b,  c+ = (1 - p eta lam) c + p eta lam m,
    and each worker's deviation from the mean contracts by (1 - eta a - eta lam)."""
    P, d, T = 6, 20, 25
    w = inputs.make_quadratic(P, 1, d, eta=0.05, lambda_l=0.0, lambda_g=0.0, tau=1, steps=T, sigma=0.0, config_id=132)
    a, b = w.arrays["a"][:d].astype(F64), w.arrays["b"][:d].astype(F64)
    eta, lam = float(F32(0.05)), float(F32(0.3))
    o = orc.EagdOracle(w.x0, orc.Quadratic(w.arrays["a"], w.arrays["b"], 0.0, None), 0.05, 0.3)
    x0 = w.x0[:, :d].astype(F64)
    m, c = x0.mean(axis=0), x0.mean(axis=0)
    dev = x0 - m
    o.run(T)
    for _ in range(T):
        m, c = (1 - eta * a - eta * lam) * m + eta * lam * c + eta * a * b, (1 - P * eta * lam) * c + P * eta * lam * m
        dev = (1 - eta * a - eta * lam) * dev
    assert np.allclose(o.center[:d], c, rtol=0, atol=5e-6)
    assert np.allclose(o.x[:, :d], m + dev, rtol=0, atol=5e-6)
