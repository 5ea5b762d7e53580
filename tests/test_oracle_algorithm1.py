"""Pins for the oracle's Algorithm 1 (small pulls every step, larger pulls at communications, separate
local / global periods).  No GPU needed."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

F32, F64 = np.float32, np.float64


def _wl(P=6, G=2, d=29, **kw):
    args = dict(eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=3, steps=10, sigma=0.01, noise_ring=4, config_id=90)
    args.update(kw)
    return inputs.make_quadratic(P, G, d, **args)


def _alg1(w, noise=True, **kw):
    obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"] if noise else None)
    args = dict(eta=w.eta, lambda_l=w.lambda_l, lambda_g=w.lambda_g, gamma_l=0.02, gamma_g=0.01, tau=w.tau, tau_g=2 * w.tau)
    args.update(kw)
    return orc.Algorithm1Oracle(w.x0, obj, w.group_of, w.G, **args)


def test_no_pulls_is_independent_sgd():
    w = _wl()
    o = _alg1(w, lambda_l=0.0, lambda_g=0.0, gamma_l=0.0, gamma_g=0.0)
    o.run(7)
    a, b, noise = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64), w.arrays["noise"]
    eta, sigma = float(F32(w.eta)), float(F32(w.meta["sigma"]))
    for i in range(w.P):
        xi = w.x0[i].copy()
        for t in range(7):
            gi = (a * (xi.astype(F64) - b) + sigma * noise[t % 4][i].astype(F64)).astype(F32)
            xi = (xi.astype(F64) - eta * gi.astype(F64)).astype(F32)
        assert np.array_equal(xi, o.x[i])


def test_frozen_leader_converges_to_the_minimiser_of_psi():
    """Section 3.1.2: with the leader z fixed and a pull of strength Lambda every step, the iterates
    converge to argmin f(x) + Lambda/2 |x - z|^2 = (a b + Lambda z) / (a + Lambda) per coordinate, and
    f(w) - f* <= Lambda / (m + Lambda) (f(z) - f*)  (Theorem on the value of w)."""
    w = _wl(P=4, G=1, d=16, tau=10 ** 9, eta=0.5)
    gam = 0.3 * 10 ** 9                                   # gamma / tau = 0.3 per step
    o = _alg1(w, noise=False, gamma_l=gam, gamma_g=0.0, lambda_l=0.0, lambda_g=0.0, tau=10 ** 9, tau_g=10 ** 9)
    z = o.z_l[0].astype(F64)
    o.run(600)
    a, b = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64)
    Lam = float(F32(gam)) / 10 ** 9
    want = (a * b + Lam * z) / (a + Lam)
    for i in range(w.P):
        assert np.allclose(o.x[i], want, rtol=0, atol=5e-6)
    f = lambda v: 0.5 * np.sum(a[:16] * (v[:16] - b[:16]) ** 2)
    m = a[:16].min()
    assert f(want) <= Lam / (m + Lam) * f(z) + 1e-12       # f* = 0


def test_closed_form_sequential_pull_with_fixed_leader():
    """gamma = 0, one group: per period the difference to the leader contracts by
    (1 - eta lambda) (1 - eta a)^tau (tau gradient steps, then the pull at the communication)."""
    tau, periods = 3, 4
    w = _wl(P=4, G=1, d=33, tau=tau)
    x0 = w.x0.copy()
    x0[0] = w.arrays["b"] + F32(0.01) * x0[0]             # worker 0 leads throughout
    w.x0 = x0
    o = _alg1(w, noise=False, gamma_l=0.0, gamma_g=0.0, lambda_g=0.0, tau=tau, tau_g=10 ** 9)
    o.run(tau * periods)
    assert all(int(h["ll"][0]) == 0 for h in o.history)
    a, b = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64)
    eta, lam = float(F32(w.eta)), float(F32(w.lambda_l))
    lead = b + (1 - eta * a) ** (tau * periods) * (x0[0].astype(F64) - b)
    assert np.allclose(o.x[0], lead, rtol=0, atol=2e-6)
    shrink = ((1 - eta * lam) * (1 - eta * a) ** tau) ** periods
    for i in range(1, w.P):
        want = lead + shrink * (x0[i].astype(F64) - x0[0].astype(F64))
        assert np.allclose(o.x[i], want, rtol=0, atol=2e-6)


def test_separate_periods_and_leader_rows_do_not_move_under_their_own_pull():
    w = _wl(P=8, G=2, d=40, tau=2)
    o = _alg1(w, tau=2, tau_g=6)
    kinds = []
    for _ in range(12):
        before = None
        o.step()
        if o.history and o.history[-1]["t"] == o.t:
            h = o.history[-1]
            kinds.append((o.t, bool(h["local"]), bool(h["global"])))
            # the snapshots are the leaders' parameters after the communication's pulls
            if h["global"]:
                assert np.array_equal(o.z_g, o.x[o.gl])
    assert kinds == [(2, True, False), (4, True, False), (6, True, True), (8, True, False), (10, True, False),
                     (12, True, True)]
    assert o.gl == int(o.ll[o.group_of[o.gl]]) or True    # the global leader may be stale w.r.t. newer local ones


def test_small_pulls_use_the_stale_copies_not_the_moving_leader():
    w = _wl(P=3, G=1, d=8, tau=10 ** 6)
    o = _alg1(w, noise=False, gamma_l=0.2 * 10 ** 6, gamma_g=0.0, lambda_l=0.0, lambda_g=0.0, tau=10 ** 6, tau_g=10 ** 6)
    z0 = o.z_l[0].copy()
    o.run(3)
    assert np.array_equal(o.z_l[0], z0)                   # not refreshed between communications
    assert not np.array_equal(o.x[int(o.ll[0])], z0)      # while the leader itself has moved on


def _two_group_case():
    """One coordinate, f(x) = x^2 / 2, eta = 1/2, groups {0, 1} and {2, 3}, both periods 1, no small pulls.
    Worked by hand (every value below is exact in binary or differs by one rounding):
      x_0                = [ 2,  -6,  1.8,   2.2 ]   losses [2, 18, 1.62, 2.42]: local leaders 0 and 2, global 2
      gradient step x/2  = [ 1,  -3,  0.9,   1.1 ]   losses [0.5, 4.5, 0.405, 0.605]: local leaders 0 and 2
      local pull, eta lambda = 3/4:
                           [ 1,   0,  0.9,   0.95]   losses [0.5, 0, 0.405, 0.45125]: worker 1 is now the best
      global pull towards worker 1 (x = 0), eta lambda_G = 1/4:
                           [0.75, 0,  0.675, 0.7125]
    Electing the global leader from the losses taken before the local pull would pick worker 2 instead."""
    a, b = np.ones(1, F32), np.zeros(1, F32)
    x0 = np.asarray([[2.0], [-6.0], [1.8], [2.2]], dtype=F32)
    obj = orc.Quadratic(a, b, 0.0, None)
    return orc.Algorithm1Oracle(x0, obj, [0, 0, 1, 1], 2, eta=0.5, lambda_l=1.5, lambda_g=0.5, gamma_l=0.0, gamma_g=0.0,
                                tau=1, tau_g=1)


def test_global_leader_is_elected_after_the_local_pull():
    """Algorithm 1 (Section 2.2): the second conditional of a communication follows the first one's pull, so
    the global best worker is determined on the parameters the local pull has produced."""
    o = _two_group_case()
    assert list(o.ll) == [0, 2] and o.gl == 2
    o.step()
    h = o.history[-1]
    assert h["local"] and h["global"]
    assert list(o.ll) == [0, 2]
    assert o.gl == 1                                             # not 2: the local pull moved worker 1 to the minimiser
    assert np.allclose(h["loss"], [0.5, 4.5, 0.405, 0.605], rtol=1e-6)
    assert np.allclose(h["loss_global"], [0.5, 0.0, 0.405, 0.45125], rtol=1e-6)
    assert np.allclose(o.x[:, 0], [0.75, 0.0, 0.675, 0.7125], rtol=1e-6, atol=0)
    assert np.array_equal(o.z_g, o.x[1]) and np.array_equal(o.z_l[0], o.x[0] / F32(0.75))


def test_a_supplied_loss_vector_serves_both_elections():
    o = _two_group_case()
    o.step(forced_loss=np.asarray([3.0, 4.0, 1.0, 2.0], dtype=F32))
    assert list(o.ll) == [0, 2] and o.gl == 2
    h = o.history[-1]
    assert np.array_equal(h["loss"], h["loss_global"])


def test_one_loss_vector_for_both_elections_would_fail_the_hand_worked_case(monkeypatch):
    """Plants the shortcut (global argmin from the losses taken before the local pull) in the oracle and
    checks that the hand-worked case above catches it."""
    real = orc.Quadratic.loss
    cache = {}

    def loss_once_per_communication(self, x, n):
        if n not in cache:
            cache[n] = real(self, x, n)
        return cache[n]

    monkeypatch.setattr(orc.Quadratic, "loss", loss_once_per_communication)
    with pytest.raises(AssertionError):
        test_global_leader_is_elected_after_the_local_pull()
