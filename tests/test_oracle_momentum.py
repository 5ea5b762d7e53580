"""Pins for the oracle's Section 4.1 optimiser (Nesterov momentum + weight decay around the LSGD step):
reductions to Eq. (1), to a library optimiser, and closed forms on the diagonal quadratic.  No GPU needed."""
import numpy as np

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

F32, F64 = np.float32, np.float64


def _workload(P=6, G=2, d=29, **kw):
    args = dict(eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=9, sigma=0.01, noise_ring=4, config_id=44)
    args.update(kw)
    return inputs.make_quadratic(P, G, d, **args)


def _oracle(w, noise=True, **over):
    obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"] if noise else None)
    hp = dict(eta=w.eta, lambda_l=w.lambda_l, lambda_g=w.lambda_g, tau=w.tau)
    hp.update(over)
    return orc.LsgdOracle(w.x0, obj, w.group_of, w.G, **hp)


def test_zero_momentum_and_decay_is_eq1():
    """mu = wd = 0: d = g, v+ = g, u = g, so the step is Eq. (1) again (values equal; +-0 compare equal)."""
    w = _workload()
    plain = _oracle(w)
    mom = _oracle(w, momentum=0.0, weight_decay=0.0)
    for _ in range(w.steps):
        plain.step()
        mom.step()
        assert np.array_equal(plain.x, mom.x)
    assert [h["gl"] for h in plain.history] == [h["gl"] for h in mom.history]


def test_without_pulls_it_is_the_library_nesterov_sgd():
    """lambda = 0: every worker runs Nesterov-momentum SGD with L2 weight decay on its own; the same recipe in
    a library optimiser (float64 tensors, same gradients) must agree to float32 storage accuracy."""
    import torch
    w = _workload(sigma=0.0)
    mu, wd, steps = 0.9, 1e-2, 25
    o = _oracle(w, noise=False, lambda_l=0.0, lambda_g=0.0, momentum=mu, weight_decay=wd)
    o.run(steps)
    a = torch.from_numpy(w.arrays["a"].astype(F64))
    b = torch.from_numpy(w.arrays["b"].astype(F64))
    for i in range(w.P):
        p = torch.nn.Parameter(torch.from_numpy(w.x0[i].astype(F64)))
        opt = torch.optim.SGD([p], lr=float(F32(w.eta)), momentum=float(F32(mu)), nesterov=True, weight_decay=float(F32(wd)))
        for _ in range(steps):
            p.grad = (a * (p.detach() - b)).to(torch.float64)
            opt.step()
        ref = p.detach().numpy()
        assert np.max(np.abs(o.x[i].astype(F64) - ref)) <= 2e-6 * max(1.0, np.max(np.abs(ref)))


def test_closed_form_on_the_quadratic_is_a_two_by_two_recurrence():
    """Batch gradient, no pulls, no decay: with e = x - b the pair (e, v) moves by a fixed 2 x 2 matrix per
    coordinate, (e+, v+) = [[1 - eta a (1 + mu), -eta mu^2], [a, mu]] (e, v); n steps are its n-th power."""
    w = _workload(sigma=0.0)
    mu, n = 0.9, 30
    o = _oracle(w, noise=False, lambda_l=0.0, lambda_g=0.0, momentum=mu, weight_decay=0.0)
    o.run(n)
    eta, mu64 = float(F32(w.eta)), float(F32(mu))
    a, b = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64)
    for k in range(w.d):
        M = np.array([[1.0 - eta * a[k] * (1.0 + mu64), -eta * mu64 * mu64], [a[k], mu64]])
        Mn = np.linalg.matrix_power(M, n)
        for i in range(w.P):
            e0 = float(w.x0[i, k]) - b[k]
            e_n, v_n = Mn @ np.array([e0, 0.0])
            assert abs(o.x[i, k] - (b[k] + e_n)) <= 3e-6 * max(1.0, abs(b[k] + e_n))
            assert abs(o.v[i, k] - v_n) <= 3e-6 * max(1.0, abs(v_n))


def test_weight_decay_moves_the_fixed_point():
    """With decay the iteration minimises f(x) + (wd / 2) |x|^2, whose minimiser on the diagonal quadratic is
    a b / (a + wd), whatever the momentum."""
    w = _workload(sigma=0.0, d=11)
    wd = 0.25
    o = _oracle(w, noise=False, lambda_l=0.0, lambda_g=0.0, momentum=0.5, weight_decay=wd, eta=0.2)
    o.run(1500)
    a, b = w.arrays["a"].astype(F64), w.arrays["b"].astype(F64)
    target = a * b / (a + float(F32(wd)))
    assert np.max(np.abs(o.x.astype(F64) - target[None, :])) <= 1e-5


def test_pulls_stay_outside_the_momentum_buffer():
    """One pull step: the buffer is what the lambda = 0 run produces (bit for bit), and x differs from that
    run by exactly the two pull terms of Eq. (1) taken at x_t."""
    w = _workload(sigma=0.0, tau=1)
    mu, wd = 0.9, 1e-3
    with_pull = _oracle(w, noise=False, momentum=mu, weight_decay=wd)
    no_pull = _oracle(w, noise=False, lambda_l=0.0, lambda_g=0.0, momentum=mu, weight_decay=wd)
    # a non-zero buffer first, identical in both
    for o in (with_pull, no_pull):
        o.v[:] = (0.1 * w.arrays["noise"][0]).astype(F32)
    x0 = with_pull.x.astype(F64)
    with_pull.step()
    no_pull.step()
    assert np.array_equal(with_pull.v, no_pull.v)
    ll, gl = with_pull.history[0]["ll"], with_pull.history[0]["gl"]
    eta, cl, cg = float(F32(w.eta)), float(F32(w.lambda_l)), float(F32(w.lambda_g))
    for i in range(w.P):
        zl, zg = x0[ll[w.group_of[i]]], x0[gl]
        expect = no_pull.x[i].astype(F64) - eta * cl * (x0[i] - zl) - eta * cg * (x0[i] - zg)
        assert np.max(np.abs(with_pull.x[i].astype(F64) - expect)) <= 2.5e-7 * max(1.0, np.max(np.abs(expect)))
    # the global leader feels no pull at all: its step is the lambda = 0 step exactly
    assert np.array_equal(with_pull.x[gl], no_pull.x[gl])
