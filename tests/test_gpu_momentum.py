"""GPU parity of the Section 4.1 optimiser (Nesterov momentum + weight decay around the LSGD step), through
the C ABI, against the CPU oracle: parameters AND momentum buffers bit-identical in the default arithmetic,
within the trajectory tolerance in the two faster modes; mu = wd = 0 equals the plain path; the MLP objective
keeps its bf16 weight copy in step."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu

F32 = np.float32
TOL = 1e-5


def rel_err(x, ref, floor):
    return float((np.abs(x.astype(np.float64) - ref) / np.maximum(np.abs(ref), floor)).max())


def _pop(w, **kw):
    from paper_1905_10395_b200.runner import Population
    return Population(w, **kw)


@pytest.mark.parametrize("arith,exact", [(0, True), (1, False), (2, False)])
def test_external_gradients_ragged_unequal_groups(arith, exact):
    group_of = np.asarray([2, 0, 1, 1, 0, 2, 2, 1, 0], dtype=np.int32)
    w = inputs.make_external(9, 3, 70001, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=3, steps=10, loss_ring=5,
                             config_id=52, group_of=group_of)
    mu, wd = 0.9, 1e-4
    pop = _pop(w, arithmetic=arith, momentum=mu, weight_decay=wd)
    pop.run(10, record=True)
    o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau, momentum=mu, weight_decay=wd)
    o.run(10)
    assert [h["gl"] for h in pop.history] == [h["gl"] for h in o.history]
    for hg, ho in zip(pop.history, o.history):
        assert np.array_equal(hg["ll"], ho["ll"])
    x, v = pop.x_host(), pop.v.cpu().numpy()
    if exact:
        assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
        assert np.array_equal(v.view(np.uint32), o.v.view(np.uint32))
    assert rel_err(x, o.x, 1.0 if arith == 2 else 1e-3) <= TOL
    assert rel_err(v, o.v, 1.0 if arith == 2 else 1e-3) <= TOL
    assert np.all(x[:, w.d:] == 0) and np.all(v[:, w.d:] == 0)
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_quadratic_with_noise_bit_exact_and_single_worker():
    for (P, G, d) in [(6, 2, 1037), (1, 1, 33), (64, 8, 260)]:
        w = inputs.make_quadratic(P, G, d, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=8, sigma=0.01,
                                  noise_ring=4, config_id=53)
        pop = _pop(w, momentum=0.9, weight_decay=1e-3)
        pop.run(8, record=True)
        o = orc.LsgdOracle(w.x0, orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"]),
                           w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau, momentum=0.9, weight_decay=1e-3)
        o.run(8)
        assert [h["gl"] for h in pop.history] == [h["gl"] for h in o.history]
        assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32)), (P, G, d)
        assert np.array_equal(pop.v.cpu().numpy().view(np.uint32), o.v.view(np.uint32)), (P, G, d)
        pop.close()


@pytest.mark.parametrize("P,G,d", [(1, 1, 3), (20, 4, 2311), (64, 8, 148 * 768 + 8), (150, 75, 260)])
def test_momentum_shapes_on_both_kernels(P, G, d):
    # one worker and d below a 16-byte column; a ragged last chunk of workers; more tiles than CTAs with a ragged
    # last tile; and so many groups that the leader block does not fit (register-staged fallback kernel)
    w = inputs.make_external(P, G, d, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=5, loss_ring=3, config_id=96)
    from paper_1905_10395_b200.runner import Population
    pop = Population(w, momentum=0.9, weight_decay=1e-4)
    pop.run(5, record=True)
    o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau, momentum=0.9, weight_decay=1e-4)
    o.run(5)
    for hg, ho in zip(pop.history, o.history):
        assert hg["gl"] == ho["gl"] and np.array_equal(hg["ll"], ho["ll"])
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    assert np.array_equal(pop.v.cpu().numpy().view(np.uint32), o.v.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_zero_momentum_and_decay_equals_the_plain_path():
    w = inputs.make_external(5, 2, 9000, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=6, loss_ring=3,
                             config_id=54)
    a = _pop(w)
    b = _pop(w, momentum=0.0, weight_decay=0.0)
    a.run(6)
    b.run(6)
    assert np.array_equal(a.x_host(), b.x_host())
    # the buffer then simply holds the last gradient
    assert np.array_equal(b.v.cpu().numpy()[:, :w.d], w.arrays["g"][:, :w.d])
    a.close()
    b.close()


def test_unsupported_combinations_are_refused():
    import torch
    from paper_1905_10395_b200 import api
    x = torch.zeros(2, 32, device="cuda")
    g = torch.zeros(2, 32, device="cuda")
    v = torch.zeros(2, 32, device="cuda")
    base = dict(P=2, G=1, group_of=np.zeros(2, np.int32), d=32, ld=32, eta=0.1, lambda_l=0.1, lambda_g=0.1, tau=1,
                objective=api.OBJ_EXTERNAL, x=x, g=g, v=v, momentum=0.9)
    for bad in (dict(flags=api.FLAG_MLP_FUSED_STEP), dict(flags=api.FLAG_ALGORITHM1, leader_copies=torch.zeros(2, 32, device="cuda")),
                dict(momentum=float("nan")), dict(weight_decay=float("inf"))):
        kw = dict(base)
        kw.update(bad)
        cfg, keep = api.make_config(**kw)
        with pytest.raises(api.LsgdError):
            api.Lsgd(cfg, keep)
    # a quadratic without a gradient buffer cannot carry a momentum buffer
    a = torch.ones(32, device="cuda")
    desc = api.QuadraticDesc(a.data_ptr(), a.data_ptr(), 0.0)
    kw = dict(base)
    kw.update(objective=api.OBJ_QUADRATIC, desc=desc, g=None)
    cfg, keep = api.make_config(**kw)
    with pytest.raises(api.LsgdError):
        api.Lsgd(cfg, keep)


def test_mlp_population_with_momentum():
    w = inputs.make_mlp(4, 2, dims=(40, 72, 136, 7), pool=256, heldout=40, batch=24, n_classes=7, steps=6, tau=2,
                        config_id=81)
    mu, wd = 0.9, 1e-4
    A = w.arrays
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    o = orc.LsgdOracle(w.x0, orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="bf16emu"),
                       w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau, momentum=mu, weight_decay=wd)
    import torch
    pop = _pop(w, momentum=mu, weight_decay=wd)
    for t in range(6):
        o.step()
        fl = torch.from_numpy(o.history[t // w.tau]["loss"]).cuda() if t % w.tau == 0 else None
        pop.step(forced_loss=fl)
    x, ref = pop.x_host().astype(np.float64), o.x.astype(np.float64)
    dx, dref = x - w.x0, ref - w.x0
    for i in range(w.P):
        assert np.linalg.norm(dx[i] - dref[i]) <= 2e-2 * np.linalg.norm(dref[i]), i
    v, vref = pop.v.cpu().numpy().astype(np.float64), o.v.astype(np.float64)
    for i in range(w.P):
        assert np.linalg.norm(v[i] - vref[i]) <= 2e-2 * np.linalg.norm(vref[i]), i
    assert pop.lsgd.check_device() == 0
    pop.close()
