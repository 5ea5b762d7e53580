"""Degenerate and extreme shapes of the update / election path, against the oracle (bit-exact)."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu


def _check(w, steps, **kw):
    from paper_1905_10395_b200.runner import Population
    pop = Population(w, **kw)
    pop.run(steps, record=True)
    o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau)
    o.run(steps)
    for hg, ho in zip(pop.history, o.history):
        assert hg["gl"] == ho["gl"] and np.array_equal(hg["ll"], ho["ll"])
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


@pytest.mark.parametrize("P,G,d", [(1, 1, 1), (1, 1, 1000), (2, 2, 3), (5, 5, 37), (3, 1, 2), (26, 2, 5000), (27, 3, 5000)])
def test_tiny_and_boundary_populations(P, G, d):
    # one worker (its own leader: pure SGD), every worker its own group, d below one 16-byte column,
    # and the population sizes on both sides of the staged / register-staged kernel switch
    w = inputs.make_external(P, G, d, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=5, loss_ring=3, config_id=110)
    _check(w, 5)


@pytest.mark.parametrize("P,G,d", [(33, 1, 777), (64, 8, 3001), (40, 40, 1100), (100, 7, 2500), (60, 30, 600),
                                   (28, 2, 148 * 768 * 2 + 4)])
def test_populations_streamed_in_chunks(P, G, d):
    # populations too large to stage whole: the rows of a column tile pass through shared memory in chunks
    # (ragged last chunk, ragged last tile, leader blocks of 2 .. 41 slots, several tiles per CTA)
    w = inputs.make_external(P, G, d, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=5, loss_ring=3, config_id=115)
    _check(w, 5)


@pytest.mark.parametrize("P,G,d", [(1, 1, 1), (3, 3, 5), (9, 2, 769), (70, 7, 1537)])
def test_fused_quadratic_degenerate_shapes(P, G, d):
    # the inline-gradient forms of the chunked kernel: one worker, every worker its own group, d below one
    # 16-byte column, one column past a tile, a ragged last chunk of workers
    w = inputs.make_quadratic(P, G, d, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=5, noise_ring=3, config_id=116)
    from paper_1905_10395_b200.runner import Population
    pop = Population(w, fused_quadratic=True)
    pop.run(5, record=True)
    o = orc.LsgdOracle(w.x0, orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"]), w.group_of,
                       w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)
    o.run(5)
    for hg, ho in zip(pop.history, o.history):
        assert hg["gl"] == ho["gl"] and np.array_equal(hg["ll"], ho["ll"])
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_single_worker_is_plain_sgd():
    w = inputs.make_external(1, 1, 257, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=1, steps=4, config_id=111)
    from paper_1905_10395_b200.runner import Population
    pop = Population(w)
    pop.run(4)
    x = w.x0[0].astype(np.float64)
    for _ in range(4):
        x = (x - float(np.float32(w.eta)) * w.arrays["g"][0].astype(np.float64)).astype(np.float32).astype(np.float64)
    assert np.array_equal(pop.x_host()[0], x.astype(np.float32))
    pop.close()


def test_largest_supported_population():
    # P = 4096 workers (the documented maximum) in 61 unequal groups
    rng = np.random.default_rng(0)
    P, G = 4096, 61
    m = np.concatenate([np.arange(G), rng.integers(0, G, P - G)]).astype(np.int32)
    rng.shuffle(m)
    w = inputs.make_external(P, G, 96, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=1, steps=3, loss_ring=3, config_id=112,
                             group_of=m)
    _check(w, 3)


def test_too_many_workers_is_refused():
    import torch
    from paper_1905_10395_b200 import api
    P = 4097
    x = torch.zeros(P, 32, device="cuda")
    cfg, keep = api.make_config(P=P, G=1, group_of=np.zeros(P, np.int32), d=32, ld=32, eta=0.1, lambda_l=0.1,
                                lambda_g=0.1, tau=1, objective=api.OBJ_EXTERNAL, x=x, g=x)
    with pytest.raises(api.LsgdError) as e:
        api.lsgd_create(cfg)
    assert e.value.status == api.ERR_UNSUPPORTED


def test_long_period_and_stale_leaders():
    # tau larger than the run: a single election at t = 0, plain steps afterwards
    w = inputs.make_external(6, 2, 4100, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=1000, steps=7, config_id=113)
    _check(w, 7)


def test_all_losses_equal_or_nan():
    w = inputs.make_external(8, 2, 640, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=1, steps=3, loss_ring=3, config_id=114)
    w.arrays["loss_ring"][0, :] = 0.25
    w.arrays["loss_ring"][1, :] = np.nan
    w.arrays["loss_ring"][2, :] = np.inf
    _check(w, 3)
