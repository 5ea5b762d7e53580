"""GPU parity of the EAGD comparison line (LSGD_FLAG_EAGD) against oracle.EagdOracle: supplement, "Low-Rank
Matrix Completion Experiments".  Workers and center are expected bit-identical in the default arithmetic for the
element-wise objectives and within 1e-5 for the dense completion objective (its gradient is a long sum)."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu


def _rel(x, ref):
    return float((np.abs(x.astype(np.float64) - ref) / np.maximum(np.abs(ref), 1e-3)).max())


@pytest.mark.parametrize("tau,P,d", [(1, 8, 5000 + 12), (3, 5, 70000)])
def test_external_gradients_bit_exact(tau, P, d):
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_external(P, 1, d, eta=0.05, lambda_l=0.3, lambda_g=0.0, tau=tau, steps=7, config_id=150)
    pop = Population(w, eagd=True)
    pop.run(7)
    o = orc.EagdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.eta, w.lambda_l, tau=tau)
    o.run(7)
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    assert np.array_equal(pop.center_host().view(np.uint32), o.center.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


@pytest.mark.parametrize("fused", [False, True])
def test_quadratic_with_noise_and_groups_that_play_no_role(fused):
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_quadratic(12, 3, (1 << 14) + 20, eta=0.05, lambda_l=0.2, lambda_g=0.0, tau=2, steps=8, config_id=151)
    pop = Population(w, eagd=True, fused_quadratic=fused)
    pop.run(8)
    o = orc.EagdOracle(w.x0, orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"]), w.eta,
                       w.lambda_l, tau=2)
    o.run(8)
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    assert np.array_equal(pop.center_host().view(np.uint32), o.center.view(np.uint32))
    pop.close()


@pytest.mark.parametrize("n,r", [(100, 1), (203, 10)])
def test_dense_completion_the_papers_settings(n, r):
    """The experiment of the paper's Figure 1 for the EAGD side: 8 workers, eta 5e-4, lambda 1/5, tau 1."""
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_psd(P=8, n=n, r=r, steps=6)
    pop = Population(w, eagd=True)
    pop.run(6)
    o = orc.EagdOracle(w.x0, orc.PsdCompletion(n, r, w.arrays["M"]), w.eta, w.lambda_l, tau=1)
    o.run(6)
    assert _rel(pop.x_host(), o.x) <= 1e-5
    assert _rel(pop.center_host(), o.center) <= 1e-5
    pop.close()


def test_argument_rules():
    import torch
    from paper_1905_10395_b200 import api
    w = inputs.make_external(4, 2, 256, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=1, steps=1, config_id=152)
    x = torch.zeros(4, 256, device="cuda")
    copies = torch.zeros(3, 256, device="cuda")
    kw = dict(P=4, G=2, group_of=w.group_of, d=256, ld=256, eta=0.1, lambda_l=0.1, tau=1, objective=api.OBJ_EXTERNAL, x=x,
              g=x, flags=api.FLAG_EAGD)
    for over, status in [(dict(lambda_g=0.1, leader_copies=copies), api.ERR_INVALID_ARG),      # one strength only
                         (dict(lambda_g=0.0), api.ERR_INVALID_ARG),                            # no center buffer
                         (dict(lambda_g=0.0, leader_copies=copies, flags=api.FLAG_EAGD | api.FLAG_ALGORITHM1, tau_g=2),
                          api.ERR_UNSUPPORTED)]:
        cfg, keep = api.make_config(**{**kw, **over})
        with pytest.raises(api.LsgdError) as e:
            api.lsgd_create(cfg)
        assert e.value.status == status
