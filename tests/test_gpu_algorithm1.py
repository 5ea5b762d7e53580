"""GPU parity for the schedule of the paper's Algorithm 1 (LSGD_FLAG_ALGORITHM1): small pulls towards the
stale leader copies on every step, larger pulls and re-elections at the local / global communication
periods.  Compared with oracle.Algorithm1Oracle; in the default arithmetic the parameters are expected
bit-identical."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu

F32 = np.float32
ALG = dict(gamma_l=0.2, gamma_g=0.1, tau_g=6)


def _oracle(w, alg=ALG):
    A = w.arrays
    if w.objective == "external":
        obj = orc.External(A["g"], A["loss_ring"])
    elif w.objective == "quadratic":
        obj = orc.Quadratic(A["a"], A["b"], w.meta["sigma"], A.get("noise"))
    else:
        m = w.meta
        obj = orc.MatComp(m["n_rows"], m["n_cols"], m["rank"], A["obs_r"], A["obs_c"], A["obs_v"], A["batch_pos"],
                          A["heldout_pos"])
    return orc.Algorithm1Oracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, alg["gamma_l"], alg["gamma_g"],
                                w.tau, alg["tau_g"])


def _run(w, steps, alg=ALG, **kw):
    from paper_1905_10395_b200.runner import Population
    pop = Population(w, algorithm1=alg, **kw)
    pop.run(steps, record=True)
    o = _oracle(w, alg)
    o.run(steps)
    assert len(pop.history) == len(o.history)
    for hg, ho in zip(pop.history, o.history):
        assert hg["t"] == ho["t"]
        assert np.array_equal(hg["ll"], ho["ll"]) and hg["gl"] == ho["gl"], (hg, ho)
    return pop, o


def test_external_ragged_unequal_groups_bit_exact():
    group_of = np.asarray([2, 0, 1, 1, 0, 2, 2], dtype=np.int32)
    w = inputs.make_external(7, 3, 4999, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=13, loss_ring=7, config_id=95,
                             group_of=group_of)
    pop, o = _run(w, 13)
    x = pop.x_host()
    assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
    import torch
    torch.cuda.synchronize()
    copies = pop.leader_copies.cpu().numpy()
    for j in range(w.G):
        assert np.array_equal(copies[j], o.z_l[j])
    assert np.array_equal(copies[w.G], o.z_g)
    assert pop.lsgd.check_device() == 0
    pop.close()


@pytest.mark.parametrize("fused", [False, True])
def test_quadratic_multi_leader_bit_exact(fused):
    w = inputs.config(1, d=(1 << 15) + 24, tau=2, steps=12)
    pop, o = _run(w, 12, fused_quadratic=fused)
    assert any(h.get("local") and h.get("global") for h in o.history)
    for hg, ho in zip(pop.history, o.history):
        # after a communication with both periods due the library holds the second loss vector (taken after
        # the local pull), which is the one the global election used
        assert np.allclose(hg["loss"], ho.get("loss_global", ho["loss"]), rtol=3e-7, atol=0)
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    pop.close()


def test_global_leader_is_elected_after_the_local_pull():
    """The hand-worked two-group case of tests/test_oracle_algorithm1.py (Algorithm 1, Section 2.2): the local
    pull moves worker 1 onto the minimiser, so the global election that follows it must pick worker 1, not the
    worker that was best before the pull."""
    d, ld = 1, 32
    a, b = np.zeros(ld, F32), np.zeros(ld, F32)
    a[0] = 1.0
    x0 = np.zeros((4, ld), F32)
    x0[:, 0] = [2.0, -6.0, 1.8, 2.2]
    w = inputs.Workload(name="alg1-order", objective="quadratic", P=4, G=2, d=d, ld=ld,
                        group_of=np.asarray([0, 0, 1, 1], np.int32), eta=0.5, lambda_l=1.5, lambda_g=0.5, tau=1, steps=1,
                        x0=x0, arrays={"a": a, "b": b, "noise": None}, meta={"sigma": 0.0})
    alg = dict(gamma_l=0.0, gamma_g=0.0, tau_g=1)
    for fused in (False, True):
        pop, o = _run(w, 1, alg=alg, fused_quadratic=fused)
        assert pop.history[-1]["gl"] == 1 and list(pop.history[-1]["ll"]) == [0, 2]
        x = pop.x_host()
        assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
        assert np.allclose(x[:, 0], [0.75, 0.0, 0.675, 0.7125], rtol=1e-6, atol=0)
        assert np.allclose(pop.history[-1]["loss"], [0.5, 0.0, 0.405, 0.45125], rtol=1e-6)
        pop.close()


def test_zero_searching_scope_and_larger_shape():
    # gamma = 0: plain steps between communications; several CTAs per row
    w = inputs.make_external(16, 4, (1 << 20) + 8, eta=0.01, lambda_l=0.1, lambda_g=0.05, tau=3, steps=9, config_id=96)
    alg = dict(gamma_l=0.0, gamma_g=0.0, tau_g=6)
    pop, o = _run(w, 9, alg=alg)
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    pop.close()


def test_matcomp_small():
    w = inputs.make_matcomp(5, 2, n_rows=300, n_cols=200, rank=7, n_obs=5000, n_heldout=1000, batch=700, steps=9, tau=3,
                            config_id=97)
    pop, o = _run(w, 9)
    err = np.abs(pop.x_host().astype(np.float64) - o.x) / np.maximum(np.abs(o.x), 1e-3)
    assert err.max() <= 1e-5
    pop.close()


def test_protocol_errors():
    import torch
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_external(4, 2, 256, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=4, config_id=98)
    pop = Population(w, algorithm1=ALG)
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.step()                                  # no initial election yet
    assert e.value.status == api.ERR_STATE
    pop.step()                                           # initial election + first step: t = 1
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.elect(pop.loss_ring[0])                 # t = 1 is not a communication step
    assert e.value.status == api.ERR_STATE
    pop.close()
    x = torch.zeros(4, 256, device="cuda")
    cfg, keep = api.make_config(P=4, G=2, group_of=w.group_of, d=256, ld=256, eta=0.1, lambda_l=0.1, lambda_g=0.1, tau=2,
                                objective=api.OBJ_EXTERNAL, x=x, g=x, flags=api.FLAG_ALGORITHM1, tau_g=4)
    with pytest.raises(api.LsgdError) as e:
        api.lsgd_create(cfg)                             # leader_copies missing
    assert e.value.status == api.ERR_INVALID_ARG
