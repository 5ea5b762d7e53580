"""The device status word (lsgd_check_device / LSGD_ERR_DEVICE_FLAG), exercised without faulting anything:
a bounded wait that is made to run out on a barrier nothing completes, batch positions outside the observed
list (range-checked before any dereference, so the entries are skipped), and gradient contributions outside
the fixed-point accumulator's range.  After each report the handle must still work."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu


def _matcomp(**kw):
    args = dict(n_rows=120, n_cols=90, rank=6, n_obs=3000, n_heldout=400, batch=500, steps=3, tau=1, config_id=120)
    args.update(kw)
    return inputs.make_matcomp(4, 2, **args)


def _matcomp_oracle(w, batch_pos=None):
    m, A = w.meta, w.arrays
    return orc.MatComp(m["n_rows"], m["n_cols"], m["rank"], A["obs_r"], A["obs_c"], A["obs_v"],
                       A["batch_pos"] if batch_pos is None else batch_pos, A["heldout_pos"])


def test_bounded_wait_runs_out_and_is_reported_and_the_handle_still_works():
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_external(6, 2, 5000, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=4, config_id=121)
    pop = Population(w)
    pop.run(2)
    assert pop.lsgd.check_device() == 0
    for which in (0, 1):                                           # the update kernels' wait, the product kernels' wait
        assert pop.lsgd.selftest_wait_timeout(100_000, which) == 1     # the wait gave up after ~50 us
        assert pop.lsgd.check_device() == api.DEVFLAG_WAIT_TIMEOUT     # LSGD_ERR_DEVICE_FLAG with this bit
        assert pop.lsgd.check_device() == 0                            # reading clears it
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.selftest_wait_timeout(10 ** 9)                    # budgets are capped
    assert e.value.status == api.ERR_INVALID_ARG
    pop.run(2)                                                     # the context and the handle are intact
    o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau)
    o.run(4)
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_out_of_range_batch_positions_are_skipped_and_reported():
    import torch
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = _matcomp()
    B, n_obs = w.meta["batch"], len(w.arrays["obs_r"])
    pos = w.arrays["batch_pos"][0].copy()                          # [P, B]
    pos[1, 7] = -1
    pos[2, B - 1] = n_obs
    pop = Population(w)
    pop.lsgd.grad(torch.from_numpy(pos).cuda())
    flags = pop.lsgd.check_device()
    assert flags == api.DEVFLAG_BAD_INDEX
    g = pop.g.cpu().numpy()
    # the rest of the gradient: the oracle on the remaining entries (it divides by their number, the kernel by B)
    for i in range(w.P):
        keep = pos[i][(pos[i] >= 0) & (pos[i] < n_obs)]
        ref = _matcomp_oracle(w, batch_pos=[[keep] * w.P]).grad(w.x0, 0)[i].astype(np.float64) * (len(keep) / B)
        err = np.abs(g[i] - ref) / np.maximum(np.abs(ref), 1e-3)
        assert err.max() <= 1e-5, (i, err.max())
    # a clean batch afterwards: no flag, and the step equals the oracle's
    pop.lsgd.grad(pop.batches[0])
    pop.lsgd.elect(None)
    pop.lsgd.step()
    assert pop.lsgd.check_device() == 0
    o = orc.LsgdOracle(w.x0, _matcomp_oracle(w), w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)
    o.step()
    err = np.abs(pop.x_host().astype(np.float64) - o.x) / np.maximum(np.abs(o.x), 1e-3)
    assert err.max() <= 1e-5
    pop.close()


@pytest.mark.parametrize("poison", ["huge", "nan"])
def test_contributions_outside_the_accumulator_range_are_reported_not_saturated(poison):
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = _matcomp(config_id=122)
    x0 = w.x0.copy()
    x0[3, : w.d] = 1e12 if poison == "huge" else np.nan            # a diverged worker; the others are healthy
    w.x0 = x0
    pop = Population(w)
    pop.lsgd.grad(pop.batches[0])
    assert pop.lsgd.check_device() == api.DEVFLAG_OVERFLOW
    g = pop.g.cpu().numpy()
    ref = _matcomp_oracle(w).grad(w.x0, 0)
    for i in range(3):                                             # the healthy workers' gradients are unaffected
        err = np.abs(g[i].astype(np.float64) - ref[i]) / np.maximum(np.abs(ref[i]), 1e-3)
        assert err.max() <= 1e-5
    assert np.all(g[3] == 0)                                       # nothing of the poisoned worker was added
    pop.lsgd.grad(pop.batches[1])                                  # the accumulator is clean for the next call
    assert pop.lsgd.check_device() == api.DEVFLAG_OVERFLOW         # (the poisoned worker reports again)
    pop.close()
