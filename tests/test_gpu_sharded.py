"""Group-per-device mapping on the GPU: several ranks emulated in lock-step on one device (no rank's kernels
wait on another's), each with its own handle, guest row and lsgd_set_leaders -- against the single-population
oracle, bit for bit.  Also lsgd_set_leaders by itself on every form of the pull kernel."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs, sharded

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world,P,G,d", [(2, 12, 4, 1000), (4, 64, 8, 3001), (3, 90, 6, 520)])
def test_external_objective_sharded_equals_single_population(world, P, G, d):
    steps = 9
    w = inputs.make_external(P, G, d, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=steps, loss_ring=5, config_id=150)
    w.arrays["loss_ring"][3, :] = 0.25                  # all tied: the lowest global index wins
    engines = [sharded.CudaShardEngine(w, r, world) for r in range(world)]
    sharded.run_lockstep(engines, steps)
    o = orc.LsgdOracle(w.x0, orc.External(w.arrays["g"], w.arrays["loss_ring"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau)
    o.run(steps)
    owners = set()
    for e in engines:
        assert np.array_equal(e.x_local().view(np.uint32), o.x[e.shard.workers].view(np.uint32))
        assert e.global_leader_global == o.gl
        assert e.lsgd.check_device() == 0
    assert np.array_equal(np.concatenate([e.local_leaders_global for e in engines]), o.ll)
    for h in o.history:
        owners.add(int(w.group_of[h["gl"]]) * world // G)
    assert len(owners) > 1 or world == 1                # the global leader did move between ranks
    for e in engines:
        e.close()


def test_quadratic_objective_sharded_equals_single_population():
    # gradient evaluated inside the step, election on the exact f(x_i) computed on each rank for its own workers
    w = inputs.make_quadratic(16, 4, 5000, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=8, config_id=151)
    engines = [sharded.CudaShardEngine(w, r, 2) for r in range(2)]
    sharded.run_lockstep(engines, 8)
    o = orc.LsgdOracle(w.x0, orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"]), w.group_of,
                       w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)
    o.run(8)
    for e in engines:
        assert np.array_equal(e.x_local().view(np.uint32), o.x[e.shard.workers].view(np.uint32))
        assert e.global_leader_global == o.gl
        e.close()


@pytest.mark.parametrize("P,G,d", [(12, 3, 2000), (40, 5, 2000), (200, 100, 300)])
def test_set_leaders_overrides_the_election(P, G, d):
    """Leaders given by the caller, the global one NOT among the local ones, through the staged, the chunked and
    the register-staged form of the pull kernel; and the argument checks."""
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_external(P, G, d, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=1, steps=2, loss_ring=2, config_id=152)
    pop = Population(w)
    with pytest.raises(api.LsgdError) as e:              # nothing elected yet: "keep" has nothing to keep
        pop.lsgd.set_leaders(None, 0)
    assert e.value.status == api.ERR_STATE
    members = [np.nonzero(w.group_of == j)[0] for j in range(G)]
    ll = np.array([m[-1] for m in members], dtype=np.int32)       # last member of every group
    gl = int(members[0][0])                                         # first member of group 0: not a local leader
    bad = ll.copy()
    bad[0] = members[1][0]
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.set_leaders(bad, gl)
    assert e.value.status == api.ERR_BAD_GROUPS
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.set_leaders(ll, P)
    assert e.value.status == api.ERR_BAD_GROUPS
    x = w.x0.copy()
    for _ in range(2):
        pop.lsgd.grad(None)
        pop.lsgd.set_leaders(ll, gl)
        pop.lsgd.step()
        orc.update(x, w.arrays["g"], w.group_of, ll, gl, w.eta, w.lambda_l, w.lambda_g, True)
    got_ll, got_gl = pop.lsgd.leaders()
    assert np.array_equal(got_ll, ll) and got_gl == gl
    assert np.array_equal(pop.x_host().view(np.uint32), x.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()
