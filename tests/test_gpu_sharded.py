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


def test_device_keys_equal_the_independently_packed_keys_and_pick_the_global_leader():
    """lsgd_shard_best_key / lsgd_shard_pick_global against the CPU packing of the same published key format, on
    losses with ties, signed zeros, infinities and NaN."""
    import itertools
    import torch
    from paper_1905_10395_b200 import api
    from tests._shard_cpu_engine import argmin_by_rule, pack_key
    P = 5                                                   # 4 own workers + a guest row
    x = torch.zeros(P, 32, device="cuda")
    cfg, keep = api.make_config(P=P, G=3, group_of=np.asarray([0, 0, 1, 1, 2], np.int32), d=32, ld=32, eta=0.1, lambda_l=0.1,
                                lambda_g=0.1, tau=1, objective=api.OBJ_EXTERNAL, x=x, g=x)
    h = api.Lsgd(cfg, keep)
    gidx = np.asarray([7, 9, 12, 40], dtype=np.int32)
    gidx_d = torch.from_numpy(gidx).cuda()
    key = torch.zeros(1, dtype=torch.int64, device="cuda")
    vals = [-np.inf, -1.0, -0.0, 0.0, 1.0, np.inf, np.nan]
    with pytest.raises(api.LsgdError) as e:
        h.shard_best_key(4, gidx_d, key)                    # before any election
    assert e.value.status == api.ERR_STATE
    for n, combo in enumerate(itertools.product(vals, repeat=4)):
        if n % 7:                                           # every 7th combination: 343 device round trips
            continue
        loss = np.asarray(list(combo) + [np.nan], dtype=np.float32)
        h.elect(torch.from_numpy(loss).cuda())
        h.shard_best_key(4, gidx_d, key)
        mine = int(key.cpu().numpy().view(np.uint64)[0])
        p = argmin_by_rule(loss[:4], gidx)
        assert mine == pack_key(loss[p], gidx[p]), combo
        other = pack_key(0.0, 8)                            # another device's key: zero loss at global worker 8
        keys = torch.from_numpy(np.asarray([other, mine], dtype=np.uint64).view(np.int64)).cuda()
        winner, g_index, best_local = h.shard_pick_global(keys, 2, 1, 4)
        assert best_local == p
        want = 0 if other < mine else 1
        assert winner == want and g_index == (8 if want == 0 else gidx[p]), combo
        assert h.leaders()[1] == (4 if want == 0 else p)    # guest row, or this device's own winner
    h.destroy()
