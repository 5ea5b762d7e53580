"""GPU parity of the MLP population objective (bf16 tensor-core products, fp32 accumulation) against
the oracle's bf16-emulation mode.  Tolerance from the workload statement: 2e-2 relative on parameters
and on losses.  Leaders must agree unless the oracle's own margin is a near-tie (< 2e-2 relative), in
which case the run is repeated with the oracle's loss vectors forced into the election."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = 2e-2
LOSS_FLOOR = 1.0     # cross-entropy has a natural O(1) scale (chance level ln 10 = 2.3)
PARAM_FLOOR = 1e-3   # floor of the elementwise relative parameter error
FREE_RUN_OUTLIERS = 2e-2   # free-running trajectories: fraction of entries allowed beyond the elementwise bound


def loss_close(got, ref):
    return bool(np.all(np.abs(got.astype(np.float64) - ref) <= TOL * np.maximum(np.abs(ref), LOSS_FLOOR)))


def _oracle(w):
    A = w.arrays
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    obj = orc.Mlp(segs, A["pool_x"], A["pool_y"], A["batch_idx"], A["held_x"], A["held_y"], mode="bf16emu",
                  loss_window=int(w.meta.get("loss_window", 0)))
    return orc.LsgdOracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)


def _run_pair(w, steps, flags=0):
    import torch
    from paper_1905_10395_b200.runner import Population
    o = _oracle(w)
    train_ref = []
    for _ in range(steps):
        o.step()
        train_ref.append(o.obj.last_train_loss.copy())
    pop = Population(w, flags=flags)
    train_gpu = []
    for _ in range(steps):
        pop.step(record=True)
        train_gpu.append(pop.lsgd.train_loss())
    same = all(hg["gl"] == ho["gl"] and np.array_equal(hg["ll"], ho["ll"]) for hg, ho in zip(pop.history, o.history))
    forced = False
    if not same:
        for hg, ho in zip(pop.history, o.history):
            if hg["gl"] != ho["gl"] or not np.array_equal(hg["ll"], ho["ll"]):
                srt = np.sort(ho["loss"])
                assert (srt[1] - srt[0]) <= TOL * abs(srt[0]), "leaders differ without a near-tie"
                break
        pop.close()
        pop = Population(w, flags=flags)
        train_gpu = []
        for t in range(steps):
            fl = torch.from_numpy(o.history[t // w.tau]["loss"]).cuda() if t % w.tau == 0 else None
            pop.step(forced_loss=fl, record=True)
            train_gpu.append(pop.lsgd.train_loss())
        forced = True
    return pop, o, train_gpu, train_ref, forced


def elementwise_errors(x, ref, x_before):
    """The elementwise figures of the parity statement for this objective:
    parameters   |x - ref| / max(|ref|, 1e-3) for every entry of every worker (the metric of the fp32
                 configurations, here with the 2e-2 bound of the bf16 products): its maximum, and the fraction of
                 entries beyond 2e-2;
    change       max |dx - dref| / max(|dref|, largest |dref| of the same worker), dx = x - x_before."""
    e = np.abs(x - ref) / np.maximum(np.abs(ref), PARAM_FLOOR)
    dx, dref = x - x_before, ref - x_before
    floor = np.abs(dref).max(axis=1, keepdims=True)
    e_delta = float((np.abs(dx - dref) / np.maximum(np.abs(dref), floor)).max())
    return float(e.max()), float((e > TOL).mean()), e_delta


def _check(pop, o, w, train_gpu, train_ref, forced):
    """A FREE-RUNNING trajectory.  On this workload it amplifies differences of accumulation order by about 3x
    per step while the losses overshoot (eta = 0.05 on inputs of norm ~60): two CPU evaluations of the oracle's
    own definition, one accumulating in float64 and one in float32, already differ by more than 2e-2 on some
    entries after two steps (tests/test_oracle_mlp_sensitivity.py).  So here the elementwise error is bounded in
    the bulk (at most FREE_RUN_OUTLIERS of the entries beyond 2e-2) and norm-wise; the elementwise 2e-2 bound
    on EVERY entry is asserted step by step from the oracle's state in
    test_config3_every_step_from_the_oracle_state."""
    x = pop.x_host().astype(np.float64)
    ref = o.x.astype(np.float64)
    e_param, frac, e_delta = elementwise_errors(x, ref, w.x0.astype(np.float64))
    print(f"free-running: elementwise parameter error max {e_param:.3e}, beyond 2e-2: {frac:.3e} of the entries, "
          f"change error {e_delta:.3e}")
    assert frac <= FREE_RUN_OUTLIERS, (e_param, frac)
    scale = np.abs(ref).max()
    assert np.abs(x - ref).max() <= TOL * scale
    # the discriminating number: error of the parameter change, norm-wise per worker
    dx, dref = x - w.x0, ref - w.x0
    for i in range(w.P):
        assert np.linalg.norm(dx[i] - dref[i]) <= TOL * np.linalg.norm(dref[i]), i
    # elementwise: all but a few entries (a ReLU whose pre-activation is within accumulation error of
    # zero switches a whole sample's contribution on or off) within TOL of the largest change
    assert np.mean(np.abs(dx - dref) > TOL * np.abs(dref).max()) <= 1e-4
    for tg, tr in zip(train_gpu, train_ref):
        assert loss_close(tg, tr)
    if not forced:
        for hg, ho in zip(pop.history, o.history):
            assert loss_close(hg["loss"], ho["loss"])
    assert np.all(x[:, :][:, _pad_mask(w)] == 0)
    assert pop.lsgd.check_device() == 0


def _pad_mask(w):
    segs, d = inputs.mlp_layout(w.meta["dims"])
    m = np.ones(d, dtype=bool)
    for s in segs:
        m[s["w"]:s["w"] + s["n_in"] * s["n_out"]] = False
        m[s["b"]:s["b"] + s["n_out"]] = False
    return m


def test_mlp_small_ragged_population():
    w = inputs.make_mlp(3, 2, dims=(40, 72, 136, 7), pool=256, heldout=40, batch=24, n_classes=7, steps=6, tau=2,
                        config_id=80, group_of=np.asarray([0, 1, 1], dtype=np.int32))
    rng = np.random.default_rng(2)
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    for s in segs:                                           # non-zero biases
        w.x0[:, s["b"]:s["b"] + s["n_out"]] = (0.1 * rng.standard_normal((w.P, s["n_out"]))).astype(np.float32)
    pop, o, tg, tr, forced = _run_pair(w, 6)
    _check(pop, o, w, tg, tr, forced)
    pop.close()


def test_mlp_one_step_gradient_matches_oracle():
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_mlp(2, 1, pool=512, heldout=128, batch=128, steps=1, tau=1, config_id=81)
    o = _oracle(w)
    g_ref = o.obj.grad(w.x0, 0).astype(np.float64)
    pop = Population(w)
    pop.lsgd.grad(pop.batches[0])
    import torch
    torch.cuda.synchronize()
    g = pop.g.cpu().numpy().astype(np.float64)
    segs, _ = inputs.mlp_layout(w.meta["dims"])
    for s in segs:
        for lo, n in ((s["w"], s["n_in"] * s["n_out"]), (s["b"], s["n_out"])):
            a, b = g[:, lo:lo + n], g_ref[:, lo:lo + n]
            assert np.linalg.norm(a - b) <= TOL * np.linalg.norm(b), (lo, n)
            assert np.mean(np.abs(a - b) > TOL * np.abs(b).max()) <= 1e-4, (lo, n)
    assert np.all(g[:, _pad_mask(w)] == 0)
    pop.close()


@pytest.mark.parametrize("fused", [False, True])
def test_config3_mlp_population_ten_steps(fused):
    # fused = the configuration the benchmark times (LSGD_FLAG_MLP_FUSED_STEP)
    from paper_1905_10395_b200 import api
    w = inputs.config(3, steps=10)
    pop, o, tg, tr, forced = _run_pair(w, 10, flags=api.FLAG_MLP_FUSED_STEP if fused else 0)
    _check(pop, o, w, tg, tr, forced)
    pop.close()


ACC_EPS = 2.0 ** -18      # bound on the error of a float32 sum of ~1000 products, relative to sum |h||W| + |b|
RND_EPS = 2.0 ** -8       # one bf16 unit in the last place, relative (round-to-nearest is within half of it)


class OneWorkerMlp(orc.Mlp):
    """The oracle's MLP objective for ONE worker (x is a single row).  With ``given`` = (h1, h2) the backward pass
    runs on those stored hidden activations instead of the oracle's own -- everything else (the products, the
    roundings of the deltas, the mask h > 0, the sums) is the base class's arithmetic -- and ``check_given``
    verifies first that each given activation is a valid bf16 rounding of relu(z) for the oracle's own float64
    pre-activation z of that layer."""

    def __init__(self, base: orc.Mlp, worker: int, t: int, given=None):
        idx = base.batch_idx[t % len(base.batch_idx)][worker]
        super().__init__(base.segs, base.data_x, base.data_y, [[idx]], base.held_x, base.held_y)
        self.given = given

    def _forward(self, xi, inp):
        if self.given is None:
            return super()._forward(xi, inp)
        Ws, bs = self._weights(xi)
        hs = [self.rd(inp).astype(np.float64)] + [np.asarray(h, dtype=np.float64) for h in self.given]
        return Ws, hs, hs[-1] @ Ws[-1].T + bs[-1]

    def check_given(self, xi):
        """Layer by layer, from the GIVEN input of that layer: |h - relu(z)| <= one bf16 ulp of |z| plus the
        accumulation bound (which also covers a ReLU decision taken within rounding of zero)."""
        Ws, bs = self._weights(xi)
        inp = self.rd(self.data_x[self.batch_idx[0][0]]).astype(np.float64)
        worst = 0.0
        for l, h in enumerate(self.given):
            z = inp @ Ws[l].T + bs[l]
            slack = RND_EPS * np.abs(z) + ACC_EPS * (np.abs(inp) @ np.abs(Ws[l]).T + np.abs(bs[l]))
            worst = max(worst, float((np.abs(h - np.maximum(z, 0.0)) / np.maximum(slack, 1e-300)).max()))
            inp = np.asarray(h, dtype=np.float64)
        return worst


def _row_after_step(x_t, i, g_i, o, w, pull):
    """Worker i's parameters after the step of Eq. (1) from state x_t with gradient g_i and the oracle's leaders."""
    if not pull:
        sub = x_t[i:i + 1].copy()
        orc.update(sub, g_i[None, :], [0], (), -1, w.eta, w.lambda_l, w.lambda_g, False)
        return sub[0]
    ll_i = int(o.ll[int(w.group_of[i])])
    sub = np.stack([x_t[i], x_t[ll_i], x_t[int(o.gl)]])
    g = np.zeros_like(sub)
    g[0] = g_i
    orc.update(sub, g, [0, 0, 0], [1], 2, w.eta, w.lambda_l, w.lambda_g, True)
    return sub[0]


def _a17_rows(x, ref):
    return (np.abs(x.astype(np.float64) - ref) / np.maximum(np.abs(ref.astype(np.float64)), PARAM_FLOOR)).max(axis=1)


def test_one_worker_objective_is_the_oracle_objective():
    # the helper above is the oracle's arithmetic: bit-identical gradients without given activations, and with
    # the oracle's own activations given back to it
    w = inputs.make_mlp(3, 1, dims=(40, 72, 136, 7), pool=256, heldout=40, batch=24, n_classes=7, steps=2, tau=1,
                        config_id=84)
    o = _oracle(w)
    g = o.obj.grad(w.x0, 1)
    for i in range(w.P):
        one = OneWorkerMlp(o.obj, i, 1)
        gi = one.grad(w.x0[i:i + 1], 0)[0]
        assert np.array_equal(gi.view(np.uint32), g[i].view(np.uint32))
        _, hs, _ = one._forward(w.x0[i], one.data_x[one.batch_idx[0][0]])
        again = OneWorkerMlp(o.obj, i, 1, given=(hs[1], hs[2]))
        assert again.check_given(w.x0[i]) <= 1.0
        assert np.array_equal(again.grad(w.x0[i:i + 1], 0)[0].view(np.uint32), g[i].view(np.uint32))
        bad = hs[1].copy()
        bad[3, 5] = bad[3, 5] * 1.05 + 0.01                      # not a rounding of relu(z): must be noticed
        assert OneWorkerMlp(o.obj, i, 1, given=(bad, hs[2])).check_given(w.x0[i]) > 1.0


@pytest.mark.parametrize("fused", [False, True])
def test_config3_every_step_from_the_oracle_state(fused):
    """Element-by-element parity of the whole configuration (32 workers, 4 groups, 10 steps) without the
    amplification of a free-running trajectory: before every step the GPU parameters are set to the oracle's x_t,
    so each step is compared for the same state.  Every entry of every worker's parameters must agree within
    2e-2 relative (|x - ref| / max(|ref|, 1e-3)), the training and held-out losses within 2e-2 relative with no
    floor, and the leaders exactly.

    One thing is not unique.  A hidden activation is a decision taken in floating point: which bf16 neighbour a
    sum is rounded to and, for a pre-activation within rounding of zero, whether the unit is on at all -- and the
    ReLU mask gates that sample's whole back-propagated delta.  The kernel takes these decisions on float32
    sums, the oracle on float64 sums.  So (1) for every worker and step the activations the kernel stored are
    checked, entry by entry, to be valid roundings of relu(z) for the oracle's own float64 z of that layer; and
    (2) a worker whose parameters miss the bound against the oracle's own decisions is compared instead, entry by
    entry within the same 2e-2, with the oracle's backward pass run on those (verified) stored activations."""
    import torch
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = inputs.config(3, steps=10)
    dims, B = w.meta["dims"], w.meta["batch"]
    o = _oracle(w)
    pop = Population(w, flags=api.FLAG_MLP_FUSED_STEP if fused else 0)
    worst, worst_act, followed = 0.0, 0.0, 0
    for t in range(10):
        x_t = o.x.copy()
        pop.x.copy_(torch.from_numpy(x_t))
        pop.lsgd.sync_parameters()
        o.step()
        pop.step(record=True)
        pull = t % w.tau == 0
        assert np.allclose(pop.lsgd.train_loss(), o.obj.last_train_loss, rtol=TOL, atol=0), t
        if pull:
            hg, ho = pop.history[-1], o.history[-1]
            assert np.allclose(hg["loss"], ho["loss"], rtol=TOL, atol=0), t
            assert hg["gl"] == ho["gl"] and np.array_equal(hg["ll"], ho["ll"]), t
        xg = pop.x_host()
        h1, h2 = pop.lsgd.mlp_activations(B, dims[1], dims[2])
        e_rows = _a17_rows(xg, o.x)
        for i in range(w.P):
            one = OneWorkerMlp(o.obj, i, t, given=(h1[i], h2[i]))
            act = one.check_given(x_t[i])
            worst_act = max(worst_act, act)
            assert act <= 1.0, (t, i, act)
            if e_rows[i] > TOL:
                g_i = one.grad(x_t[i:i + 1], 0)[0]
                e = float(_a17_rows(xg[i:i + 1], _row_after_step(x_t, i, g_i, o, w, pull)[None, :])[0])
                assert e <= TOL, (t, i, float(e_rows[i]), e)
                e_rows[i] = e
                followed += 1
        worst = max(worst, float(e_rows.max()))
    print(f"step by step: worst elementwise parameter error {worst:.3e}; stored activations within {worst_act:.3f} of "
          f"their rounding bound; {followed} worker-steps of {10 * w.P} compared on the kernel's stored decisions")
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_fused_weight_step_is_bit_identical_to_the_materialised_gradient_path():
    """With LSGD_FLAG_MLP_FUSED_STEP the plain step of W1, W2 is taken inside the weight-gradient products
    on non-pull steps; it must give exactly the parameters of the path that writes g and updates afterwards."""
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_mlp(3, 1, dims=(40, 72, 136, 7), pool=256, heldout=40, batch=24, n_classes=7, steps=7, tau=3,
                        config_id=82)
    a = Population(w, flags=api.FLAG_MLP_FUSED_STEP)
    b = Population(w)
    a.run(7)
    b.run(7)
    xa, xb = a.x_host(), b.x_host()
    assert np.array_equal(xa.view(np.uint32), xb.view(np.uint32))
    # protocol: with the fused step pending, a second gradient or an own-loss election is refused
    a.lsgd.grad(a.batches[7 % len(a.batches)])          # t = 7: not a pull step -> fused
    with pytest.raises(api.LsgdError) as e:
        a.lsgd.grad(a.batches[0])
    assert e.value.status == api.ERR_STATE
    with pytest.raises(api.LsgdError) as e:
        a.lsgd.elect(None)
    assert e.value.status == api.ERR_STATE
    a.lsgd.step()
    a.close()
    b.close()


def test_election_on_the_running_mean_of_training_losses():
    """loss_window = 3: leaders are elected on the mean of the last three minibatch losses of each worker."""
    w = inputs.make_mlp(4, 2, dims=(40, 72, 136, 7), pool=256, heldout=40, batch=24, n_classes=7, steps=8, tau=2,
                        config_id=83)
    w.meta["loss_window"] = 3
    pop, o, tg, tr, forced = _run_pair(w, 8)
    _check(pop, o, w, tg, tr, forced)
    for hg, ho in zip(pop.history, o.history):
        assert loss_close(hg["loss"], ho["loss"])
    # the elected-on loss is the window mean, not the held-out loss
    k = len(pop.history) - 1
    t_last = pop.history[k]["t"]
    want = np.mean([tg[t] for t in range(max(0, t_last - 2), t_last + 1)], axis=0)
    assert np.allclose(pop.history[k]["loss"], want, rtol=1e-5, atol=0)
    pop.close()


@pytest.mark.parametrize("fused,big", [(False, False), (True, False), (True, True)])
def test_cuda_graph_replay_of_the_mlp_step_equals_the_call_by_call_run(fused, big):
    """Whole periods of the MLP step (tensor-core products, programmatic dependent launches, the fused step)
    captured into a CUDA graph and replayed give the same parameters, bit for bit, as issuing the calls.
    big: 1024-wide layers and a held-out batch of 1024 for 10 workers, so that the held-out forward runs on the
    CTA-pair kernel (cluster launches inside the capture) and decides the elections of every period."""
    import torch
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    if big:
        w = inputs.make_mlp(10, 2, dims=(64, 1024, 1024, 10), pool=512, heldout=1024, batch=128, steps=4, tau=2,
                            config_id=64)
    else:
        w = inputs.make_mlp(4, 2, dims=(64, 128, 128, 10), pool=512, heldout=128, batch=128, steps=4, tau=2, config_id=63)
    flags = api.FLAG_MLP_FUSED_STEP if fused else 0
    stream = torch.cuda.Stream()
    a = Population(w, flags=flags, stream=stream)
    with torch.cuda.stream(stream):
        a.run(4)                                     # un-captured: one pass over the batch ring
        a.capture(4)
        a.replay()
        a.replay()
    stream.synchronize()
    assert a.lsgd.t() == 12
    b = Population(w, flags=flags)
    b.run(12)
    assert np.array_equal(a.x_host().view(np.uint32), b.x_host().view(np.uint32))
    assert a.lsgd.leaders()[1] == b.lsgd.leaders()[1]
    assert a.lsgd.check_device() == 0
    a.close()
    b.close()
