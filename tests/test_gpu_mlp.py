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


def _check(pop, o, w, train_gpu, train_ref, forced):
    x = pop.x_host().astype(np.float64)
    ref = o.x.astype(np.float64)
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


def test_config3_single_steps_from_the_oracle_state():
    """Per-step parity without the amplification of a free-running trajectory: before every step the
    GPU parameters are set to the oracle's, so each step's losses and parameter change are compared
    for the same x_t.  Losses here must agree to 2e-2 relative with no floor."""
    import torch
    from paper_1905_10395_b200.runner import Population
    w = inputs.config(3, P=8, G=2, steps=8)
    o = _oracle(w)
    pop = Population(w)
    for t in range(8):
        x_t = o.x.copy()
        pop.x.copy_(torch.from_numpy(x_t))
        pop.lsgd.sync_parameters()
        o.step()
        pop.step(record=True)
        assert np.allclose(pop.lsgd.train_loss(), o.obj.last_train_loss, rtol=TOL, atol=0), t
        if t % w.tau == 0:
            hg, ho = pop.history[-1], o.history[-1]
            assert np.allclose(hg["loss"], ho["loss"], rtol=TOL, atol=0), t
            assert hg["gl"] == ho["gl"] and np.array_equal(hg["ll"], ho["ll"]), t
        dx = pop.x_host().astype(np.float64) - x_t
        dref = o.x.astype(np.float64) - x_t
        for i in range(w.P):
            assert np.linalg.norm(dx[i] - dref[i]) <= TOL * np.linalg.norm(dref[i]), (t, i)
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


@pytest.mark.parametrize("fused", [False, True])
def test_cuda_graph_replay_of_the_mlp_step_equals_the_call_by_call_run(fused):
    """Whole periods of the MLP step (tensor-core products, programmatic dependent launches, the fused step)
    captured into a CUDA graph and replayed give the same parameters, bit for bit, as issuing the calls."""
    import torch
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
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
