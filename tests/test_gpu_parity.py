"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer results (leaders) are compared bit-exactly; fp32 trajectories with the metric

    rel = max |x_gpu - x_ref| / max(|x_ref|, FLOOR),   FLOOR = 1e-3

and the bound 1e-5 after 10 steps.  In the default arithmetic (fp64 evaluation, one rounding) the
update is additionally expected to be bit-identical to the oracle's."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu

F32 = np.float32
FLOOR = 1e-3
TOL = 1e-5


def rel_err(x, ref, floor=FLOOR):
    return float((np.abs(x.astype(np.float64) - ref) / np.maximum(np.abs(ref), floor)).max())


def _pop(w, **kw):
    from paper_1905_10395_b200.runner import Population
    return Population(w, **kw)


def _oracle(w, **over):
    A = w.arrays
    if w.objective == "external":
        obj = orc.External(A["g"], A["loss_ring"])
    elif w.objective == "quadratic":
        obj = orc.Quadratic(A["a"], A["b"], w.meta["sigma"], A.get("noise"))
    elif w.objective == "matcomp":
        m = w.meta
        obj = orc.MatComp(m["n_rows"], m["n_cols"], m["rank"], A["obs_r"], A["obs_c"], A["obs_v"],
                          A["batch_pos"], A["heldout_pos"])
    elif w.objective == "psd":
        obj = orc.PsdCompletion(w.meta["n"], w.meta["r"], A["M"])
    else:
        raise ValueError
    return orc.LsgdOracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau)


def _leaders_equal(pop, o):
    assert len(pop.history) == len(o.history)
    for hg, ho in zip(pop.history, o.history):
        assert hg["t"] == ho["t"]
        assert np.array_equal(hg["ll"], ho["ll"]), (hg, ho)
        assert hg["gl"] == ho["gl"]


# ------------------------------------------------------------------------------------ election ----
def test_election_bit_exact_random_groups_ties_and_specials():
    import torch
    from paper_1905_10395_b200 import api
    rng = np.random.default_rng(7)
    specials = np.asarray([-np.inf, -1.0, -0.0, 0.0, 1.0, np.inf, np.nan, 0.5, 0.25], dtype=F32)
    for trial in range(60):
        P = int(rng.integers(1, 300)) if trial % 3 else int(rng.integers(1, 9))
        G = int(rng.integers(1, P + 1))
        m = np.concatenate([np.arange(G), rng.integers(0, G, P - G)]).astype(np.int32)
        rng.shuffle(m)
        x = torch.zeros(P, 32, device="cuda")
        g = torch.zeros(P, 32, device="cuda")
        cfg, keep = api.make_config(P=P, G=G, group_of=m, d=32, ld=32, eta=0.1, lambda_l=0.1, lambda_g=0.1, tau=1,
                                    objective=api.OBJ_EXTERNAL, x=x, g=g)
        h = api.Lsgd(cfg, keep)
        for rep in range(3):
            if rep == 0:
                loss = specials[rng.integers(0, len(specials), P)]
            elif rep == 1:
                loss = rng.integers(0, 3, P).astype(F32)
            else:
                loss = rng.standard_normal(P).astype(F32)
            h.elect(torch.from_numpy(loss).cuda())
            ll, gl = h.leaders()
            ll_ref, gl_ref = orc.elect(loss, m, G)
            assert np.array_equal(ll, ll_ref) and gl == gl_ref, (P, G, rep)
            got = h.loss()
            assert np.array_equal(got.view(np.uint32), loss.view(np.uint32))
        cg, cl = h.leader_counts()
        assert cg.sum() == 3 and cl.sum() == 3 * G
        assert h.check_device() == 0
        h.destroy()


# ----------------------------------------------------------------------------- external update ----
@pytest.mark.parametrize("arith,exact", [(0, True), (1, False), (2, False)])
def test_external_update_ragged_unequal_groups(arith, exact):
    group_of = np.asarray([2, 0, 1, 1, 0, 2, 2], dtype=np.int32)          # unequal, interleaved
    w = inputs.make_external(7, 3, 4999, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=10,
                             loss_ring=5, config_id=50, group_of=group_of)
    pop = _pop(w, arithmetic=arith)
    pop.run(10, record=True)
    o = _oracle(w)
    o.run(10)
    _leaders_equal(pop, o)
    x = pop.x_host()
    if exact:
        assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
    # fp32 arithmetic (mode 2) cannot bound the error of a cancelling result relative to the result
    # itself, only relative to the O(1) operands; the fp64 modes meet the bound with the 1e-3 floor
    assert rel_err(x, o.x, floor=1.0 if arith == 2 else FLOOR) <= TOL
    assert np.all(x[:, w.d:] == 0)
    assert pop.lsgd.check_device() == 0
    pop.close()


@pytest.mark.parametrize("leader_rows", ["last", "first", "rotating"])
def test_in_place_update_reads_time_t_leaders(leader_rows):
    # every right-hand side is x_t although x is overwritten: put the leader in the first / last row
    # and change it every step
    P, G, d = 12, 3, 300000                                               # several CTAs, ragged tail
    w = inputs.make_external(P, G, d, eta=0.1, lambda_l=0.3, lambda_g=0.2, tau=1, steps=6, loss_ring=6,
                             config_id=51)
    ring = w.arrays["loss_ring"]
    for n in range(len(ring)):
        ring[n] = 1.0 + np.arange(P, dtype=F32)
        lead = {"last": P - 1, "first": 0, "rotating": (5 * n + 3) % P}[leader_rows]
        ring[n, lead] = 0.0
        ring[n, (lead + 4) % P] = 0.5
    pop = _pop(w)
    pop.run(6, record=True)
    o = _oracle(w)
    o.run(6)
    _leaders_equal(pop, o)
    assert np.array_equal(pop.x_host().view(np.uint32), o.x.view(np.uint32))
    pop.close()


def test_zero_pull_and_leader_rows_match_plain_step_bitwise():
    import torch
    # the leader's own pull term is exactly zero in every arithmetic mode
    for arith in (0, 1, 2):
        w = inputs.make_external(6, 2, 2048, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=1, steps=1,
                                 config_id=52)
        pull = _pop(w, arithmetic=arith)
        pull.run(1, record=True)
        w0 = inputs.make_external(6, 2, 2048, eta=0.05, lambda_l=0.0, lambda_g=0.0, tau=1, steps=1,
                                  config_id=52)
        plain = _pop(w0, arithmetic=arith)
        plain.run(1)
        gl = pull.history[0]["gl"]
        assert np.array_equal(pull.x_host()[gl], plain.x_host()[gl])
        pull.close()
        plain.close()


# ----------------------------------------------------------------------------------- quadratic ----
@pytest.mark.parametrize("fused", [False, True])
def test_config0_single_leader_quadratic(fused):
    w = inputs.config(0)
    pop = _pop(w, fused_quadratic=fused)
    pop.run(w.steps, record=True)
    o = _oracle(w)
    o.run(w.steps)
    _leaders_equal(pop, o)
    for hg, ho in zip(pop.history, o.history):
        assert np.allclose(hg["loss"], ho["loss"], rtol=3e-7, atol=0)
    x = pop.x_host()
    assert rel_err(x, o.x) <= TOL
    assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
    pop.close()


@pytest.mark.parametrize("fused,arith", [(False, 0), (True, 0), (True, 2)])
def test_config1_reduced_multi_leader_quadratic(fused, arith):
    w = inputs.config(1, d=(1 << 16) + 40, steps=12)                      # ragged: not a tile multiple
    pop = _pop(w, fused_quadratic=fused, arithmetic=arith)
    pop.run(10, record=True)
    o = _oracle(w)
    o.run(10)
    _leaders_equal(pop, o)
    for hg, ho in zip(pop.history, o.history):      # with the fused gradient the loss is summed inside the previous step
        assert np.allclose(hg["loss"], ho["loss"], rtol=3e-7 if arith == 0 else 1e-5, atol=0)
    x = pop.x_host()
    if arith == 0:
        assert rel_err(x, o.x) <= TOL
        assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
    else:
        # fp32 arithmetic cannot bound the error of a cancelling result relative to the result
        # itself; it is bounded relative to the operands, which are O(1)
        assert rel_err(x, o.x, floor=1.0) <= TOL
    pop.close()


def test_config1_full_size_at_step_10_and_step_100():
    """The whole configuration: 64 workers in 8 groups, d = 2^20, tau = 4, the noise ring reused cyclically,
    compared on every entry after 10 steps and again at the end of the 100-step run."""
    w = inputs.config(1)
    pop = _pop(w, fused_quadratic=True)
    o = _oracle(w)
    done = 0
    for upto in (10, 100):
        pop.run(upto - done, record=True)
        o.run(upto - done)
        done = upto
        _leaders_equal(pop, o)
        for hg, ho in zip(pop.history, o.history):
            assert np.allclose(hg["loss"], ho["loss"], rtol=3e-7, atol=0), (upto, hg["t"])
        x = pop.x_host()
        e = rel_err(x, o.x)
        assert e <= TOL, (upto, e)
    assert len(o.history) == 25
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_quadratic_noise_free_lgd_and_closed_form():
    # batch LGD on the diagonal quadratic: GPU iterates against the closed-form linear recursion
    wl = inputs.config(0)
    wl.x0[0] = wl.arrays["b"] + F32(0.01) * wl.x0[0]
    wl.arrays["noise"] = None
    wl.meta["sigma"] = 0.0
    pop = _pop(wl, fused_quadratic=True, upload_noise=False)
    T = 10
    pop.run(T, record=True)
    assert all(h["gl"] == 0 for h in pop.history)
    a, b = wl.arrays["a"].astype(np.float64), wl.arrays["b"].astype(np.float64)
    eta, lam = float(F32(wl.eta)), float(F32(wl.lambda_l))
    x = pop.x_host()
    w_t = b + (1 - eta * a) ** T * (wl.x0[0].astype(np.float64) - b)
    assert np.allclose(x[0], w_t, rtol=0, atol=2e-6)
    for i in range(1, wl.P):
        x_t = w_t + (1 - eta * (a + lam)) ** T * (wl.x0[i].astype(np.float64) - wl.x0[0].astype(np.float64))
        assert np.allclose(x[i], x_t, rtol=0, atol=2e-6)
    pop.close()


# ----------------------------------------------------------------------------- matrix completion ----
def test_matcomp_small_with_duplicates():
    w = inputs.make_matcomp(5, 2, n_rows=300, n_cols=200, rank=7, n_obs=5000, n_heldout=1000, batch=700,
                            steps=10, tau=3, config_id=53)
    pop = _pop(w)
    pop.run(10, record=True)
    o = _oracle(w)
    o.run(10)
    _leaders_equal(pop, o)
    for hg, ho in zip(pop.history, o.history):
        assert np.allclose(hg["loss"], ho["loss"], rtol=1e-6, atol=0)
    assert rel_err(pop.x_host(), o.x) <= TOL
    assert pop.lsgd.check_device() == 0
    pop.close()


@pytest.mark.parametrize("rank", [3, 10, 20])
def test_matcomp_fused_step_is_bit_identical_to_the_materialised_gradient_path(rank):
    """With LSGD_FLAG_MATCOMP_FUSED_STEP a plain step is taken straight from the fixed-point gradient sums
    (g is not written): same x, bit for bit, as gradient kernel + update kernel, and within tolerance of the
    oracle.  Ranks on all three lane-group widths of the sparse kernels."""
    from paper_1905_10395_b200 import api
    w = inputs.make_matcomp(6, 2, n_rows=257, n_cols=190, rank=rank, n_obs=6000, n_heldout=1500, batch=900,
                            steps=9, tau=4, config_id=54)
    a = _pop(w, flags=api.FLAG_MATCOMP_FUSED_STEP)
    b = _pop(w)
    a.run(9, record=True)
    b.run(9, record=True)
    assert np.array_equal(a.x_host().view(np.uint32), b.x_host().view(np.uint32))
    o = _oracle(w)
    o.run(9)
    _leaders_equal(a, o)
    assert rel_err(a.x_host(), o.x) <= TOL
    # protocol: a second gradient while the sums of the first wait for lsgd_step is refused (t = 9: not a pull step)
    a.lsgd.grad(a.batches[9 % len(a.batches)])
    with pytest.raises(api.LsgdError) as e:
        a.lsgd.grad(a.batches[9 % len(a.batches)])
    assert e.value.status == api.ERR_STATE
    a.lsgd.step()
    assert a.lsgd.check_device() == 0
    a.close()
    b.close()


@pytest.mark.parametrize("fused", [False, True])
def test_config2_matrix_completion(fused):
    # fused = the configuration the benchmark times (LSGD_FLAG_MATCOMP_FUSED_STEP)
    from paper_1905_10395_b200 import api
    w = inputs.config(2, steps=10)
    pop = _pop(w, flags=api.FLAG_MATCOMP_FUSED_STEP if fused else 0)
    pop.run(10, record=True)
    o = _oracle(w)
    o.run(10)
    _leaders_equal(pop, o)
    assert rel_err(pop.x_host(), o.x) <= TOL
    pop.close()


# ------------------------------------------------------------------- full-size fused update (C4) ----
@pytest.mark.parametrize("tau", [1, 16])
def test_config4_full_size_sampled_columns(tau):
    """The bench workload in the bench's launch configuration.  The update is separable by column
    once the leaders are known, so the oracle is run on a sample of columns (first / last tiles and
    random ones) and compared bit-exactly."""
    w = inputs.config(4, tau=tau)
    steps = 3 if tau == 1 else 18
    rng = np.random.default_rng(4)
    cols = np.unique(np.concatenate([np.arange(0, 2048), np.arange(w.d - 2048, w.d),
                                     rng.integers(0, w.d, 20000)]))
    sub = inputs.Workload(name="C4-sample", objective="external", P=w.P, G=w.G, d=len(cols), ld=len(cols),
                          group_of=w.group_of, eta=w.eta, lambda_l=w.lambda_l, lambda_g=w.lambda_g, tau=tau,
                          steps=steps, x0=np.ascontiguousarray(w.x0[:, cols]),
                          arrays={"g": np.ascontiguousarray(w.arrays["g"][:, cols]),
                                  "loss_ring": w.arrays["loss_ring"]})
    pop = _pop(w)
    pop.run(steps, record=True)
    o = _oracle(sub)
    o.run(steps)
    _leaders_equal(pop, o)
    import torch
    got = pop.x[:, torch.from_numpy(cols).cuda()].cpu().numpy()
    assert np.array_equal(got.view(np.uint32), o.x.view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


# ------------------------------------------------------------------------------------ protocol ----
def test_step_protocol_errors():
    import torch
    from paper_1905_10395_b200 import api
    w = inputs.make_quadratic(4, 2, 64, eta=0.1, lambda_l=0.1, lambda_g=0.1, tau=2, steps=2, config_id=54)
    pop = _pop(w)
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.step()                                                   # no gradient yet
    assert e.value.status == api.ERR_STATE
    pop.lsgd.grad(pop.batches[0])
    with pytest.raises(api.LsgdError) as e:
        pop.lsgd.step()                                                   # pull step before any election
    assert e.value.status == api.ERR_STATE
    pop.lsgd.elect(None)
    pop.lsgd.step()
    assert pop.lsgd.t() == 1
    pop.lsgd.grad(pop.batches[1])
    pop.lsgd.step()                                                       # t = 1: plain step, no election
    assert pop.lsgd.t() == 2
    pop.close()


def test_center_variable_bit_exact():
    import torch
    w = inputs.make_external(11, 3, 70001, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=3, config_id=55)
    pop = _pop(w)
    pop.run(3)
    out = torch.empty(w.ld, device="cuda")
    pop.lsgd.center(out)
    o = _oracle(w)
    o.run(3)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), orc.center_variable(o.x).view(np.uint32))
    pop.close()


# -------------------------------------------------- dense PSD completion (the paper's own experiment) ----
@pytest.mark.parametrize("n,r", [(100, 1), (203, 10), (1000, 50), (257, 128)])
def test_psd_completion_lgd(n, r):
    """LGD at the paper's settings (eta 5e-4, lambda 1/5, 8 workers, tau 1), ragged n and all rank regimes."""
    w = inputs.make_psd(P=8, n=n, r=r, steps=10, config_id=56)
    pop = _pop(w)
    pop.run(10, record=True)
    o = _oracle(w)
    o.run(10)
    _leaders_equal(pop, o)
    for hg, ho in zip(pop.history, o.history):
        assert np.allclose(hg["loss"], ho["loss"], rtol=1e-6, atol=0)
    assert rel_err(pop.x_host(), o.x) <= TOL
    assert pop.lsgd.check_device() == 0
    pop.close()


def test_matcomp_gradient_is_reproducible_bit_for_bit():
    # heavy duplication (batch 3000 over 60 rows / 50 columns): the scatter-add must not depend on atomics order
    w = inputs.make_matcomp(4, 2, n_rows=60, n_cols=50, rank=10, n_obs=2500, n_heldout=256, batch=3000, steps=4, tau=2,
                            config_id=57)
    runs = []
    for _ in range(3):
        pop = _pop(w)
        pop.run(4)
        runs.append(pop.x_host().copy())
        pop.close()
    assert np.array_equal(runs[0].view(np.uint32), runs[1].view(np.uint32))
    assert np.array_equal(runs[0].view(np.uint32), runs[2].view(np.uint32))
    o = _oracle(w)
    o.run(4)
    assert rel_err(runs[0], o.x) <= TOL


@pytest.mark.parametrize("kind", ["quadratic", "matcomp", "matcomp_fused"])
def test_cuda_graph_replay_matches_the_oracle(kind):
    """Whole communication periods captured into a CUDA graph and replayed (lsgd_advance_step keeps the
    library's step counter in line) give the same trajectory as issuing the calls one by one."""
    import torch
    if kind == "quadratic":
        w = inputs.config(0, d=3000, tau=2, steps=12, noise_ring=4)
    else:
        w = inputs.make_matcomp(4, 2, n_rows=300, n_cols=200, rank=7, n_obs=5000, n_heldout=512, batch=700, steps=4,
                                tau=2, config_id=58)
    from paper_1905_10395_b200 import api
    stream = torch.cuda.Stream()
    pop = _pop(w, fused_quadratic=(kind == "quadratic"), stream=stream,
               flags=api.FLAG_MATCOMP_FUSED_STEP if kind == "matcomp_fused" else 0)
    with torch.cuda.stream(stream):
        pop.run(4)                                   # un-captured warm-up: one pass over the batch ring
        pop.capture(4)
        pop.replay()
        pop.replay()
    stream.synchronize()
    assert pop.lsgd.t() == 12
    o = _oracle(w)
    o.run(12)
    x = pop.x_host()
    if kind == "quadratic":
        assert np.array_equal(x.view(np.uint32), o.x.view(np.uint32))
    else:
        assert rel_err(x, o.x) <= TOL
    ll, gl = pop.lsgd.leaders()
    assert gl == o.gl and np.array_equal(ll, o.ll)
    pop.close()
