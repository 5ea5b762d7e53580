"""Out-of-bounds check without a sanitizer: the caller's x and g sit inside larger allocations whose guard bands
(before, after, and the padding columns of every row beyond the last 16-byte column of d) hold a bit pattern that
no kernel may change.  One case per form of the update kernel, plus the momentum step and the inline quadratic."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu

PAD = 4096                      # floats on each side (16 KiB: more than one bulk-copy piece)
SENTINEL = 0x7FA5A5A5           # a NaN payload: any arithmetic on it would also change the bits


def _guarded(host: np.ndarray, d: int):
    import torch
    P, ld = host.shape
    big = torch.empty(P * ld + 2 * PAD, dtype=torch.int32, device="cuda")
    big.fill_(SENTINEL)
    view = big[PAD:PAD + P * ld].view(torch.float32).view(P, ld)
    view.copy_(torch.from_numpy(host))
    first_pad = (d + 3) // 4 * 4
    if first_pad < ld:
        view[:, first_pad:].view(torch.int32).fill_(SENTINEL)
    return big, view, first_pad


def _intact(big, view, first_pad):
    import torch
    torch.cuda.synchronize()
    ok = bool((big[:PAD] == SENTINEL).all()) and bool((big[-PAD:] == SENTINEL).all())
    if first_pad < view.shape[1]:
        ok = ok and bool((view[:, first_pad:].view(torch.int32) == SENTINEL).all())
    return ok


@pytest.mark.parametrize("P,G,d,kind", [(12, 3, 1001, "external"), (40, 5, 2503, "external"), (200, 100, 301, "external"),
                                        (12, 3, 1001, "momentum"), (40, 5, 2503, "momentum"), (200, 100, 301, "momentum"),
                                        (9, 3, 1001, "quadratic"), (70, 7, 2503, "quadratic")])
def test_kernels_stay_inside_the_callers_buffers(P, G, d, kind):
    from paper_1905_10395_b200.runner import Population
    steps = 4
    if kind == "quadratic":
        w = inputs.make_quadratic(P, G, d, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=2, steps=steps, noise_ring=2, config_id=160)
        xb, x, fp = _guarded(w.x0, d)
        pop = Population(w, x=x, fused_quadratic=True)
        obj = orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], w.arrays["noise"])
        bands = [(xb, x, fp)]
        kw = {}
    else:
        w = inputs.make_external(P, G, d, eta=0.05, lambda_l=0.3, lambda_g=0.2, tau=2, steps=steps, loss_ring=3, config_id=161)
        xb, x, fp = _guarded(w.x0, d)
        gb, g, _ = _guarded(w.arrays["g"], d)
        kw = dict(momentum=0.9, weight_decay=1e-4) if kind == "momentum" else {}
        pop = Population(w, x=x, g=g, **kw)
        obj = orc.External(w.arrays["g"], w.arrays["loss_ring"])
        bands = [(xb, x, fp), (gb, g, fp)]
    pop.run(steps)                                   # pull and plain steps alternate (tau = 2)
    for band in bands:
        assert _intact(*band)
    o = orc.LsgdOracle(w.x0, obj, w.group_of, w.G, w.eta, w.lambda_l, w.lambda_g, w.tau, **kw)
    o.run(steps)
    got = x[:, :d].cpu().numpy()
    assert np.array_equal(got.view(np.uint32), o.x[:, :d].view(np.uint32))
    assert pop.lsgd.check_device() == 0
    pop.close()


@pytest.mark.parametrize("fused", [False, True])
def test_matrix_completion_kernels_stay_inside_the_callers_buffers(fused):
    from paper_1905_10395_b200 import api
    from paper_1905_10395_b200.runner import Population
    w = inputs.make_matcomp(5, 2, n_rows=301, n_cols=199, rank=7, n_obs=5000, n_heldout=1000, batch=700, steps=6, tau=3,
                            config_id=162)
    xb, x, fp = _guarded(w.x0, w.d)
    gb, g, _ = _guarded(np.zeros_like(w.x0), w.d)
    pop = Population(w, x=x, g=g, flags=api.FLAG_MATCOMP_FUSED_STEP if fused else 0)
    pop.run(6)
    # g is rewritten as a whole [P][ld] array (its padding columns become zero), so only its outer bands count
    assert _intact(xb, x, fp) and _intact(gb, g, g.shape[1])
    m, A = w.meta, w.arrays
    o = orc.LsgdOracle(w.x0, orc.MatComp(m["n_rows"], m["n_cols"], m["rank"], A["obs_r"], A["obs_c"], A["obs_v"],
                                         A["batch_pos"], A["heldout_pos"]), w.group_of, w.G, w.eta, w.lambda_l,
                       w.lambda_g, w.tau)
    o.run(6)
    got, ref = x[:, : w.d].cpu().numpy().astype(np.float64), o.x[:, : w.d].astype(np.float64)
    assert float((np.abs(got - ref) / np.maximum(np.abs(ref), 1e-3)).max()) <= 1e-5
    assert pop.lsgd.check_device() == 0
    pop.close()
