"""GPU test of lsgd_quadratic_loss_noalloc, the entry point for callers that may not allocate device
memory (pool-managed regions, no-allocation-after-start-up loops, guests in a foreign CUDA context).

It keeps its scratch in a fixed array inside the library, so the checks are: the result equals the
regular path's (lsgd_elect with the objective's own loss, which uses cudaMalloc'd scratch) bit for
bit, on two calls in a row with different inputs -- the second call finds the first call's values
still in the shared array -- and an over-capacity problem is refused.  Collected last on purpose."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from paper_1905_10395_b200 import inputs

pytestmark = pytest.mark.gpu


def _regular_loss(w):
    from paper_1905_10395_b200.runner import Population
    pop = Population(w, fused_quadratic=True)
    pop.lsgd.elect(None)
    loss = pop.lsgd.loss()
    return pop, loss


def test_noalloc_loss_matches_regular_entry_point_twice_in_a_row():
    import torch
    from paper_1905_10395_b200 import api
    shapes = [(7, 3, 40000 + 13), (5, 1, 9000)]         # several chunks with a ragged tail, then a smaller one
    for call, (P, G, d) in enumerate(shapes):
        w = inputs.make_quadratic(P, G, d, eta=0.05, lambda_l=0.1, lambda_g=0.05, tau=1, steps=1, noise_ring=1,
                                  config_id=70 + call)
        pop, want = _regular_loss(w)
        out = torch.full((P,), float("nan"), device="cuda")
        api.lsgd_quadratic_loss_noalloc(pop.x, pop.a, pop.b, P, w.d, w.ld, out,
                                        torch.cuda.current_stream().cuda_stream)
        got = out.cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (call, got, want)
        # and against the oracle's election loss, within the tolerance the parity tests use for losses
        ref = orc.Quadratic(w.arrays["a"], w.arrays["b"], w.meta["sigma"], None).loss(w.x0, 0)
        assert np.allclose(got, ref, rtol=3e-7, atol=0)
        pop.close()


def test_noalloc_rejects_problems_beyond_the_fixed_scratch():
    import torch
    from paper_1905_10395_b200 import api
    P, d = 64, 8192 * 1025                               # 64 * 1025 partials > 65536
    dummy = torch.zeros(64, device="cuda")
    with pytest.raises(api.LsgdError) as e:              # rejected on the host: nothing is dereferenced
        api.lsgd_quadratic_loss_noalloc(dummy, dummy, dummy, P, d, d, dummy)
    assert e.value.status == api.ERR_TOO_LARGE
