"""The pins are only worth something if a plausible mistake in the oracle trips them.  Each case plants
one mistake IN THE ORACLE (on the CPU; nothing here touches the GPU path) and checks that at least
one named pin fails."""
import numpy as np
import pytest

from oracle import lsgd_oracle as orc
from tests import test_oracle_pins as pins

F32, F64 = np.float32, np.float64


def _update_variant(kind):
    def update(x, g, group_of, ll, gl, eta, lambda_l, lambda_g, pull):
        eta, lambda_l, lambda_g = float(F32(eta)), float(F32(lambda_l)), float(F32(lambda_g))
        P = x.shape[0]
        snap = x.astype(F64)
        for i in range(P):
            src = x.astype(F64) if kind == "gauss_seidel" else snap      # later rows see updated leaders
            xi = src[i]
            new = xi - eta * g[i].astype(F64)
            if pull:
                zl, zg = src[int(ll[int(group_of[i])])], src[int(gl)]
                cl, cg = eta * lambda_l, eta * lambda_g
                if kind == "unscaled":
                    cl, cg = lambda_l, lambda_g
                if kind == "drop_global":
                    cg = 0.0
                if kind == "wrong_sign":
                    cl, cg = -cl, -cg
                if kind == "swapped_leaders":
                    zl, zg = zg, zl
                if kind == "pull_on_new":                                 # pulls evaluated after the gradient step
                    new = new - cl * (new - zl) - cg * (new - zg)
                else:
                    new = new - cl * (xi - zl) - cg * (xi - zg)
            elif kind == "pull_every_step":
                pass
            x[i] = new.astype(F32)
    return update


UPDATE_CASES = {
    "unscaled": [pins.test_update_matches_written_out_form, pins.test_closed_form_single_leader_tau1],
    "drop_global": [pins.test_two_pulls_equal_one_combined_pull, pins.test_closed_form_multi_leader_with_period],
    "wrong_sign": [pins.test_update_matches_written_out_form],
    "swapped_leaders": [pins.test_closed_form_multi_leader_with_period],
    "gauss_seidel": [pins.test_closed_form_multi_leader_with_period, pins.test_two_pulls_equal_one_combined_pull],
    "pull_on_new": [pins.test_update_matches_written_out_form, pins.test_closed_form_single_leader_tau1],
}


def _fails(fn, *args):
    try:
        fn(*args)
    except AssertionError:
        return True
    return False


@pytest.mark.parametrize("kind", sorted(UPDATE_CASES))
def test_update_mistakes_are_caught(kind, monkeypatch):
    monkeypatch.setattr(orc, "update", _update_variant(kind))
    assert any(_fails(fn) for fn in UPDATE_CASES[kind]), kind


def test_correct_update_variant_passes(monkeypatch):
    # the harness itself: the same re-implementation without a planted mistake passes every pin used above
    monkeypatch.setattr(orc, "update", _update_variant("none"))
    for fns in UPDATE_CASES.values():
        for fn in fns:
            fn()


def test_election_mistakes_are_caught(monkeypatch):
    good = orc.elect

    def ties_to_highest(loss, group_of, G):
        P = len(loss)
        ll, gl = good(np.asarray(loss)[::-1], np.asarray(group_of)[::-1], G)
        return np.asarray([P - 1 - v for v in ll], dtype=np.int32), P - 1 - gl

    def nan_is_smallest(loss, group_of, G):
        l = np.where(np.isnan(loss), -np.inf, loss).astype(F32)
        return good(l, group_of, G)

    def global_over_first_group(loss, group_of, G):
        ll, _ = good(loss, group_of, G)
        return ll, int(ll[0])

    for bad in (ties_to_highest, nan_is_smallest, global_over_first_group):
        monkeypatch.setattr(orc, "elect", bad)
        assert _fails(pins.test_election_matches_brute_force_exhaustively) or _fails(pins.test_election_tie_examples), bad.__name__


def test_schedule_mistakes_are_caught(monkeypatch):
    # pulling on every step instead of every tau-th, and electing off by one
    orig = orc.LsgdOracle.step

    def pull_every_step(self, forced_loss=None):
        tau, self.tau = self.tau, 1
        try:
            orig(self, forced_loss)
        finally:
            self.tau = tau

    monkeypatch.setattr(orc.LsgdOracle, "step", pull_every_step)
    assert _fails(pins.test_closed_form_multi_leader_with_period)


def test_gradient_mistakes_are_caught(monkeypatch):
    good = orc.Quadratic.grad

    def grad_without_a(self, x, t):
        a, self.a = self.a, np.ones_like(self.a)
        try:
            return good(self, x, t)
        finally:
            self.a = a

    monkeypatch.setattr(orc.Quadratic, "grad", grad_without_a)
    assert _fails(pins.test_quadratic_gradient_and_loss) and _fails(pins.test_closed_form_single_leader_tau1)
    monkeypatch.setattr(orc.Quadratic, "grad", good)

    good_mc = orc.MatComp.grad

    def mc_grad_transposed(self, x, t):                     # dX and dY exchanged
        g = good_mc(self, x, t)
        nx, ny = self.n_rows * self.rank, self.n_cols * self.rank
        out = np.zeros_like(g)
        k = min(nx, ny)
        out[:, :k] = g[:, nx:nx + k]
        out[:, nx:nx + k] = g[:, :k]
        return out

    monkeypatch.setattr(orc.MatComp, "grad", mc_grad_transposed)
    assert _fails(pins.test_matcomp_gradient_finite_differences_with_duplicates)
    monkeypatch.setattr(orc.MatComp, "grad", good_mc)

    good_round = orc.bf16_round
    monkeypatch.setattr(orc, "bf16_round", lambda a: (np.asarray(a, F32).view(np.uint32) & 0xFFFF0000).view(F32))  # truncation
    assert _fails(pins.test_mlp_bf16emu_is_close_to_fp32_and_rounding_matches_library)
    monkeypatch.setattr(orc, "bf16_round", good_round)


# ---- the Section 4.1 optimiser ------------------------------------------------------------------------
from tests import test_oracle_momentum as mpins  # noqa: E402


def _momentum_variant(kind):
    def momentum_update(x, v, g, group_of, ll, gl, eta, lambda_l, lambda_g, pull, mu, wd):
        eta, lambda_l, lambda_g, mu, wd = (float(F32(q)) for q in (eta, lambda_l, lambda_g, mu, wd))
        snap = x.astype(F64)
        for i in range(x.shape[0]):
            xi = snap[i]
            d = g[i].astype(F64) + (-wd if kind == "decay_sign" else wd) * xi
            pulls = 0.0
            if pull:
                pulls = lambda_l * (xi - snap[int(ll[int(group_of[i])])]) + lambda_g * (xi - snap[int(gl)])
            if kind == "pull_in_buffer":                       # the pulls treated as part of the gradient
                d = d + pulls
                pulls = 0.0
            vn = mu * v[i].astype(F64) + d
            if kind == "classical":                            # heavy ball: step along the buffer itself
                u = vn
            elif kind == "lookahead_on_old_buffer":
                u = d + mu * v[i].astype(F64)
            else:
                u = d + mu * vn
            x[i] = (xi - eta * u - eta * pulls).astype(F32)
            v[i] = vn.astype(F32)
    return momentum_update


MOMENTUM_CASES = {
    "classical": [mpins.test_without_pulls_it_is_the_library_nesterov_sgd,
                  mpins.test_closed_form_on_the_quadratic_is_a_two_by_two_recurrence],
    "lookahead_on_old_buffer": [mpins.test_closed_form_on_the_quadratic_is_a_two_by_two_recurrence],
    "decay_sign": [mpins.test_weight_decay_moves_the_fixed_point, mpins.test_without_pulls_it_is_the_library_nesterov_sgd],
    "pull_in_buffer": [mpins.test_pulls_stay_outside_the_momentum_buffer],
}


@pytest.mark.filterwarnings("ignore::RuntimeWarning")      # a planted sign error may diverge
@pytest.mark.parametrize("kind", sorted(MOMENTUM_CASES))
def test_momentum_mistakes_are_caught(kind, monkeypatch):
    monkeypatch.setattr(orc, "momentum_update", _momentum_variant(kind))
    for fn in MOMENTUM_CASES[kind]:
        assert _fails(fn), (kind, fn.__name__)


def test_correct_momentum_variant_passes(monkeypatch):
    monkeypatch.setattr(orc, "momentum_update", _momentum_variant("none"))
    for fns in MOMENTUM_CASES.values():
        for fn in fns:
            fn()
    mpins.test_zero_momentum_and_decay_is_eq1()
