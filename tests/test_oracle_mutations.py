"""The pins must catch plausible mistakes: each test plants one in the oracle (on the CPU, by
monkeypatching) and checks that a pin from the other test files then fails."""
import math

import numpy as np
import pytest

from oracle import localsgd_oracle as orc
from tests import test_oracle_adacomm as pins_tau
from tests import test_oracle_average as pins_avg
from tests import test_oracle_gradients as pins_grad
from tests import test_oracle_pasgd as pins_loop


def _fails(fn, *args):
    try:
        fn(*args)
    except AssertionError:
        return True
    except Exception:
        return True          # a crash is also a detected mistake
    return False


def test_pins_pass_on_the_unmodified_oracle():
    pins_grad.test_gradient_matches_central_differences((5, 4, 3), orc.LOSS_SOFTMAX_CE, True)
    pins_loop.test_m1_is_plain_sgd(0.9)
    pins_avg.test_brute_force_scalar_fp32_chain(4)
    pins_tau.test_hand_table()


def test_dropped_batch_normalisation_is_caught(monkeypatch):
    real = orc.loss_and_grad
    monkeypatch.setattr(orc, "loss_and_grad", lambda s, x, X, y: (real(s, x, X, y)[0], real(s, x, X, y)[1] * X.shape[0]))
    assert _fails(pins_grad.test_gradient_matches_central_differences, (5, 4, 3), orc.LOSS_SOFTMAX_CE, True)
    assert _fails(pins_loop.test_m1_is_plain_sgd, 0.0)


def test_wrong_sign_in_a_layer_gradient_is_caught(monkeypatch):
    real = orc.loss_and_grad

    def flipped(spec, x, X, y):
        loss, g = real(spec, x, X, y)
        g = g.copy()
        n0 = spec.dims[1] * spec.dims[0]
        g[:n0] = -g[:n0]                       # first-layer weight gradient with the wrong sign
        return loss, g

    monkeypatch.setattr(orc, "loss_and_grad", flipped)
    assert _fails(pins_grad.test_gradient_matches_central_differences, (5, 4, 3), orc.LOSS_SOFTMAX_CE, True)
    assert _fails(pins_grad.test_matches_torch_autograd, (12, 9, 7, 5), orc.LOSS_SOFTMAX_CE, True)


def test_momentum_mistakes_are_caught(monkeypatch):
    # dampened momentum: v = mu v + (1 - mu) g
    monkeypatch.setattr(orc, "sgd_momentum_step",
                        lambda x, v, g, lr, mu: (np.asarray(x, np.float64) - lr * (mu * np.asarray(v, np.float64) + (1 - mu) * g),
                                                 mu * np.asarray(v, np.float64) + (1 - mu) * g))
    assert _fails(pins_loop.test_m1_is_plain_sgd, 0.9)
    assert _fails(pins_loop.test_tau1_is_synchronous_sgd_on_the_m_fold_batch, 0.9)


def test_learning_rate_inside_the_buffer_is_caught_only_by_a_changing_rate(monkeypatch):
    # v = mu v + lr g; x -= v is identical at constant lr: the pins cannot (and need not) tell them apart
    monkeypatch.setattr(orc, "sgd_momentum_step",
                        lambda x, v, g, lr, mu: (np.asarray(x, np.float64) - (mu * np.asarray(v, np.float64) * lr + lr * g),
                                                 mu * np.asarray(v, np.float64) + g))
    pins_loop.test_m1_is_plain_sgd(0.9)


def test_averaging_mistakes_are_caught(monkeypatch):
    def wrong_divisor(X):
        s = X[0].copy()
        for j in range(1, X.shape[0]):
            s = s + X[j]
        X[:] = (s / np.float32(max(1, X.shape[0] - 1)))[None, :]
    monkeypatch.setattr(orc, "average_replicas", wrong_divisor)
    assert _fails(pins_avg.test_brute_force_scalar_fp32_chain, 4)
    assert _fails(pins_avg.test_within_rounding_bound_of_exact_rational_mean, 4)
    assert _fails(pins_loop.test_tau1_is_synchronous_sgd_on_the_m_fold_batch, 0.0)

    def reversed_order(X):
        s = X[-1].copy()
        for j in range(X.shape[0] - 2, -1, -1):
            s = s + X[j]
        X[:] = (s / np.float32(X.shape[0]))[None, :]
    monkeypatch.setattr(orc, "average_replicas", reversed_order)
    assert _fails(pins_avg.test_order_matters_and_is_index_order)

    def double_precision_sum(X):
        X[:] = X.astype(np.float64).mean(axis=0).astype(np.float32)[None, :]
    monkeypatch.setattr(orc, "average_replicas", double_precision_sum)
    assert _fails(pins_avg.test_order_matters_and_is_index_order)

    def forgets_last_replica(X):
        s = X[0].copy()
        for j in range(1, X.shape[0] - 1):
            s = s + X[j]
        X[:] = (s / np.float32(X.shape[0]))[None, :]
    monkeypatch.setattr(orc, "average_replicas", forgets_last_replica)
    assert _fails(pins_avg.test_within_rounding_bound_of_exact_rational_mean, 8)


def test_averaging_before_the_update_is_caught(monkeypatch):
    # a loop that averages every tau steps but one step early / late changes the averaging points
    real = orc.run_pasgd

    def off_by_one(spec, x1, X, y, offs, batch, lr, mu, tau, **kw):
        return real(spec, x1, X, y, offs, batch, lr, mu, tau + 1, **kw)
    monkeypatch.setattr(orc, "run_pasgd", off_by_one)
    assert _fails(pins_loop.test_replicas_identical_after_every_average_and_differ_inside)
    assert _fails(pins_loop.test_tau1_is_synchronous_sgd_on_the_m_fold_batch, 0.0)


def test_controller_mistakes_are_caught(monkeypatch):
    monkeypatch.setattr(orc, "adacomm_next_tau", lambda F_t, F_0, tau_0: max(1, math.ceil(F_t / F_0 * tau_0)))   # no sqrt
    assert _fails(pins_tau.test_hand_table)
    monkeypatch.setattr(orc, "adacomm_next_tau", lambda F_t, F_0, tau_0: max(1, int(round(math.sqrt(F_t / F_0) * tau_0))))
    assert _fails(pins_tau.test_hand_table)          # round instead of ceil
    monkeypatch.setattr(orc, "adacomm_next_tau", lambda F_t, F_0, tau_0: max(1, math.floor(math.sqrt(F_t / F_0) * tau_0)))
    assert _fails(pins_tau.test_result_is_the_smallest_integer_not_below)
    monkeypatch.setattr(orc, "adacomm_next_tau", lambda F_t, F_0, tau_0: math.ceil(math.sqrt(F_t / F_0) * tau_0))   # no clamp
    assert _fails(pins_tau.test_hand_table)


def test_refined_controller_mistakes_are_caught(monkeypatch):
    real = orc.adacomm_next_tau_refined

    def cube_power(F_t, F_0, tau_0, tau_prev, gamma=0.5, slack=0, lr_0=1.0, lr_l=1.0, lr_changed=False):
        # the (lr_0/lr_l)^{3/2} form that Section 4.3.2 reports as diverging
        return real(F_t * (lr_0 / lr_l) ** 2, F_0, tau_0, tau_prev, gamma, slack, lr_0, lr_l, lr_changed)
    monkeypatch.setattr(orc, "adacomm_next_tau_refined", cube_power)
    assert _fails(pins_tau.test_refined_hand_table)
    assert _fails(pins_tau.test_refined_rule_properties)

    def not_strict(F_t, F_0, tau_0, tau_prev, gamma=0.5, slack=0, lr_0=1.0, lr_l=1.0, lr_changed=False):
        c = orc.adacomm_next_tau(F_t * lr_0 / lr_l, F_0, tau_0)
        return c if (lr_changed or c + slack <= tau_prev) else max(1, math.ceil(gamma * tau_prev))   # <= instead of <
    monkeypatch.setattr(orc, "adacomm_next_tau_refined", not_strict)
    assert _fails(pins_tau.test_refined_hand_table)

    def floor_gamma(F_t, F_0, tau_0, tau_prev, gamma=0.5, slack=0, lr_0=1.0, lr_l=1.0, lr_changed=False):
        c = orc.adacomm_next_tau(F_t * lr_0 / lr_l, F_0, tau_0)
        return c if (lr_changed or c + slack < tau_prev) else max(1, math.floor(gamma * tau_prev))
    monkeypatch.setattr(orc, "adacomm_next_tau_refined", floor_gamma)
    assert _fails(pins_tau.test_refined_hand_table)


def _mutated_run_pasgd(old: str, new: str):
    """The oracle's loop with one piece of its source replaced (a mistake planted on the CPU).  The mutant is
    compiled with the oracle module's own globals, so it sees the same (possibly monkeypatched) helpers."""
    import inspect
    src = inspect.getsource(orc.run_pasgd)
    assert src.count(old) == 1, old
    src = src.replace(old, new).replace("def run_pasgd(", "def _mutant_run_pasgd(", 1)
    exec(compile(src, "<mutated run_pasgd>", "exec"), vars(orc))
    return vars(orc).pop("_mutant_run_pasgd")


@pytest.mark.parametrize("old,new", [
    ("pending[0] <= k and cur_tau == 1", "pending[0] <= k"),                 # decay applied while the period is above 1
    ("pending[0] <= k and cur_tau == 1", "pending[0] < k and cur_tau == 1"),  # a decay due exactly now is missed
    ("if pending and pending[0] <= k and cur_tau == 1:", "while pending and pending[0] <= k and cur_tau == 1:"),  # all due decays at once
    ("refined.get(\"slack\", 0), lr_0, lr, changed)", "refined.get(\"slack\", 0), lr_0, lr, False)"),   # no growth after a decay
    ("adacomm_next_tau_refined(F_t, F_0, tau_0, cur_tau,", "adacomm_next_tau_refined(F_t, F_0, tau_0, tau_0,"),   # compares with tau_0, not the period in force
])
def test_decay_scheduling_mistakes_are_caught(monkeypatch, old, new):
    pins_tau.check_deferred_decay_trace(monkeypatch)          # passes on the oracle as it stands
    monkeypatch.setattr(orc, "run_pasgd", _mutated_run_pasgd(old, new))
    with pytest.raises(AssertionError):                       # the pin itself must object, not a crash
        pins_tau.check_deferred_decay_trace(monkeypatch)


def test_grouped_averaging_mistakes_are_caught(monkeypatch):
    real = orc.average_replicas_grouped

    def device_order_reversed(X, groups):
        q = X.shape[0] // groups
        perm = np.concatenate([np.arange(g * q, (g + 1) * q) for g in range(groups - 1, -1, -1)])
        Y = np.ascontiguousarray(X[perm]); real(Y, groups); X[:] = Y[0][None, :]
    monkeypatch.setattr(orc, "average_replicas_grouped", device_order_reversed)
    assert _fails(pins_avg.test_grouped_brute_force_scalar_fp32_chain, 16, 8)

    def divides_by_group_size(X, groups):
        real(X, groups); X *= np.float32(groups)
    monkeypatch.setattr(orc, "average_replicas_grouped", divides_by_group_size)
    assert _fails(pins_avg.test_grouped_brute_force_scalar_fp32_chain, 8, 2)
    assert _fails(pins_avg.test_grouped_within_rounding_bound_of_exact_rational_mean, 8, 2)

    def ignores_the_grouping(X, groups):
        orc.average_replicas(X)
    monkeypatch.setattr(orc, "average_replicas_grouped", ignores_the_grouping)
    assert _fails(pins_avg.test_grouped_order_is_a_different_rounding_order)
