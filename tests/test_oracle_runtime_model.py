"""Pins of the runtime-model oracle (Sections 2-4: delay model, runtime per iteration, speed-up, Theorems 1-2)."""
import math

import numpy as np

from oracle import runtime_model_oracle as rm


def test_philox_known_answer_vector():
    # published known-answer test of Philox4x32-10 (Random123 distribution, kat_vectors): all-zero counter and key
    assert rm.philox4x32_10((0, 0, 0, 0), (0, 0)) == (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)
    # a bijection of the counter for a fixed key: distinct counters give distinct blocks
    seen = {rm.philox4x32_10((c, 0, 0, 0), (7, 9)) for c in range(256)}
    assert len(seen) == 256
    # every output bit is used: mean of 4096 words close to 2^31
    words = [w for c in range(1024) for w in rm.philox4x32_10((c, 1, 2, 3), (4, 5))]
    assert abs(np.mean(words) / 2 ** 31 - 1.0) < 0.03


def test_delay_model_scalings():
    assert rm.delay(0.5, 16, rm.SCALING_CONSTANT) == 0.5
    assert rm.delay(0.5, 16, rm.SCALING_LOG2) == 2.0
    assert rm.delay(0.5, 16, rm.SCALING_TREE) == 4.0         # 2 log2 m
    assert rm.delay(0.5, 16, rm.SCALING_LINEAR) == 8.0
    assert rm.delay(3.0, 1, rm.SCALING_TREE) == 0.0


def test_runtime_definitions_on_a_hand_example():
    # 2 workers, 3 local steps; written out by hand
    Y = np.array([[1.0, 4.0], [2.0, 1.0], [3.0, 1.0]])
    assert rm.t_sync(Y[0], 0.5) == 4.5
    # worker means 2.0 and 2.0 -> max 2, + D / tau
    assert rm.t_pavg(Y, 0.6) == 2.0 + 0.2
    # tau = 1 reduces PASGD to fully synchronous SGD
    assert rm.t_pavg(Y[:1], 0.5) == rm.t_sync(Y[0], 0.5)


def test_speedup_closed_form_and_constant_simulation():
    assert abs(rm.speedup_constant(0.9, 100) - 1.9 / 1.009) < 1e-15
    assert rm.speedup_constant(0.9, 1) == 1.0
    # almost 2x at alpha = 0.9 for a large period, never more than 1 + alpha
    assert 1.85 < rm.speedup_constant(0.9, 50) < 1.9
    for tau in (1, 2, 10):
        s, p = rm.simulate(4, tau, 5, 2.0, 1.8, seed=3, exponential=False)
        assert abs(s / p - rm.speedup_constant(0.9, tau)) < 1e-12


def test_expected_maximum_of_exponentials_is_the_harmonic_sum():
    """Section 3.2: E[Y_{m:m}] = y * sum_{i<=m} 1/i for exponential Y."""
    m, y, n = 16, 1.0, 4000
    s, _ = rm.simulate(m, 1, n, y, 0.0, seed=11)
    H = sum(1.0 / i for i in range(1, m + 1))
    # Var[Y_{m:m}] = y^2 sum 1/i^2 < 1.65: three standard errors
    assert abs(s - y * H) < 3 * math.sqrt(1.65 / n)


def test_local_updates_mitigate_stragglers():
    """Section 3.2: the mean of tau exponentials has variance y^2 / tau, so E[max] shrinks with tau, towards y."""
    y, tau = 2.0, 8
    means = []
    for p in range(3000):
        means.append(np.mean([rm.compute_time(5, p, k, 0, y, True) for k in range(tau)]))
    assert abs(np.mean(means) - y) < 0.05
    assert abs(np.var(means) / (y * y / tau) - 1.0) < 0.12
    prev = None
    for t in (1, 4, 16):
        _, p = rm.simulate(16, t, 600 // t + 50, 1.0, 0.0, seed=2)
        assert p > 1.0
        if prev is not None:
            assert p < prev
        prev = p


def test_tau_star_minimises_the_error_bound():
    """Theorem 2 against a brute-force minimiser of Theorem 1's bound (figure constants of Section 3.3)."""
    F1, Finf, lr, L, s2, m, Y, D = 1.0, 0.0, 0.08, 1.0, 1.0, 16, 1.0, 1.0
    for T in (50.0, 500.0, 5000.0):
        ts = rm.tau_star(F1, Finf, D, lr, L, s2, T)
        grid = np.linspace(max(ts / 4, 1e-3), ts * 4, 20001)
        vals = [2 * (F1 - Finf) / (lr * T) * (Y + D / t) + lr * L * s2 / m + lr * lr * L * L * s2 * (t - 1) for t in grid]
        assert abs(grid[int(np.argmin(vals))] - ts) / ts < 1e-3
    # the bound itself at integer periods, and its two regimes: early on a large period wins, late a small one
    early = [rm.error_bound(20.0, F1, Finf, lr, L, s2, m, t, Y, D) for t in (1, 10)]
    late = [rm.error_bound(20000.0, F1, Finf, lr, L, s2, m, t, Y, D) for t in (1, 10)]
    assert early[1] < early[0] and late[0] < late[1]
    # the period sequence of Section 4.1 decreases with the objective value: tau_l / tau_0 = sqrt(F_l / F_0)
    t0 = rm.tau_star(1.0, 0.0, D, lr, L, s2, 60.0)
    tl = rm.tau_star(0.25, 0.0, D, lr, L, s2, 60.0)
    assert abs(tl / t0 - 0.5) < 1e-12
