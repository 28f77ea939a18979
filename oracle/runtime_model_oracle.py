"""CPU oracle of the runtime / delay model of local-update SGD (arXiv 1810.08313, Sections 2-4).

TEST INFRASTRUCTURE: only tests/, __graft_entry__.smoke() and bench.py's cpu_baseline leg may import this
module.  It shares no code with the CUDA library; the library's host functions of the same names are
written separately (csrc/runtime_model.cu).

What is here, each from its passage:
  delay()                 D = D_0 * s(m), the delay model of Section 2 ("Local Computation Times and
                          Communication Delay"), with the scalings the text names (constant, log2 m, the
                          2 log2 m reduction tree, linear).
  t_sync(), t_pavg()      runtime per iteration of fully synchronous SGD and of PASGD, Section 3.1:
                          T_sync = max_i Y_i + D ;  T_P-Avg = max_i mean_k Y_{i,k} + D / tau.
  speedup_constant()      (1 + alpha) / (1 + alpha / tau), alpha = D / Y, Section 3.2.
  error_bound()           the bound of Theorem 1 at wall-clock time T.
  tau_star()              Theorem 2: the period that minimises that bound.
  philox4x32_10()         the counter-based generator of Salmon et al. (SC'11), from its published
                          definition; it is the one source of randomness of simulate().
  simulate()              Monte-Carlo means of T_sync and T_P-Avg for exponential (or constant) Y.

Pins (tests/test_oracle_runtime_model.py): the published known-answer vector of Philox4x32-10, E[Y_{m:m}] =
y * H_m for exponential Y (Section 3.2), Var[mean of tau exponentials] = y^2 / tau, the constant-Y speed-up
closed form reproduced by simulate(), tau_star against a brute-force minimiser of error_bound(), and the
monotonicity statements of Section 3.2.
"""
from __future__ import annotations

import math
from typing import Tuple

import numpy as np

SCALING_CONSTANT = 0      # s(m) = 1
SCALING_LOG2 = 1          # s(m) = log2 m
SCALING_TREE = 2          # s(m) = 2 log2 m   (reduction tree, Section 2)
SCALING_LINEAR = 3        # s(m) = m


def delay(D0: float, m: int, scaling: int) -> float:
    """D = D_0 * s(m)  (Section 2, delay model)."""
    if m < 1:
        raise ValueError("m >= 1")
    if scaling == SCALING_CONSTANT:
        s = 1.0
    elif scaling == SCALING_LOG2:
        s = math.log2(m)
    elif scaling == SCALING_TREE:
        s = 2.0 * math.log2(m)
    elif scaling == SCALING_LINEAR:
        s = float(m)
    else:
        raise ValueError("unknown scaling")
    return D0 * s


def t_sync(Y: np.ndarray, D: float) -> float:
    """One iteration of fully synchronous SGD: Y[i] is worker i's compute time.  T = max_i Y_i + D."""
    return float(np.max(np.asarray(Y, dtype=np.float64))) + D


def t_pavg(Y: np.ndarray, D: float) -> float:
    """One period of PASGD, per iteration: Y[k][i] is worker i's time at local step k (tau = Y.shape[0]).
    T = max_i (sum_k Y[k][i] / tau) + D / tau."""
    Y = np.asarray(Y, dtype=np.float64)
    tau = Y.shape[0]
    ybar = np.zeros(Y.shape[1], dtype=np.float64)
    for k in range(tau):
        ybar = ybar + Y[k]
    ybar = ybar / tau
    return float(np.max(ybar)) + D / tau


def speedup_constant(alpha: float, tau: int) -> float:
    """E[T_sync] / E[T_P-Avg] for constant Y and D, alpha = D / Y  (Section 3.2)."""
    return (1.0 + alpha) / (1.0 + alpha / tau)


def error_bound(T: float, F1: float, Finf: float, lr: float, L: float, sigma2: float, m: int, tau: int,
                Y: float, D: float) -> float:
    """Theorem 1: 2 (F(x_1) - F_inf) / (lr T) * (Y + D / tau) + lr L sigma^2 / m + lr^2 L^2 sigma^2 (tau - 1)."""
    return 2.0 * (F1 - Finf) / (lr * T) * (Y + D / tau) + lr * L * sigma2 / m + lr * lr * L * L * sigma2 * (tau - 1)


def tau_star(F1: float, Finf: float, D: float, lr: float, L: float, sigma2: float, T: float) -> float:
    """Theorem 2: tau* = sqrt( 2 (F(x_1) - F_inf) D / (lr^3 L^2 sigma^2 T) )."""
    return math.sqrt(2.0 * (F1 - Finf) * D / (lr ** 3 * L * L * sigma2 * T))


# ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3") ----------
_M0, _M1 = 0xD2511F53, 0xCD9E8D57          # round multipliers
_W0, _W1 = 0x9E3779B9, 0xBB67AE85          # key increments (golden ratio, sqrt(3) - 1)
_MASK = 0xFFFFFFFF


def philox4x32_10(counter: Tuple[int, int, int, int], key: Tuple[int, int]) -> Tuple[int, int, int, int]:
    c0, c1, c2, c3 = counter
    k0, k1 = key
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = (p0 >> 32) & _MASK, p0 & _MASK
        hi1, lo1 = (p1 >> 32) & _MASK, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK, lo1, (hi0 ^ c3 ^ k1) & _MASK, lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def uniform_open(x: int) -> float:
    """32 random bits -> a double in (0, 1): (x + 0.5) / 2^32."""
    return (x + 0.5) / 4294967296.0


def compute_time(seed: int, period: int, k: int, worker: int, y_mean: float, exponential: bool) -> float:
    """Y_{i,k} of the given period: exponential with mean y (inverse CDF of one Philox output) or the constant y.
    Counter = (period low, period high, k, worker), key = (seed low, seed high), first output word."""
    if not exponential:
        return y_mean
    x = philox4x32_10((period & _MASK, (period >> 32) & _MASK, k & _MASK, worker & _MASK),
                      (seed & _MASK, (seed >> 32) & _MASK))[0]
    return -y_mean * math.log(uniform_open(x))


def simulate(m: int, tau: int, n_periods: int, y_mean: float, D: float, seed: int,
             exponential: bool = True) -> Tuple[float, float]:
    """Means over the run of the per-iteration runtime of fully synchronous SGD (every local step followed by
    a broadcast) and of PASGD with period tau, both on the same draws Y_{i,k}  (Section 3.1)."""
    sum_sync = 0.0
    sum_pavg = 0.0
    for p in range(n_periods):
        Y = np.empty((tau, m), dtype=np.float64)
        for k in range(tau):
            for i in range(m):
                Y[k, i] = compute_time(seed, p, k, i, y_mean, exponential)
        for k in range(tau):
            sum_sync += t_sync(Y[k], D)
        sum_pavg += t_pavg(Y, D)
    return sum_sync / (n_periods * tau), sum_pavg / n_periods
