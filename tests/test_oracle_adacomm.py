"""Pins for the oracle's AdaComm rule (Section 4.2, basic update rule)."""
import math
import os

import pytest

from oracle import localsgd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "adacomm_table.txt")


def _rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                a = line.split()
                rows.append((float(a[0]), float(a[1]), int(a[2]), int(a[3])))
    return rows


def test_hand_table():
    rows = _rows()
    assert len(rows) >= 10
    for F_t, F_0, tau_0, want in rows:
        assert orc.adacomm_next_tau(F_t, F_0, tau_0) == want, (F_t, F_0, tau_0)


def test_monotone_in_loss_and_scale_free():
    prev = 0
    for i in range(0, 400):
        F_t = i / 100.0
        t = orc.adacomm_next_tau(F_t, 1.0, 20)
        assert t >= prev and t >= 1
        prev = t
        # only the ratio matters: scaling both losses by a power of two is exact
        assert orc.adacomm_next_tau(F_t * 8.0, 8.0, 20) == t


def test_result_is_the_smallest_integer_not_below():
    # ceil property checked with exact integer arithmetic: n-1 < sqrt(r)*tau0 <= n
    from fractions import Fraction
    for num, den, tau_0 in [(1, 3, 20), (2, 7, 13), (5, 9, 50), (7, 8, 3), (1, 1000, 20), (3, 2, 11)]:
        n = orc.adacomm_next_tau(float(num), float(den), tau_0)
        r = Fraction(num, den) * tau_0 * tau_0      # (sqrt(r) tau0)^2, exact
        assert r <= n * n
        if n > 1:
            assert r > (n - 1) * (n - 1)


@pytest.mark.parametrize("args", [(1.0, 0.0, 20), (1.0, -1.0, 20), (-0.1, 1.0, 20), (float("nan"), 1.0, 20),
                                  (1.0, float("inf"), 20), (float("inf"), 1.0, 20), (1.0, 1.0, 0)])
def test_invalid_inputs_raise(args):
    with pytest.raises(ValueError):
        orc.adacomm_next_tau(*args)


def test_schedule_from_trace():
    F = [2.0, 1.0, 0.5, 0.125, 0.02]
    assert orc.tau_schedule_from_trace(2.0, 20, F) == [20, 15, 10, 5, 2]
