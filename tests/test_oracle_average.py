"""Pins for the oracle's averaging step (Section 2, PASGD update rule, case
k mod tau = 0; operator J = 1 1^T / m of the proof's notation)."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import localsgd_oracle as orc


def test_m1_is_identity():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((1, 37)).astype(np.float32)
    Y = X.copy()
    orc.average_replicas(Y)
    assert np.array_equal(X.view(np.uint32), Y.view(np.uint32))


def test_equal_replicas_m2_unchanged_and_larger_m_within_rounding():
    # x + x is exact, so m = 2 reproduces equal replicas bit for bit.  For m >= 3 the
    # sequential fp32 sum x, 2x, fl(3x), ... rounds, so the mean of equal replicas may
    # move by a few ulp: averaging is NOT idempotent in fp32, only replica equality holds.
    rng = np.random.default_rng(1)
    row = rng.standard_normal(101).astype(np.float32)
    X = np.repeat(row[None], 2, axis=0).copy()
    orc.average_replicas(X)
    assert np.array_equal(X[0].view(np.uint32), row.view(np.uint32))
    for m in (4, 8, 16, 32):
        X = np.repeat(row[None], m, axis=0).copy()
        orc.average_replicas(X)
        assert np.max(np.abs(X[0] - row) / np.abs(row)) < m * 2.0 ** -24
        assert all(np.array_equal(X[0].view(np.uint32), X[j].view(np.uint32)) for j in range(m))


@pytest.mark.parametrize("m", [2, 3, 4, 7, 16])
def test_brute_force_scalar_fp32_chain(m):
    # the definition, one scalar at a time with numpy float32 scalars
    rng = np.random.default_rng(2)
    X = (rng.random((m, 23), dtype=np.float32) * 2 - 1).astype(np.float32)
    want = np.empty(23, dtype=np.float32)
    for p in range(23):
        s = np.float32(X[0, p])
        for j in range(1, m):
            s = np.float32(s + np.float32(X[j, p]))
        want[p] = np.float32(s / np.float32(m))
    orc.average_replicas(X)
    for j in range(m):
        assert np.array_equal(X[j].view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("m", [3, 4, 8, 16])
def test_within_rounding_bound_of_exact_rational_mean(m):
    rng = np.random.default_rng(4)
    X = (rng.random((m, 50), dtype=np.float32) * 2 - 1).astype(np.float32)
    exact = [sum(Fraction(float(X[j, p])) for j in range(m)) / m for p in range(50)]
    orc.average_replicas(X)
    u = 2.0 ** -24
    for p in range(50):
        # m-1 adds of magnitudes <= m, one division: |err| <= m * m * u  (loose, but a wrong
        # divisor, a dropped replica or a doubled one is far outside it)
        assert abs(Fraction(float(X[0, p])) - exact[p]) <= m * m * u


def test_all_replicas_bitwise_identical_afterwards():
    rng = np.random.default_rng(5)
    X = rng.standard_normal((5, 1000)).astype(np.float32)
    orc.average_replicas(X)
    for j in range(1, 5):
        assert np.array_equal(X[0].view(np.uint32), X[j].view(np.uint32))


def test_order_matters_and_is_index_order():
    # 1e8 + 1 - 1e8: (x0 + x1) + x2 in fp32 loses the 1; the other order keeps it
    X = np.array([[1e8], [1.0], [-1e8]], dtype=np.float32)
    orc.average_replicas(X)
    assert X[0, 0] == np.float32(0.0)
    X = np.array([[1e8], [-1e8], [1.0]], dtype=np.float32)
    orc.average_replicas(X)
    assert X[0, 0] == np.float32(1.0) / np.float32(3.0)


def test_rejects_other_dtypes():
    with pytest.raises(TypeError):
        orc.average_replicas(np.zeros((2, 3)))
