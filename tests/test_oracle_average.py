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


# ---- grouped order: replicas spread over several devices (Section 2; one partial sum per device) -------------

@pytest.mark.parametrize("m,groups", [(4, 2), (8, 2), (8, 4), (16, 4), (6, 3), (16, 8)])
def test_grouped_brute_force_scalar_fp32_chain(m, groups):
    # the definition one scalar at a time: sequential partial per device, then the partials in device order
    rng = np.random.default_rng(12)
    X = (rng.random((m, 19), dtype=np.float32) * 2 - 1).astype(np.float32)
    q = m // groups
    want = np.empty(19, dtype=np.float32)
    for p in range(19):
        total = None
        for g in range(groups):
            part = np.float32(X[g * q, p])
            for j in range(1, q):
                part = np.float32(part + np.float32(X[g * q + j, p]))
            total = part if total is None else np.float32(total + part)
        want[p] = np.float32(total / np.float32(m))
    orc.average_replicas_grouped(X, groups)
    for j in range(m):
        assert np.array_equal(X[j].view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("m", [1, 2, 4, 8, 16])
def test_one_group_and_m_groups_are_the_sequential_order(m):
    # one device: nothing is regrouped; one replica per device: the partials ARE the replicas, summed in index order
    rng = np.random.default_rng(13)
    X = rng.standard_normal((m, 300)).astype(np.float32)
    want = X.copy(); orc.average_replicas(want)
    for groups in (1, m):
        Y = X.copy(); orc.average_replicas_grouped(Y, groups)
        assert np.array_equal(Y.view(np.uint32), want.view(np.uint32))


def test_grouped_order_is_a_different_rounding_order():
    # (1e8 + 1) + (-1e8 + 1): the sequential chain loses both ones one at a time,
    # the grouped order loses each inside its pair too, but (1e8 + -1e8) grouped the other way keeps them
    X = np.array([[1e8], [-1e8], [1.0], [1.0]], dtype=np.float32)
    Y = X.copy(); orc.average_replicas(Y)                      # ((1e8 - 1e8) + 1) + 1 = 2 -> 0.5
    assert Y[0, 0] == np.float32(0.5)
    Z = X.copy(); orc.average_replicas_grouped(Z, 2)           # (1e8 - 1e8) + (1 + 1) = 2 -> 0.5
    assert Z[0, 0] == np.float32(0.5)
    X = np.array([[1e8], [1.0], [-1e8], [1.0]], dtype=np.float32)
    Y = X.copy(); orc.average_replicas(Y)                      # ((1e8 + 1) - 1e8) + 1 = 1 -> 0.25
    assert Y[0, 0] == np.float32(0.25)
    Z = X.copy(); orc.average_replicas_grouped(Z, 2)           # (1e8 + 1) + (-1e8 + 1) = 1e8 - 1e8 = 0 -> 0
    assert Z[0, 0] == np.float32(0.0)
    # on ordinary data some element differs in the last bit, and every element stays within the rounding bound
    rng = np.random.default_rng(14)
    X = rng.standard_normal((16, 4000)).astype(np.float32)
    Y = X.copy(); orc.average_replicas(Y)
    Z = X.copy(); orc.average_replicas_grouped(Z, 4)
    assert not np.array_equal(Y.view(np.uint32), Z.view(np.uint32))
    assert np.max(np.abs(Y[0] - Z[0])) <= 16 * 16 * 2.0 ** -24


@pytest.mark.parametrize("m,groups", [(8, 2), (16, 4)])
def test_grouped_within_rounding_bound_of_exact_rational_mean(m, groups):
    rng = np.random.default_rng(15)
    X = (rng.random((m, 40), dtype=np.float32) * 2 - 1).astype(np.float32)
    exact = [sum(Fraction(float(X[j, p])) for j in range(m)) / m for p in range(40)]
    orc.average_replicas_grouped(X, groups)
    for p in range(40):
        assert abs(Fraction(float(X[0, p])) - exact[p]) <= m * m * 2.0 ** -24
    assert all(np.array_equal(X[0].view(np.uint32), X[j].view(np.uint32)) for j in range(m))


def test_grouped_rejects_uneven_groups_and_other_dtypes():
    with pytest.raises(ValueError):
        orc.average_replicas_grouped(np.zeros((6, 3), np.float32), 4)
    with pytest.raises(TypeError):
        orc.average_replicas_grouped(np.zeros((4, 3)), 2)
