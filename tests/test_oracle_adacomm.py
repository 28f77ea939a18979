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


# ---- refinements of Section 4.3 -------------------------------------------------------------------

GOLDEN_REFINED = os.path.join(os.path.dirname(__file__), "golden", "adacomm_refined_table.txt")


def _refined_rows():
    rows = []
    with open(GOLDEN_REFINED) as f:
        for line in f:
            a = line.split("#")[0].split()
            if len(a) == 10:
                rows.append((float(a[0]), float(a[1]), int(a[2]), int(a[3]), float(a[4]), int(a[5]), float(a[6]),
                             float(a[7]), bool(int(a[8])), int(a[9])))
    return rows


def test_refined_hand_table():
    rows = _refined_rows()
    assert len(rows) >= 10
    for *args, want in rows:
        assert orc.adacomm_next_tau_refined(*args) == want, args


def test_refined_rule_properties():
    import numpy as np
    rng = np.random.default_rng(0)
    for _ in range(2000):
        F_0 = float(rng.uniform(0.1, 3)); F_t = float(rng.uniform(0, 3)); tau_0 = int(rng.integers(1, 64))
        prev = int(rng.integers(1, 64)); gamma = float(rng.choice([0.25, 0.5, 0.75, 1.0])); s = int(rng.integers(0, 4))
        t = orc.adacomm_next_tau_refined(F_t, F_0, tau_0, prev, gamma, s)
        basic = orc.adacomm_next_tau(F_t, F_0, tau_0)
        assert t >= 1
        # with equal learning rates the candidate is the basic rule's value
        if basic + s < prev:
            assert t == basic
        else:
            assert t == max(1, math.ceil(gamma * prev)) and t <= prev        # never grows without an lr change
    # a sequence of saturated decisions halves the period down to 1 and stays there
    t, seq = 20, []
    for _ in range(7):
        t = orc.adacomm_next_tau_refined(5.0, 1.0, 20, t, 0.5, 0)
        seq.append(t)
    assert seq == [10, 5, 3, 2, 1, 1, 1]
    # the lr-coupled candidate scales with sqrt(lr_0 / lr_l), not with its 3/2 power
    assert orc.adacomm_next_tau_refined(1.0, 1.0, 10, 1000, 0.5, 0, 1.0, 0.25, True) == 20
    assert orc.adacomm_next_tau_refined(1.0, 1.0, 10, 1000, 0.5, 0, 1.0, 0.0625, True) == 40


@pytest.mark.parametrize("kw", [dict(gamma=0.0), dict(gamma=1.5), dict(slack=-1), dict(lr_l=0.0), dict(tau_prev=0),
                                dict(lr_0=float("nan"))])
def test_refined_invalid_inputs(kw):
    args = dict(F_t=1.0, F_0=1.0, tau_0=20, tau_prev=20, gamma=0.5, slack=0, lr_0=0.1, lr_l=0.1)
    args.update(kw)
    with pytest.raises(ValueError):
        orc.adacomm_next_tau_refined(**args)


# ---- scheduling of learning-rate decays inside the loop (Section 4.3.2, last paragraph) ------------------------

GOLDEN_DECAY = os.path.join(os.path.dirname(__file__), "golden", "adacomm_deferred_decay_trace.txt")


def _decay_trace():
    rows, periods = [], None
    with open(GOLDEN_DECAY) as f:
        for line in f:
            if line.startswith("# periods"):
                periods = [int(v) for v in line.split()[2:]]
            a = line.split("#")[0].split()
            if len(a) == 4:
                rows.append((int(a[0]), float(a[1]), float(a[2]), int(a[3])))
    return rows, periods


def run_scripted_refined_loop(monkeypatch):
    """run_pasgd(refined=...) on a tiny model with the probe losses scripted by the golden trace: the training
    steps run as usual, only the loss the controller sees is replaced, so the schedule is a function of the
    scripted F_t alone.  Returns the oracle's result and the trace."""
    import numpy as np
    from paper_1810_08313_b200 import workloads as wl
    rows, periods = _decay_trace()
    script = [1.0] + [F for _, F, _, _ in rows]          # F_0 first, then one loss per decision
    calls = []

    def scripted_loss(spec, x, X, y):
        calls.append(len(calls))
        return script[len(calls) - 1]

    monkeypatch.setattr(orc, "batch_loss", scripted_loss)
    spec = orc.ModelSpec((3, 1), orc.LOSS_MSE_HALF, False)
    X = wl.gaussian_rows(5, 64, 3)
    y = np.random.default_rng(5).standard_normal(64).astype(np.float32)
    K, m, B = 31, 2, 4
    offs = wl.batch_row_offsets(5, K, m, 64, B)
    lr0 = float(np.float32(0.1))
    res = orc.run_pasgd(spec, np.zeros(3, np.float32), X, y, offs, B, lr0, 0.0, 4, adacomm_interval=4, probe_rows=8,
                        refined={"gamma": 0.5, "slack": 0, "decay_at": [6, 7, 28], "decay_factor": 0.1})
    assert len(calls) == len(script)                      # every scripted loss was consumed, none was missing
    return res, rows, periods


def check_deferred_decay_trace(monkeypatch):
    res, rows, periods = run_scripted_refined_loop(monkeypatch)
    assert [k for k, _, _ in res.F_trace] == [k for k, _, _, _ in rows]
    assert [t for _, _, t in res.F_trace] == [t for _, _, _, t in rows]
    assert res.taus == periods
    # the learning rate after each decision (the oracle logs the decays it applied)
    lr, applied = 0.1, dict(res.lr_trace)
    for k, _, lr_after, _ in rows:
        lr = applied.get(k, lr)
        assert abs(lr - lr_after) <= 1e-6 * lr_after, (k, lr, lr_after)
    assert sorted(applied) == [12, 24, 28]


def test_deferred_decay_hand_trace(monkeypatch):
    check_deferred_decay_trace(monkeypatch)
