"""Whole PASGD runs on the GPU vs the oracle (Section 2 PASGD update rule,
Section 4.2 basic update rule)."""
import numpy as np
import pytest

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import workloads as wl
from tests.helpers import f32, max_rel_err_per_tensor, small_problem, to_device

pytestmark = pytest.mark.gpu


def _bitwise_equal_replicas(eng):
    p, v = eng.state_view()
    return bool((p[0:1] == p).all()) and bool((v[0:1] == v).all())


def test_softmax_regression_config_every_step():
    """784-dim softmax regression, m = 4, B = 32, tau = 10, 100 iterations, lr 0.05, zero start:
    free-running, parameters compared with the oracle after every period, losses at every step."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    w = wl.WORKLOADS["c1_softmax"]
    X, y = wl.make_dataset(w, n_rows=8192)
    spec = orc.ModelSpec(w.dims, w.loss, w.has_bias)
    x1 = wl.initial_point(w)
    offs = wl.batch_row_offsets(w.seed, w.n_iters, w.m, X.shape[0], w.batch)
    snaps = {}

    def hook(k, xs, vs, averaged):
        if averaged:
            snaps[k] = xs.copy()

    ref = orc.run_pasgd(spec, x1, X, y, offs, w.batch, f32(w.lr), 0.0, 10, state_hook=hook)
    xd, yd = to_device(X, y)
    eng = LocalSGD(w.m, w.dims, w.loss, w.has_bias, "fp32", lr=w.lr, momentum=0.0, batch=w.batch)
    eng.bind_dataset(xd, yd)
    eng.set_params(x1)
    loss_dev = torch.zeros((w.n_iters, w.m), dtype=torch.float32, device="cuda")
    for k0 in range(0, w.n_iters, 10):
        eng.local_steps(10, offs[k0:k0 + 10], loss_dev[k0:k0 + 10])
        eng.average()
        eng.sync()
        assert _bitwise_equal_replicas(eng)
        gx, _ = eng.get_all()
        for i in range(w.m):
            assert max_rel_err_per_tensor(gx[i], snaps[k0 + 10][i], w.dims, w.has_bias) <= 1e-5
    got = loss_dev.cpu().numpy()
    assert np.max(np.abs(got - ref.loss) / ref.loss) <= 1e-5
    assert got[-1].mean() < got[0].mean()          # it learns
    eng.close()


@pytest.mark.parametrize("mode", ["average", "keep", "reset"])
def test_native_run_matches_oracle_over_three_periods(mode):
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, tau, K = (96, 64, 48, 10), 4, 32, 5, 15
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 21)
    offs = wl.batch_row_offsets(2, K, m, 1024, B)
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(0.9), tau, momentum_mode=mode)
    xd, yd = to_device(X, y)
    eng = LocalSGD(m, dims, lr=0.05, momentum=0.9, batch=B, momentum_mode=mode)
    eng.bind_dataset(xd, yd)
    eng.set_params(x1)
    loss_dev = torch.zeros((K, m), dtype=torch.float32, device="cuda")
    out = eng.run(K, tau, offs, loss_out=loss_dev)
    eng.sync()
    assert out["taus"] == ref.taus == [5, 5, 5]
    gx, gv = eng.get_all()
    for i in range(m):
        assert max_rel_err_per_tensor(gx[i], ref.params[i], dims, True) <= 1e-4     # 15 free-running steps
        if mode == "reset":
            assert np.all(gv[i] == 0)
        else:
            assert max_rel_err_per_tensor(gv[i], ref.momentum[i], dims, True) <= 1e-3
    got = loss_dev.cpu().numpy()
    assert np.max(np.abs(got - ref.loss) / ref.loss) <= 1e-4
    p, v = eng.state_view()
    assert bool((p[0:1] == p).all())
    assert bool((v[0:1] == v).all()) == (mode != "keep")
    eng.close()


@pytest.mark.parametrize("gemm,mu", [("fp32", 0.9), ("fp32", 0.0), ("bf16", 0.9)])
def test_block_momentum_run_matches_oracle(gemm, mu):
    """Section 5.3: global momentum buffer applied at every averaging step, local buffers restart.  The
    averaging step itself is checked to the bit from injected state; the free run within tolerance."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, tau, K, beta = (96, 64, 48, 10), 4, 32, 5, 15, 0.3
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 21)
    offs = wl.batch_row_offsets(2, K, m, 1024, B)
    eng = LocalSGD(m, dims, lr=0.05, momentum=mu, batch=B, momentum_mode="block", block_momentum=beta,
                   gemm_dtype=gemm)
    xd, yd = to_device(X, y, bf16=(gemm == "bf16"))
    eng.bind_dataset(xd, yd)
    # (1) one averaging step from injected state, bit-exact
    P = spec.n_params
    st = wl.uniform_flat(5, m + 2, P)
    xs, anchor, u = st[:m].copy(), st[m].copy(), st[m + 1].copy()
    eng.set_params(x1)
    for i in range(m):
        eng.set_state(i, xs[i], xs[i])
    eng.set_block_state(anchor, u)
    eng.average()
    eng.sync()
    orc.block_momentum_average(xs, anchor, u, f32(0.05), f32(beta))
    gx, gv = eng.get_all()
    ga, gu = eng.get_block_state()
    for i in range(m):
        assert np.array_equal(gx[i].view(np.uint32), xs[i].view(np.uint32))
        if mu != 0.0:
            assert np.all(gv[i] == 0)
    assert np.array_equal(ga.view(np.uint32), anchor.view(np.uint32))
    assert np.array_equal(gu.view(np.uint32), u.view(np.uint32))
    if gemm == "bf16":
        eng.close()
        return
    # (2) free run from x_1
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(mu), tau, momentum_mode="block", block_beta=f32(beta))
    eng.set_params(x1)
    loss_dev = torch.zeros((K, m), dtype=torch.float32, device="cuda")
    out = eng.run(K, tau, offs, loss_out=loss_dev)
    eng.sync()
    assert out["taus"] == ref.taus
    gx, gv = eng.get_all()
    ga, gu = eng.get_block_state()
    for i in range(m):
        assert max_rel_err_per_tensor(gx[i], ref.params[i], dims, True) <= 1e-4
    assert max_rel_err_per_tensor(ga, ref.params[0], dims, True) <= 1e-4
    assert max_rel_err_per_tensor(gu, ref.block_u, dims, True) <= 1e-3
    got = loss_dev.cpu().numpy()
    assert np.max(np.abs(got - ref.loss) / ref.loss) <= 1e-4
    p, v = eng.state_view()
    assert bool((p[0:1] == p).all())
    eng.close()


def test_block_momentum_handle_argument_checks():
    from paper_1810_08313_b200 import binding
    from paper_1810_08313_b200.binding import LocalSGD
    with pytest.raises(binding.LsError):
        LocalSGD(2, (16, 8), batch=8, momentum_mode="block", block_momentum=1.0)
    eng = LocalSGD(2, (16, 8), batch=8, momentum_mode="reset")
    with pytest.raises(binding.LsError):
        eng.get_block_state()
    eng.close()


def test_tau1_equals_large_batch_sgd_on_gpu():
    """tau = 1 with m replicas equals one replica trained on the concatenated m*B batch
    (fully synchronous SGD, Section 2 special case), both run on the GPU."""
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, K = (64, 48, 10), 4, 16, 8
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 4)
    blocks = np.random.default_rng(0).integers(0, 1024 // (m * B), K) * (m * B)
    offs_m = np.stack([blocks + i * B for i in range(m)], axis=1).astype(np.int64)   # m adjacent blocks
    xd, yd = to_device(X, y)
    a = LocalSGD(m, dims, lr=0.05, momentum=0.9, batch=B); a.bind_dataset(xd, yd); a.set_params(x1)
    a.run(K, 1, offs_m)
    b = LocalSGD(1, dims, lr=0.05, momentum=0.9, batch=m * B); b.bind_dataset(xd, yd); b.set_params(x1)
    b.run(K, 1, blocks.reshape(K, 1).astype(np.int64))
    pa, _ = a.get_state(0); pb, _ = b.get_state(0)
    assert max_rel_err_per_tensor(pa, pb, dims, True) <= 1e-5
    a.close(); b.close()


def test_m1_equals_oracle_plain_sgd():
    from paper_1810_08313_b200.binding import LocalSGD
    dims, B, K = (64, 48, 10), 16, 6
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 512, 6)
    offs = wl.batch_row_offsets(3, K, 1, 512, B)
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(0.9), 4)
    xd, yd = to_device(X, y)
    eng = LocalSGD(1, dims, lr=0.05, momentum=0.9, batch=B); eng.bind_dataset(xd, yd); eng.set_params(x1)
    eng.run(K, 4, offs)
    p, v = eng.get_state(0)
    assert max_rel_err_per_tensor(p, ref.params[0], dims, True) <= 1e-5
    eng.close()


def test_eval_loss_and_adacomm_run():
    """AdaComm run: the decisions logged by the native loop are recomputed bit-exactly by the
    oracle's rule from the logged losses; the losses themselves match the oracle's."""
    from paper_1810_08313_b200 import binding
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, K, tau0, I, probe = (96, 64, 10), 4, 32, 60, 8, 10, 256
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 2048, 33)
    offs = wl.batch_row_offsets(9, K, m, 2048, B)
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), 0.0, tau0, adacomm_interval=I, probe_rows=probe)
    xd, yd = to_device(X, y)
    eng = LocalSGD(m, dims, lr=0.05, momentum=0.0, batch=B); eng.bind_dataset(xd, yd); eng.set_params(x1)
    F0 = eng.eval_loss(0, 0, probe)
    assert abs(F0 - ref.F_0) / ref.F_0 <= 1e-5
    assert abs(eng.eval_loss(0, 512, 64) - orc.batch_loss(spec, x1, X[512:576], y[512:576])) <= 1e-5 * ref.F_0
    out = eng.run(K, tau0, offs, interval=I, probe_rows=probe)
    # bit-exact tau schedule from the GPU's own logged loss trace
    want_taus = orc.tau_schedule_from_trace(out["F_0"], tau0, [float(F) for F in out["decision_F"]])
    assert out["decision_tau"] == want_taus
    assert [binding.adacomm_next_tau(float(F), out["F_0"], tau0) for F in out["decision_F"]] == want_taus
    # and the run follows the oracle's: same decision points, losses within fp32 tolerance, same periods
    assert out["decision_k"] == [k for k, _, _ in ref.F_trace]
    for F, (_, Fr, _) in zip(out["decision_F"], ref.F_trace):
        assert abs(float(F) - Fr) / Fr <= 1e-4
    assert out["taus"] == ref.taus
    eng.close()


def test_host_batches_match_resident_dataset():
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, tau = (64, 48, 10), 3, 16, 5
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 512, 8)
    offs = wl.batch_row_offsets(4, tau, m, 512, B)
    xd, yd = to_device(X, y)
    a = LocalSGD(m, dims, lr=0.05, momentum=0.9, batch=B); a.bind_dataset(xd, yd); a.set_params(x1)
    la = torch.zeros((tau, m), device="cuda")
    a.local_steps(tau, offs, la); a.sync()
    xh = torch.empty((tau, m, B, dims[0]), dtype=torch.float32).pin_memory()
    yh = torch.empty((tau, m, B), dtype=torch.int32).pin_memory()
    for s in range(tau):
        for i in range(m):
            r0 = int(offs[s, i])
            xh[s, i] = torch.from_numpy(X[r0:r0 + B]); yh[s, i] = torch.from_numpy(y[r0:r0 + B])
    lh = torch.zeros((tau, m), dtype=torch.float32).pin_memory()
    b = LocalSGD(m, dims, lr=0.05, momentum=0.9, batch=B); b.set_params(x1)
    b.local_steps_host(tau, xh, yh, lh)
    pa, va = a.get_all(); pb, vb = b.get_all()
    assert np.array_equal(pa, pb) and np.array_equal(va, vb)
    assert np.array_equal(la.cpu().numpy(), lh.numpy())
    a.close(); b.close()


def test_least_squares_config_short():
    """Least squares 4096-dim, m = 32, B = 64, tau = 50, lr 1e-4: two periods vs the oracle."""
    from paper_1810_08313_b200.binding import LocalSGD
    w = wl.WORKLOADS["c4_lsq"]
    X, y = wl.make_dataset(w)
    spec = orc.ModelSpec(w.dims, w.loss, w.has_bias)
    K = 100
    offs = wl.batch_row_offsets(w.seed, K, w.m, w.n_rows, w.batch)
    ref = orc.run_pasgd(spec, wl.initial_point(w), X, y, offs, w.batch, f32(w.lr), 0.0, 50)
    xd, yd = to_device(X, y)
    eng = LocalSGD(w.m, w.dims, w.loss, w.has_bias, "fp32", lr=w.lr, momentum=0.0, batch=w.batch)
    eng.bind_dataset(xd, yd); eng.set_params(wl.initial_point(w))
    eng.run(K, 50, offs)
    p, _ = eng.get_state(0)
    assert max_rel_err_per_tensor(p, ref.params[0], w.dims, w.has_bias) <= 1e-5
    eng.close()


def test_refined_adacomm_run_with_deferred_lr_decay():
    """Section 4.3: saturation decay (gamma = 1/2), lr-coupled candidate, lr decay deferred until tau = 1.
    The native loop's decisions, learning rate and period list equal the oracle's."""
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, K, tau0, I, probe = (96, 64, 10), 4, 32, 120, 8, 10, 256
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 2048, 35)
    offs = wl.batch_row_offsets(11, K, m, 2048, B)
    refined = {"gamma": 0.5, "slack": 0, "decay_at": [30, 60], "decay_factor": 0.1}
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), 0.0, tau0, adacomm_interval=I, probe_rows=probe,
                        refined=refined)
    xd, yd = to_device(X, y)
    eng = LocalSGD(m, dims, lr=0.05, momentum=0.0, batch=B); eng.bind_dataset(xd, yd); eng.set_params(x1)
    out = eng.run_refined(K, tau0, offs, I, probe, gamma=0.5, slack=0, decay_at=[30, 60], decay_factor=0.1)
    assert out["decision_k"] == [k for k, _, _ in ref.F_trace]
    assert out["decision_tau"] == [t for _, _, t in ref.F_trace]
    assert out["taus"] == ref.taus
    for F, (_, Fr, _) in zip(out["decision_F"], ref.F_trace):
        assert abs(float(F) - Fr) / Fr <= 1e-4
    # the period reached 1, so at least one scheduled decay was applied, and only at decisions with tau == 1
    assert len(ref.lr_trace) >= 1
    in_force = dict(zip(out["decision_k"], [tau0] + out["decision_tau"][:-1]))     # period in force at each decision
    due = [30, 60]
    for k_dec, _ in ref.lr_trace:
        assert in_force[k_dec] == 1 and due.pop(0) <= k_dec
    # ... and no decision at which a decay was due and the period was 1 went without one
    decayed, due = {k for k, _ in ref.lr_trace}, [30, 60]
    for k_dec in out["decision_k"]:
        if due and due[0] <= k_dec and in_force[k_dec] == 1:
            assert k_dec in decayed
            due.pop(0)
    assert abs(out["lr"] - ref.lr_trace[-1][1]) <= 1e-12 * max(1.0, ref.lr_trace[-1][1]) or out["lr"] == f32(ref.lr_trace[-1][1])
    # the decisions recomputed from the GPU's own logged losses are bit-exact
    lr0, lr, prev, pending = f32(0.05), f32(0.05), tau0, [30, 60]
    for k, F, t in zip(out["decision_k"], out["decision_F"], out["decision_tau"]):
        changed = False
        if pending and pending[0] <= k and prev == 1:
            pending.pop(0); lr = float(np.float32(lr * 0.1)); changed = True
        want = orc.adacomm_next_tau_refined(float(F), out["F_0"], tau0, prev, 0.5, 0, lr0, lr, changed)
        assert t == want
        prev = t
    eng.close()


def test_wall_clock_intervals():
    """Section 4: decisions at wall-clock interval boundaries.  With T0 <= 0 every averaging point decides, which
    is the iteration scheme with interval 1 and must follow the oracle; with a real T0 the schedule depends on
    the machine, and what is checked is every decision against the rule and the interval bookkeeping."""
    import torch
    from paper_1810_08313_b200 import binding
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B, tau0, K, probe = (96, 64, 48, 10), 4, 32, 6, 60, 256
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 31)
    offs = wl.batch_row_offsets(4, K, m, 1024, B)
    xd, yd = to_device(X, y)
    eng = LocalSGD(m, dims, lr=0.05, momentum=0.9, batch=B)
    eng.bind_dataset(xd, yd)
    # (1) every averaging point decides
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(0.9), tau0, adacomm_interval=1, probe_rows=probe)
    eng.set_params(x1)
    out = eng.run_timed(K, tau0, 0.0, offs, probe)
    eng.sync()
    assert out["taus"] == ref.taus
    assert out["decision_k"] == [k for k, _, _ in ref.F_trace]
    assert out["decision_tau"] == [t for _, _, t in ref.F_trace]
    gx, _ = eng.get_all()
    assert max_rel_err_per_tensor(gx[0], ref.params[0], dims, True) <= 2e-4
    # (2) an interval longer than the run: the period never changes
    eng.set_params(x1)
    out = eng.run_timed(K, tau0, 1e9, offs, probe)
    assert out["decision_k"] == [] and out["taus"] == [tau0] * (K // tau0)
    # (3) a real interval: each decision follows the rule on its logged loss, in a later interval than the last
    eng.set_params(x1)
    T0 = 0.25
    out = eng.run_timed(K, tau0, T0, offs, probe)
    assert len(out["decision_k"]) >= 1
    last = 0
    for F, t, ms in zip(out["decision_F"], out["decision_tau"], out["decision_ms"]):
        assert t == binding.adacomm_next_tau(float(F), out["F_0"], tau0)
        assert int(ms // T0) > last or last == 0
        assert ms >= T0
        last = int(ms // T0)
    assert sum(min(t, K) for t in out["taus"]) >= K
    eng.close()


@pytest.mark.parametrize("dims,dtype,m,B,mu", [
    ((256, 128, 128, 10), "fp32", 3, 128, 0.9),        # fp32 tensor-core layers, one tile per layer and replica
    ((384, 256, 256, 10), "fp32", 4, 128, 0.0),        # no momentum buffers
    ((256, 256, 128, 10), "bf16", 5, 128, 0.9),        # bf16 with the operand copies
    ((1024, 1024, 10), "bf16", 3, 256, 0.9),           # more tiles than SMs per replica set: several rounds, strips
    ((2048, 1280, 10), "bf16", 2, 128, 0.9),           # 160 tiles on 148 CTAs: a whole round and left-over strips
    ((1536, 1280, 10), "fp32", 2, 128, 0.9),           # the same with fp32 strips (120 tiles: fewer than CTAs ... one round)
    ((100, 70, 10), "fp32", 3, 32, 0.9),               # no tensor-core layer: nothing to fuse, same call
])
def test_period_call_equals_steps_then_average(dims, dtype, m, B, mu):
    """ls_local_steps_avg (one call per period) against ls_local_steps followed by ls_average, from the same
    state and batches: every replica's parameters and momentum bit for bit, and all replicas equal (Section 2,
    PASGD update rule for k mod tau = 0)."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    bf = dtype == "bf16"
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 41, bf16=bf)
    tau = 3
    offs = wl.batch_row_offsets(13, tau, m, 1024, B)
    xd, yd = to_device(X, y, bf16=bf)
    rng = np.random.default_rng(5)
    xs = [x1 + 0.01 * rng.standard_normal(x1.size).astype(np.float32) for _ in range(m)]
    vs = [0.01 * rng.standard_normal(x1.size).astype(np.float32) for _ in range(m)]
    res = {}
    for tag in ("fused", "separate"):
        eng = LocalSGD(m, dims, gemm_dtype=dtype, lr=0.05, momentum=mu, batch=B)
        eng.bind_dataset(xd, yd)
        for i in range(m):
            eng.set_state(i, xs[i], vs[i])
        if tag == "separate":
            eng.local_steps(tau, offs)
            eng.average()
        else:
            eng.local_steps(tau, offs, average=True)
        eng.sync()
        px, pv = eng.get_all()
        F = eng.eval_loss(m - 1, 0, 2 * B)          # reads the operand copies of the last replica (bf16 models)
        res[tag] = (np.array(px), np.array(pv), F)
        eng.close()
    fx, fv, fF = res["fused"]
    for tag in ("separate",):
        ox, ov, oF = res[tag]
        assert np.array_equal(fx.view(np.uint32), ox.view(np.uint32)), tag
        assert np.array_equal(fv.view(np.uint32), ov.view(np.uint32)), tag
        assert fF == oF, tag
    assert all(np.array_equal(fx[0], fx[i]) for i in range(m))
    if mu != 0.0:        # without momentum the buffers are neither used nor averaged
        assert all(np.array_equal(fv[0], fv[i]) for i in range(m))



def test_bounded_wait_that_runs_out_is_reported_and_cleared():
    """A kernel whose bounded wait gives up records the failure and returns; every call that waits for the
    stream reports it once as LS_ERR_DEVICE_TIMEOUT, and the handle keeps working afterwards.  The wait that
    runs out is the self-test kernel's (a barrier on which nothing arrives, limit of about a millisecond):
    nothing faults or hangs."""
    import torch
    from paper_1810_08313_b200 import binding
    from paper_1810_08313_b200.binding import LocalSGD, LsError
    dims, m, B = (96, 64, 10), 3, 32
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 3)
    xd, yd = to_device(X, y)
    eng = LocalSGD(m, dims, lr=0.05, momentum=0.9, batch=B); eng.bind_dataset(xd, yd); eng.set_params(x1)
    offs = wl.batch_row_offsets(2, 12, m, 1024, B)
    # (1) ls_sync
    eng.selftest_wait_timeout(2_000_000)
    with pytest.raises(LsError) as e:
        eng.sync()
    assert e.value.code == binding.LS_ERR_DEVICE_TIMEOUT
    eng.sync()                                           # reported once, then clear
    # (2) a synchronous loss evaluation
    eng.selftest_wait_timeout(2_000_000)
    with pytest.raises(LsError) as e:
        eng.eval_loss(0, 0, 2 * B)
    assert e.value.code == binding.LS_ERR_DEVICE_TIMEOUT
    F = eng.eval_loss(0, 0, 2 * B)
    assert np.isfinite(F) and F > 0
    # (3) the native run loop stops at its next decision point instead of feeding the controller
    eng.selftest_wait_timeout(2_000_000)
    with pytest.raises(LsError) as e:
        eng.run(12, 4, offs, interval=4, probe_rows=2 * B)
    assert e.value.code == binding.LS_ERR_DEVICE_TIMEOUT
    # (4) host-fed steps
    xh = torch.from_numpy(X[:2 * m * B].reshape(2, m, B, dims[0])).pin_memory()
    yh = torch.from_numpy(y[:2 * m * B].reshape(2, m, B)).pin_memory()
    lh = torch.zeros((2, m)).pin_memory()
    eng.selftest_wait_timeout(2_000_000)
    with pytest.raises(LsError) as e:
        eng.local_steps_host(2, xh, yh, lh)
    assert e.value.code == binding.LS_ERR_DEVICE_TIMEOUT
    # the handle is as good as new: a run from a fresh start equals the oracle's
    eng.set_params(x1)
    eng.run(8, 4, offs[:8])
    eng.sync()
    ref = orc.run_pasgd(spec, x1, X, y, offs[:8], B, f32(0.05), f32(0.9), 4)
    p, _ = eng.get_state(0)
    assert max_rel_err_per_tensor(p, ref.params[0], dims, True) <= 1e-4
    assert eng.lib.ls_selftest_wait_timeout(eng.h, 0) == binding.LS_ERR_INVALID_ARG
    eng.close()


@pytest.mark.parametrize("dims,dtype,m,B,mu", [
    ((256, 256, 128, 10), "bf16", 5, 128, 0.9),        # strips of 64 columns over three layers
    ((1024, 1024, 10), "bf16", 16, 256, 0.9),          # 128 units on 148 SMs, sixteen replicas
    ((2048, 1280, 10), "bf16", 2, 128, 0.0),           # no momentum buffers; more units than SMs
    ((3072, 512, 512, 10), "fp32", 4, 128, 0.9),       # fp32 model: only the shared reads apply
])
def test_period_of_one_from_a_synchronized_start(dims, dtype, m, B, mu):
    """Communication period 1 (Section 4.2: where AdaComm ends up).  Every step starts with all replicas equal, and
    the library uses that: the update reads the old W, v once (from its synchronized copy), and for bf16 models
    the step and its averaging are one launch that never writes the per-replica values.  Both must leave the
    state of ls_local_steps + ls_average bit for bit: compared with a handle that is forced onto the general
    path (its replicas are injected one by one with identical values, so the library cannot assume equality)."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    bf = dtype == "bf16"
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 43, bf16=bf)
    K = 4
    offs = wl.batch_row_offsets(17, K, m, 1024, B)
    xd, yd = to_device(X, y, bf16=bf)
    out = {}
    for tag in ("fused", "shared_reads", "general"):
        eng = LocalSGD(m, dims, gemm_dtype=dtype, lr=0.05, momentum=mu, batch=B)
        eng.bind_dataset(xd, yd)
        eng.set_params(x1)
        losses = torch.zeros((K, m), device="cuda")
        for k in range(K):
            if tag == "fused":
                eng.local_steps(1, offs[k:k + 1], losses[k:k + 1], average=True)
            elif tag == "shared_reads":
                eng.local_steps(1, offs[k:k + 1], losses[k:k + 1])
                eng.average()
            else:
                eng.sync()
                px, pv = eng.get_all()
                for i in range(m):
                    eng.set_state(i, px[i], pv[i])          # same values, but now "unknown" to the library
                eng.local_steps(1, offs[k:k + 1], losses[k:k + 1])
                eng.average()
        eng.sync()
        px, pv = eng.get_all()
        F = eng.eval_loss(m - 1, 0, 2 * B)                  # reads the bf16 copies of the last replica
        p_dev, v_dev = eng.state_view()
        assert bool((p_dev[0:1] == p_dev).all())
        out[tag] = (px, pv, F, losses.cpu().numpy())
        eng.close()
    for tag in ("shared_reads", "general"):
        assert np.array_equal(out["fused"][0].view(np.uint32), out[tag][0].view(np.uint32)), tag
        assert np.array_equal(out["fused"][1].view(np.uint32), out[tag][1].view(np.uint32)), tag
        assert out["fused"][2] == out[tag][2], tag
        assert np.array_equal(out["fused"][3], out[tag][3]), tag
    # and it is still the method: against the oracle over the four periods
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(mu), 1)
    lerr = np.max(np.abs(out["fused"][3] - ref.loss) / ref.loss)
    assert lerr <= (2e-2 if bf else 1e-4)


@pytest.mark.parametrize("dims,m,B,mu,tau", [
    ((256, 256, 128, 10), 5, 128, 0.9, 3),             # odd replica count: the mean lands in the first buffer
    ((1024, 1024, 10), 16, 256, 0.9, 2),               # sixteen replicas, CTA-pair GEMMs
    ((2048, 1280, 10), 2, 128, 0.0, 4),                # no momentum buffers; more units than SMs
])
def test_last_step_of_a_period_fused_with_the_average(dims, m, B, mu, tau):
    """Communication periods longer than 1: the last local step of a period and the averaging step are one launch for
    the streamed layers of a bf16 model (every replica's own W, v read once, the per-replica results never
    written).  It must leave the state of ls_local_steps followed by ls_average bit for bit, period after period."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 47, bf16=True)
    periods = 3
    offs = wl.batch_row_offsets(19, periods * tau, m, 1024, B)
    xd, yd = to_device(X, y, bf16=True)
    out = {}
    for tag in ("fused", "separate"):
        eng = LocalSGD(m, dims, gemm_dtype="bf16", lr=0.05, momentum=mu, batch=B)
        eng.bind_dataset(xd, yd)
        eng.set_params(x1)
        losses = torch.zeros((periods * tau, m), device="cuda")
        eng.profile_begin()
        for j in range(periods):
            sl = slice(j * tau, (j + 1) * tau)
            if tag == "fused":
                eng.local_steps(tau, offs[sl], losses[sl], average=True)
            else:
                eng.local_steps(tau, offs[sl], losses[sl])
                eng.average()
        eng.sync()
        px, pv = eng.get_all()
        F = eng.eval_loss(m - 1, 0, 2 * B)                  # reads the bf16 copies of the last replica
        p_dev, _ = eng.state_view()
        assert bool((p_dev[0:1] == p_dev).all())
        prof = eng.profile_end()
        eng.sync()
        out[tag] = (px, pv, F, losses.cpu().numpy(), prof)
        eng.close()
    a, b = out["fused"], out["separate"]
    assert np.array_equal(a[0].view(np.uint32), b[0].view(np.uint32))
    assert np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    assert a[2] == b[2]
    assert np.array_equal(a[3], b[3])
    # the two really took different launch sequences: ("avg", 1) is the step + averaging launch
    assert a[4][("avg", 1)][1] == periods and ("avg", 1) not in b[4]
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(mu), tau)
    assert np.max(np.abs(a[3] - ref.loss) / ref.loss) <= 2e-2
