"""Pins for the oracle's PASGD loop (Section 2: PASGD update rule and the
tau = 1 special case; appendix proof: X_k (I - J) identity)."""
import numpy as np
import pytest
import torch

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import workloads as wl


def _tiny_problem(dims=(12, 9, 5), n=256, seed=7, loss=orc.LOSS_SOFTMAX_CE, bias=True):
    spec = orc.ModelSpec(dims, loss, bias)
    X = wl.gaussian_rows(seed, n, dims[0])
    if loss == orc.LOSS_SOFTMAX_CE:
        y = wl.teacher_labels(seed, X, dims) if len(dims) > 2 else wl.linear_teacher_labels(seed, X, dims[1])
    else:
        y = np.random.default_rng(seed).standard_normal(n).astype(np.float32)
    x1 = wl.random_mlp_point(seed, dims, bias)
    return spec, X, y, x1


def _torch_sgd(dims, bias, x1, X, y, batches, lr, mu):
    """Plain (momentum) SGD with torch.optim.SGD and torch's cross-entropy, fp64."""
    x = torch.tensor(np.asarray(x1, dtype=np.float64), requires_grad=True)
    opt = torch.optim.SGD([x], lr=lr, momentum=mu)
    L = len(dims) - 1
    for rows in batches:
        a = torch.tensor(X[rows], dtype=torch.float64)
        off = 0
        for l in range(L):
            n_out, n_in = dims[l + 1], dims[l]
            W = x[off:off + n_out * n_in].view(n_out, n_in); off += n_out * n_in
            b = None
            if bias:
                b = x[off:off + n_out]; off += n_out
            a = torch.nn.functional.linear(a, W, b)
            if l + 1 < L:
                a = torch.relu(a)
        loss = torch.nn.functional.cross_entropy(a, torch.tensor(y[rows], dtype=torch.long))
        opt.zero_grad()
        loss.backward()
        opt.step()
    return x.detach().numpy()


@pytest.mark.parametrize("mu", [0.0, 0.9])
def test_m1_is_plain_sgd(mu):
    spec, X, y, x1 = _tiny_problem()
    B, K = 8, 12
    offs = wl.batch_row_offsets(1, K, 1, X.shape[0], B)
    res = orc.run_pasgd(spec, x1, X, y, offs, B, lr=0.05, mu=mu, tau=5)
    batches = [np.arange(int(o), int(o) + B) for o in offs[:, 0]]
    want = _torch_sgd(spec.dims, True, x1, X, y, batches, 0.05, mu)
    # fp32 storage of the state vs torch's fp64 state
    assert np.max(np.abs(res.params[0] - want)) / np.max(np.abs(want)) < 2e-6


@pytest.mark.parametrize("mu", [0.0, 0.9])
def test_tau1_is_synchronous_sgd_on_the_m_fold_batch(mu):
    spec, X, y, x1 = _tiny_problem()
    B, K, m = 8, 10, 4
    offs = wl.batch_row_offsets(2, K, m, X.shape[0], B)
    res = orc.run_pasgd(spec, x1, X, y, offs, B, lr=0.05, mu=mu, tau=1)
    batches = [np.concatenate([np.arange(int(o), int(o) + B) for o in offs[k]]) for k in range(K)]
    want = _torch_sgd(spec.dims, True, x1, X, y, batches, 0.05, mu)
    for i in range(m):
        assert np.max(np.abs(res.params[i] - want)) / np.max(np.abs(want)) < 1e-6
    assert res.avg_points == list(range(1, K + 1))


def test_replicas_identical_after_every_average_and_differ_inside():
    spec, X, y, x1 = _tiny_problem()
    B, K, m, tau = 8, 13, 3, 4
    offs = wl.batch_row_offsets(3, K, m, X.shape[0], B)
    seen = []

    def hook(k, xs, vs, averaged):
        same = all(np.array_equal(xs[0].view(np.uint32), xs[j].view(np.uint32)) and
                   np.array_equal(vs[0].view(np.uint32), vs[j].view(np.uint32)) for j in range(1, m))
        seen.append((k, averaged, same))

    res = orc.run_pasgd(spec, x1, X, y, offs, B, lr=0.05, mu=0.9, tau=tau, state_hook=hook)
    assert res.avg_points == [4, 8, 12, 13]          # last period cut short, then averaged
    assert res.taus == [4, 4, 4, 4]
    for k, averaged, same in seen:
        assert same == averaged, (k, averaged)


def test_deviation_identity_and_mean_recursion():
    # No momentum.  Within a period started from equal models:
    #   X_k (I - J) = -eta sum_{r<k} G_r (I - J)    and   mean_k+1 = mean_k - eta mean_i g_i
    spec, X, y, x1 = _tiny_problem()
    B, m, tau, lr = 8, 4, 6, 0.05
    offs = wl.batch_row_offsets(4, tau, m, X.shape[0], B)
    xs = np.repeat(x1[None].astype(np.float64), m, axis=0)
    Gsum = np.zeros_like(xs)
    snaps = []

    def hook(k, x32, v32, averaged):
        if not averaged:
            snaps.append(x32.astype(np.float64).copy())

    orc.run_pasgd(spec, x1, X, y, offs, B, lr=lr, mu=0.0, tau=tau, state_hook=hook)
    # recompute the gradients at the oracle's own iterates and accumulate
    cur = np.repeat(x1[None].astype(np.float64), m, axis=0)
    for k in range(tau):
        G = np.stack([orc.loss_and_grad(spec, cur[i], X[int(offs[k, i]):int(offs[k, i]) + B],
                                        y[int(offs[k, i]):int(offs[k, i]) + B])[1] for i in range(m)])
        Gsum += G
        mean_next = cur.mean(axis=0) - lr * G.mean(axis=0)
        nxt = snaps[k]
        dev = nxt - nxt.mean(axis=0, keepdims=True)
        want_dev = -lr * (Gsum - Gsum.mean(axis=0, keepdims=True))
        scale = np.max(np.abs(nxt))
        assert np.max(np.abs(dev - want_dev)) / scale < 1e-6
        assert np.max(np.abs(nxt.mean(axis=0) - mean_next)) / scale < 1e-6
        cur = nxt


def test_momentum_modes():
    spec, X, y, x1 = _tiny_problem()
    B, K, m, tau = 8, 6, 3, 3
    offs = wl.batch_row_offsets(5, K, m, X.shape[0], B)
    keep = orc.run_pasgd(spec, x1, X, y, offs, B, 0.05, 0.9, tau, momentum_mode=orc.MOMENTUM_KEEP)
    avg = orc.run_pasgd(spec, x1, X, y, offs, B, 0.05, 0.9, tau, momentum_mode=orc.MOMENTUM_AVERAGE)
    rst = orc.run_pasgd(spec, x1, X, y, offs, B, 0.05, 0.9, tau, momentum_mode=orc.MOMENTUM_RESET)
    assert not np.array_equal(keep.momentum[0], keep.momentum[1])
    assert np.array_equal(avg.momentum[0], avg.momentum[1])
    assert np.all(rst.momentum == 0)
    # parameters are always synchronized at the end
    for r in (keep, avg, rst):
        assert np.array_equal(r.params[0], r.params[2])
    # first period is identical in all modes (buffers start at zero), so the mean after it agrees;
    # the modes differ afterwards
    assert not np.array_equal(keep.params[0], avg.params[0])


def test_least_squares_full_batch_follows_spectral_closed_form():
    # deterministic gradient descent on F(x) = |Ax - y|^2 / (2N):
    #   x_k - x* = (I - eta H)^k (x_1 - x*),  H = A^T A / N, x* from the normal equations
    n, d, K, lr = 64, 10, 40, 0.05
    A, yv, _ = wl.least_squares_problem(9, n, d)
    spec = orc.ModelSpec((d, 1), orc.LOSS_MSE_HALF, False)
    offs = np.zeros((K, 3), dtype=np.int64)        # every replica uses the whole dataset
    res = orc.run_pasgd(spec, np.zeros(d, np.float32), A, yv, offs, n, lr=lr, mu=0.0, tau=7)
    A64 = A.astype(np.float64); y64 = yv.astype(np.float64)
    H = A64.T @ A64 / n
    x_star = np.linalg.solve(A64.T @ A64, A64.T @ y64)
    w, V = np.linalg.eigh(H)
    want = x_star + V @ (((1 - lr * w) ** K) * (V.T @ (0 - x_star)))
    assert np.max(np.abs(res.params[0] - want)) / np.max(np.abs(want)) < 5e-6


def test_least_squares_error_floor_grows_with_tau():
    # Theorem 1's third term: the steady-state error grows with the communication period.
    n, d, m, B, K, lr = 512, 16, 8, 4, 600, 0.02
    A, yv, _ = wl.least_squares_problem(10, n, d, noise_var=0.25)
    spec = orc.ModelSpec((d, 1), orc.LOSS_MSE_HALF, False)
    offs = wl.batch_row_offsets(6, K, m, n, B)
    A64 = A.astype(np.float64); y64 = yv.astype(np.float64)
    x_star = np.linalg.solve(A64.T @ A64, A64.T @ y64)
    F_star = orc.batch_loss(spec, x_star, A, yv)
    floors = []
    for tau in (1, 10, 50):
        tail = []

        def hook(k, xs, vs, averaged, tail=tail):
            if averaged and k > K // 2:
                tail.append(orc.batch_loss(spec, xs[0], A, yv) - F_star)

        orc.run_pasgd(spec, np.zeros(d, np.float32), A, yv, offs, B, lr=lr, mu=0.0, tau=tau, state_hook=hook)
        floors.append(float(np.mean(tail)))
    assert floors[0] > 0 and floors[0] < floors[1] < floors[2]


def test_adacomm_intervals_follow_the_rule():
    spec, X, y, x1 = _tiny_problem(n=512)
    B, K, m = 8, 60, 2
    offs = wl.batch_row_offsets(8, K, m, X.shape[0], B)
    res = orc.run_pasgd(spec, x1, X, y, offs, B, lr=0.05, mu=0.0, tau=8, adacomm_interval=10, probe_rows=128)
    assert res.F_0 is not None and len(res.F_trace) >= 2
    # decisions are taken at averaging points only, at most one per interval crossing
    ks = [k for k, _, _ in res.F_trace]
    assert all(k in res.avg_points for k in ks)
    assert ks[0] == 16          # periods end at 8, 16: first point at or past k = 10
    for k, F_t, tau in res.F_trace:
        assert tau == max(1, int(np.ceil(np.sqrt(F_t / res.F_0) * 8)))
    # the period list is what the decisions dictate
    assert orc.tau_schedule_from_trace(res.F_0, 8, [F for _, F, _ in res.F_trace]) == [t for _, _, t in res.F_trace]
    # periods tile the run exactly
    assert res.avg_points[-1] == K


# ---- block momentum (Section 5.3) ---------------------------------------------------------------------

def test_block_momentum_tau1_is_synchronous_momentum_sgd():
    """tau = 1, no local momentum: G_j is the averaged mini-batch gradient, so block momentum with factor
    beta is plain momentum SGD on the m-fold batch (torch.optim.SGD(momentum=beta))."""
    spec, X, y, x1 = _tiny_problem()
    B, K, m, beta = 8, 10, 4, 0.3
    offs = wl.batch_row_offsets(2, K, m, X.shape[0], B)
    res = orc.run_pasgd(spec, x1, X, y, offs, B, lr=float(np.float32(0.05)), mu=0.0, tau=1,
                        momentum_mode=orc.MOMENTUM_BLOCK, block_beta=float(np.float32(beta)))
    batches = [np.concatenate([np.arange(int(o), int(o) + B) for o in offs[k]]) for k in range(K)]
    want = _torch_sgd(spec.dims, True, x1, X, y, batches, float(np.float32(0.05)), float(np.float32(beta)))
    for i in range(m):
        assert np.max(np.abs(res.params[i] - want)) / np.max(np.abs(want)) < 5e-6


def test_block_momentum_scalar_chain_and_special_cases():
    rng = np.random.default_rng(8)
    m, P = 4, 37
    X = rng.standard_normal((m, P)).astype(np.float32)
    anchor = rng.standard_normal(P).astype(np.float32)
    u = rng.standard_normal(P).astype(np.float32)
    lr, beta = np.float32(0.05), np.float32(0.3)
    want_x = np.empty(P, np.float32); want_u = np.empty(P, np.float32)
    for p in range(P):
        s = np.float32(X[0, p])
        for j in range(1, m):
            s = np.float32(s + X[j, p])
        mean = np.float32(s / np.float32(m))
        d = np.float32(anchor[p] - mean)
        G = np.float32(d / lr)
        un = np.float32(np.float32(beta * u[p]) + G)
        want_u[p] = un
        want_x[p] = np.float32(anchor[p] - np.float32(lr * un))
    Xc, ac, uc = X.copy(), anchor.copy(), u.copy()
    orc.block_momentum_average(Xc, ac, uc, float(lr), float(beta))
    for j in range(m):
        assert np.array_equal(Xc[j].view(np.uint32), want_x.view(np.uint32))
    assert np.array_equal(ac.view(np.uint32), want_x.view(np.uint32))
    assert np.array_equal(uc.view(np.uint32), want_u.view(np.uint32))
    # beta = 0 and an empty buffer: the new model is the plain mean up to the rounding of d / eta * eta
    Xc, ac, uc = X.copy(), anchor.copy(), np.zeros(P, np.float32)
    orc.block_momentum_average(Xc, ac, uc, float(lr), 0.0)
    Xm = X.copy(); orc.average_replicas(Xm)
    assert np.max(np.abs(Xc[0] - Xm[0])) <= 4 * 2.0 ** -24 * np.max(np.abs(np.concatenate([anchor, Xm[0]])))
    # no displacement and beta = 1: the model keeps moving along the buffer
    Xc = np.repeat(anchor[None], m, axis=0).copy(); ac = anchor.copy(); uc = np.ones(P, np.float32)
    orc.block_momentum_average(Xc, ac, uc, 0.5, 1.0)
    assert np.allclose(Xc[0], anchor - 0.5, atol=1e-6) and np.allclose(uc, 1.0, atol=1e-6)


def test_block_momentum_run_resets_local_buffers_and_synchronizes():
    spec, X, y, x1 = _tiny_problem()
    B, K, m, tau = 8, 12, 3, 4
    offs = wl.batch_row_offsets(3, K, m, X.shape[0], B)
    res = orc.run_pasgd(spec, x1, X, y, offs, B, 0.05, 0.9, tau, momentum_mode=orc.MOMENTUM_BLOCK, block_beta=0.3)
    assert np.all(res.momentum == 0)
    assert np.array_equal(res.params[0], res.params[2])
    plain = orc.run_pasgd(spec, x1, X, y, offs, B, 0.05, 0.9, tau, momentum_mode=orc.MOMENTUM_RESET)
    assert not np.array_equal(res.params[0], plain.params[0])       # the global momentum changes the trajectory
    assert np.any(res.block_u != 0)


@pytest.mark.parametrize("groups", [2, 4])
def test_grouped_averaging_tau1_is_still_synchronous_sgd(groups):
    """Replicas spread over several devices (grouped summation order): tau = 1 remains fully synchronous
    momentum SGD on the m-fold batch, and all replicas are bitwise equal after every averaging step."""
    spec, X, y, x1 = _tiny_problem()
    B, K, m = 8, 10, 4
    offs = wl.batch_row_offsets(2, K, m, X.shape[0], B)
    same = []
    res = orc.run_pasgd(spec, x1, X, y, offs, B, lr=0.05, mu=0.9, tau=1, avg_groups=groups,
                        state_hook=lambda k, xs, vs, avg: same.append(bool(avg) and bool((xs == xs[0]).all() and (vs == vs[0]).all())))
    batches = [np.concatenate([np.arange(int(o), int(o) + B) for o in offs[k]]) for k in range(K)]
    want = _torch_sgd(spec.dims, True, x1, X, y, batches, 0.05, 0.9)
    for i in range(m):
        assert np.max(np.abs(res.params[i] - want)) / np.max(np.abs(want)) < 1e-6
    assert same[1::2] == [True] * K               # the hook runs after each step and after each average
