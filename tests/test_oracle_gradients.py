"""Pins for the oracle's objective and stochastic gradient (Section 2:
F(x) = mean of per-sample losses, g(x; xi) = mean of per-sample gradients)."""
import numpy as np
import pytest
import torch

from oracle import localsgd_oracle as orc


def _fd_grad(spec, x, X, y, h=1e-6):
    g = np.zeros_like(x)
    for p in range(x.size):
        xp = x.copy(); xp[p] += h
        xm = x.copy(); xm[p] -= h
        g[p] = (orc.batch_loss(spec, xp, X, y) - orc.batch_loss(spec, xm, X, y)) / (2 * h)
    return g


@pytest.mark.parametrize("dims,loss,bias", [
    ((5, 4, 3), orc.LOSS_SOFTMAX_CE, True),
    ((5, 4, 3), orc.LOSS_SOFTMAX_CE, False),
    ((6, 5, 4, 3), orc.LOSS_SOFTMAX_CE, True),
    ((4, 3), orc.LOSS_SOFTMAX_CE, True),
    ((7, 1), orc.LOSS_MSE_HALF, False),
    ((5, 4, 1), orc.LOSS_MSE_HALF, True),
])
def test_gradient_matches_central_differences(dims, loss, bias):
    rng = np.random.default_rng(3)
    spec = orc.ModelSpec(dims, loss, bias)
    x = rng.standard_normal(spec.n_params) * 0.7
    X = rng.standard_normal((3, dims[0]))
    y = rng.integers(0, dims[-1], 3) if loss == orc.LOSS_SOFTMAX_CE else rng.standard_normal(3)
    _, g = orc.loss_and_grad(spec, x, X, y)
    fd = _fd_grad(spec, x, X, y)
    assert np.max(np.abs(g - fd)) / np.max(np.abs(fd)) < 1e-6


def test_least_squares_closed_form_gradient_and_loss():
    rng = np.random.default_rng(5)
    A = rng.standard_normal((9, 6)); yv = rng.standard_normal(9); x = rng.standard_normal(6)
    spec = orc.ModelSpec((6, 1), orc.LOSS_MSE_HALF, False)
    loss, g = orc.loss_and_grad(spec, x, A, yv)
    r = A @ x - yv
    np.testing.assert_allclose(g, A.T @ r / 9, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(loss, (r @ r) / (2 * 9), rtol=1e-13)


def _torch_mlp_loss(dims, bias, x_flat, X, y, loss):
    """The same network written with torch.nn.functional and autograd."""
    x = torch.tensor(x_flat, dtype=torch.float64, requires_grad=True)
    a = torch.tensor(X, dtype=torch.float64)
    off = 0
    L = len(dims) - 1
    for l in range(L):
        n_out, n_in = dims[l + 1], dims[l]
        W = x[off:off + n_out * n_in].view(n_out, n_in); off += n_out * n_in
        b = None
        if bias:
            b = x[off:off + n_out]; off += n_out
        a = torch.nn.functional.linear(a, W, b)
        if l + 1 < L:
            a = torch.relu(a)
    if loss == orc.LOSS_SOFTMAX_CE:
        out = torch.nn.functional.cross_entropy(a, torch.tensor(y, dtype=torch.long))
    else:
        out = 0.5 * torch.nn.functional.mse_loss(a[:, 0], torch.tensor(y, dtype=torch.float64))
    out.backward()
    return float(out.detach()), x.grad.numpy()


@pytest.mark.parametrize("dims,loss,bias", [
    ((12, 9, 7, 5), orc.LOSS_SOFTMAX_CE, True),
    ((12, 5), orc.LOSS_SOFTMAX_CE, True),
    ((12, 8, 1), orc.LOSS_MSE_HALF, False),
])
def test_matches_torch_autograd(dims, loss, bias):
    rng = np.random.default_rng(11)
    spec = orc.ModelSpec(dims, loss, bias)
    x = rng.standard_normal(spec.n_params) * 0.5
    X = rng.standard_normal((17, dims[0]))
    y = rng.integers(0, dims[-1], 17) if loss == orc.LOSS_SOFTMAX_CE else rng.standard_normal(17)
    l0, g0 = orc.loss_and_grad(spec, x, X, y)
    l1, g1 = _torch_mlp_loss(dims, bias, x, X, y, loss)
    assert abs(l0 - l1) <= 1e-12 * max(1.0, abs(l1))
    np.testing.assert_allclose(g0, g1, rtol=1e-10, atol=1e-13)


def test_uniform_logits_loss_is_log_classes():
    # zero weights => uniform softmax => loss = ln(C), gradient of bias = 1/C - onehot mean
    spec = orc.ModelSpec((6, 10), orc.LOSS_SOFTMAX_CE, True)
    rng = np.random.default_rng(0)
    X = rng.standard_normal((8, 6)); y = rng.integers(0, 10, 8)
    loss, g = orc.loss_and_grad(spec, np.zeros(spec.n_params), X, y)
    assert abs(loss - np.log(10.0)) < 1e-14
    gb = g[-10:]
    want = 0.1 - np.bincount(y, minlength=10) / 8.0
    np.testing.assert_allclose(gb, want, atol=1e-15)


def test_large_logits_do_not_overflow():
    spec = orc.ModelSpec((2, 3), orc.LOSS_SOFTMAX_CE, False)
    x = np.array([1000.0, 0, 0, 0, -1000.0, 0])
    X = np.array([[1.0, 0.0]]); y = np.array([0])
    loss, g = orc.loss_and_grad(spec, x, X, y)
    assert np.isfinite(loss) and np.all(np.isfinite(g)) and abs(loss) < 1e-12
