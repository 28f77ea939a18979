"""The allocation-free entry point ls_linear_loss_static against ls_eval_loss.

Who needs it: callers that are not allowed to allocate device memory at the moment they want a
loss value (a hook inside somebody else's memory pool, a monitor that runs when the GPU is almost
full).  The regular path keeps the output-layer kernel's scratch in a caller-allocated state block;
this entry point keeps it in a fixed array inside the library.  The test calls it twice in a row
through the C ABI (the array is shared between calls and keeps the last call's contents) and checks
both results against the existing entry point on the same weights and rows.
Collected last on purpose, so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest

from paper_1810_08313_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _reference_chunk_losses(dims, x1, X, y, loss, B, bias):
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    eng = LocalSGD(2, dims, loss, bias, "fp32", lr=0.05, momentum=0.0, batch=B)
    eng.bind_dataset(torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda())
    eng.set_params(x1)
    out = np.array([eng.eval_loss(1, c * B, B) for c in range(X.shape[0] // B)], dtype=np.float32)
    eng.close()
    return out


@pytest.mark.parametrize("dims,loss,bias,B,n", [((784, 10), "softmax_ce", True, 32, 1024),
                                                ((300, 7), "softmax_ce", False, 24, 240),
                                                ((4096, 1), "mse_half", False, 64, 512)])
def test_static_scratch_entry_point_matches_eval_loss_twice(dims, loss, bias, B, n):
    import torch
    from paper_1810_08313_b200 import binding
    if loss == "mse_half":
        X, y, _ = wl.least_squares_problem(3, n, dims[0])
    else:
        X = wl.gaussian_rows(3, n, dims[0]); y = wl.linear_teacher_labels(3, X, dims[1])
    x1 = wl.random_mlp_point(5, dims, bias)
    want = _reference_chunk_losses(dims, x1, X, y, loss, B, bias)
    W = torch.from_numpy(x1[:dims[0] * dims[1]].reshape(dims[1], dims[0]).copy()).cuda()
    b = torch.from_numpy(x1[dims[0] * dims[1]:].copy()).cuda() if bias else None
    xd, yd = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    out = torch.full((n // B,), -1.0, dtype=torch.float32, device="cuda")
    for call in range(2):
        out.fill_(-1.0)
        binding.linear_loss_static(W, b, xd, yd, B, out, loss)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.max(np.abs(got - want) / np.abs(want)) <= 1e-6, (call, got[:4], want[:4])
    # a different problem size right after: stale scratch contents must not leak into it
    half = (n // B // 2) * B
    out2 = torch.full((half // B,), -1.0, dtype=torch.float32, device="cuda")
    binding.linear_loss_static(W, b, xd[:half], yd[:half], B, out2, loss)
    torch.cuda.synchronize()
    assert np.max(np.abs(out2.cpu().numpy() - want[:half // B]) / np.abs(want[:half // B])) <= 1e-6


def test_static_scratch_entry_point_rejects_oversize_and_bad_arguments():
    import torch
    from paper_1810_08313_b200 import binding
    lib = binding._lib()
    W = torch.zeros((10, 16), device="cuda"); x = torch.zeros((64, 16), device="cuda")
    y = torch.zeros(64, dtype=torch.int32, device="cuda"); out = torch.zeros(64, device="cuda")
    call = lambda *a: lib.ls_linear_loss_static(*a)
    ok = (W.data_ptr(), None, x.data_ptr(), y.data_ptr())
    assert call(*ok, 64, 16, 10, 0, 8, out.data_ptr(), None) == binding.LS_OK
    assert call(*ok, 64, 16, 17, 0, 8, out.data_ptr(), None) == binding.LS_ERR_TOO_LARGE      # d_out > 16
    assert call(*ok, 65536 * 2, 16, 10, 0, 1024, out.data_ptr(), None) == binding.LS_ERR_TOO_LARGE  # rows
    assert call(*ok, 514, 16, 10, 0, 2, out.data_ptr(), None) == binding.LS_ERR_TOO_LARGE      # 257 chunks
    assert call(*ok, 64, 16, 10, 0, 7, out.data_ptr(), None) == binding.LS_ERR_INVALID_ARG     # ragged chunks
    assert call(None, None, x.data_ptr(), y.data_ptr(), 64, 16, 10, 0, 8, out.data_ptr(), None) == binding.LS_ERR_INVALID_ARG
    assert call(*ok, 64, 16, 10, 1, 8, out.data_ptr(), None) == binding.LS_ERR_INVALID_ARG     # MSE needs d_out == 1
    torch.cuda.synchronize()
