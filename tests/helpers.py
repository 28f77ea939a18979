"""Shared helpers of the GPU parity tests (no method arithmetic here)."""
import numpy as np

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import workloads as wl


def f32(v):
    """The double value of v after rounding to float32 (what the C ABI receives)."""
    return float(np.float32(v))


def tensor_slices(dims, has_bias):
    out, off = [], 0
    for l in range(len(dims) - 1):
        n = dims[l + 1] * dims[l]
        out.append(("W%d" % (l + 1), slice(off, off + n))); off += n
        if has_bias:
            out.append(("b%d" % (l + 1), slice(off, off + dims[l + 1]))); off += dims[l + 1]
    return out


def max_rel_err_per_tensor(got, want, dims, has_bias):
    """max over tensors of max|a-b| / max|b| (zero tensors compare absolutely)."""
    worst = 0.0
    for _, s in tensor_slices(dims, has_bias):
        a = np.asarray(got[s], dtype=np.float64); b = np.asarray(want[s], dtype=np.float64)
        den = np.max(np.abs(b))
        err = np.max(np.abs(a - b))
        worst = max(worst, err / den if den > 0 else err)
    return worst


def small_problem(dims, loss, has_bias, n_rows, seed, bf16=False):
    spec = orc.ModelSpec(tuple(dims), loss, has_bias)
    if loss == "mse_half":
        X, y, _ = wl.least_squares_problem(seed, n_rows, dims[0])
    else:
        X = wl.gaussian_rows(seed, n_rows, dims[0])
        if bf16:
            X = wl.round_to_bf16(X)
        y = wl.teacher_labels(seed, X, dims) if len(dims) > 2 else wl.linear_teacher_labels(seed, X, dims[1])
    x1 = wl.random_mlp_point(seed, dims, has_bias)
    return spec, X, y, x1


def to_device(X, y, bf16=False):
    import torch
    xd = torch.from_numpy(X).cuda()
    if bf16:
        xd = xd.to(torch.bfloat16)
    yd = torch.from_numpy(y).cuda()
    return xd.contiguous(), yd.contiguous()
