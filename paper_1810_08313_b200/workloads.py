"""Seeded synthetic inputs for local-update SGD runs.

This module only *draws inputs*: datasets, teacher labels, initial points,
mini-batch positions and flat parameter vectors.  It holds none of the
method's arithmetic (no gradient, no update, no averaging, no controller) and
imports neither the CUDA binding nor the CPU oracle; both are handed the
arrays made here.

The shapes stand in for the image-classification workloads of the paper's
Section 5.1 (3x32x32 inputs, 10 classes, 50 000 training rows, mini-batch of
128 per worker); the pixel values themselves are Gaussian noise and the labels
come from a seeded random teacher network, so no dataset is needed.

All randomness comes from numpy's Philox counter-based bit generator keyed by
(seed, stream), so any array can be regenerated independently of the others.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence, Tuple

import numpy as np

# stream ids: one independent Philox stream per kind of array
_STREAM_X = 1
_STREAM_TEACHER = 2
_STREAM_INIT = 3
_STREAM_BATCH = 4
_STREAM_NOISE = 5
_STREAM_TRUTH = 6
_STREAM_FLAT = 7


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Return float32 values rounded (nearest-even) to bf16-representable ones.

    Used so that a dataset handed to a bf16 consumer and to an fp64 consumer
    holds exactly the same numbers.
    """
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    bits = (bits + 0x7FFF + lsb) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).reshape(a.shape)


def gaussian_rows(seed: int, n_rows: int, d: int, chunk: int = 8192) -> np.ndarray:
    """float32 [n_rows][d], entries N(0,1)."""
    g = _rng(seed, _STREAM_X)
    out = np.empty((n_rows, d), dtype=np.float32)
    for r0 in range(0, n_rows, chunk):
        r1 = min(n_rows, r0 + chunk)
        out[r0:r1] = g.standard_normal((r1 - r0, d), dtype=np.float32)
    return out


def n_params(dims: Sequence[int], has_bias: bool = True) -> int:
    return sum(dims[l + 1] * dims[l] + (dims[l + 1] if has_bias else 0) for l in range(len(dims) - 1))


def random_mlp_point(seed: int, dims: Sequence[int], has_bias: bool = True, stream: int = _STREAM_INIT) -> np.ndarray:
    """A seeded point in parameter space, float32, flat.

    Layout (the one both consumers document): for each layer l = 1..L the
    weight matrix W_l as [dims[l]][dims[l-1]] row-major, then the bias b_l
    (dims[l] values) when has_bias.  W_l ~ N(0, 2/fan_in), b_l = 0.
    """
    g = _rng(seed, stream)
    parts = []
    for l in range(len(dims) - 1):
        fan_in, fan_out = dims[l], dims[l + 1]
        w = g.standard_normal((fan_out, fan_in), dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
        parts.append(w.reshape(-1))
        if has_bias:
            parts.append(np.zeros(fan_out, dtype=np.float32))
    return np.concatenate(parts).astype(np.float32)


def teacher_labels(seed: int, X: np.ndarray, dims: Sequence[int], chunk: int = 4096) -> np.ndarray:
    """int32 labels = argmax of a seeded random teacher ReLU network of shape
    `dims` applied to the rows of X (ties -> lowest index).  Only used to give
    the synthetic rows learnable labels."""
    theta = random_mlp_point(seed, dims, has_bias=True, stream=_STREAM_TEACHER)
    mats = []
    off = 0
    for l in range(len(dims) - 1):
        n = dims[l + 1] * dims[l]
        mats.append(theta[off:off + n].reshape(dims[l + 1], dims[l]))
        off += n + dims[l + 1]
    y = np.empty(X.shape[0], dtype=np.int32)
    for r0 in range(0, X.shape[0], chunk):
        a = X[r0:r0 + chunk].astype(np.float32)
        for l, w in enumerate(mats):
            a = a @ w.T
            if l + 1 < len(mats):
                a = np.maximum(a, 0)
        y[r0:r0 + chunk] = np.argmax(a, axis=1).astype(np.int32)
    return y


def linear_teacher_labels(seed: int, X: np.ndarray, n_classes: int) -> np.ndarray:
    """int32 labels = argmax(W* x) with W* ~ N(0, 1/d), no bias."""
    d = X.shape[1]
    g = _rng(seed, _STREAM_TEACHER)
    w = g.standard_normal((n_classes, d), dtype=np.float32) * np.float32(np.sqrt(1.0 / d))
    return np.argmax(X.astype(np.float32) @ w.T, axis=1).astype(np.int32)


def least_squares_problem(seed: int, n_rows: int, d: int, noise_var: float = 0.01):
    """A [n_rows][d] ~ N(0,1), x_true ~ N(0, 1/d), y = A x_true + eps,
    eps ~ N(0, noise_var).  Returns (A float32, y float32, x_true float32)."""
    A = gaussian_rows(seed, n_rows, d)
    x_true = (_rng(seed, _STREAM_TRUTH).standard_normal(d) / np.sqrt(d)).astype(np.float32)
    eps = _rng(seed, _STREAM_NOISE).standard_normal(n_rows) * np.sqrt(noise_var)
    y = (A.astype(np.float64) @ x_true.astype(np.float64) + eps).astype(np.float32)
    return A, y, x_true


def batch_row_offsets(seed: int, n_iters: int, m: int, n_rows: int, batch: int) -> np.ndarray:
    """int64 [n_iters][m]: first dataset row of the mini-batch that replica i
    uses at local iteration k.  A mini-batch is one contiguous block of `batch`
    rows; the block index is uniform with replacement over the n_rows // batch
    whole blocks.  (The rows are i.i.d., so a contiguous block is a uniform
    sample of the dataset.)"""
    n_blocks = n_rows // batch
    if n_blocks < 1:
        raise ValueError("dataset smaller than one mini-batch")
    g = _rng(seed, _STREAM_BATCH)
    return (g.integers(0, n_blocks, size=(n_iters, m), dtype=np.int64) * batch).astype(np.int64)


def uniform_flat(seed: int, m: int, P: int, stream: int = _STREAM_FLAT) -> np.ndarray:
    """float32 [m][P], uniform in (-1, 1)."""
    g = _rng(seed, stream)
    out = np.empty((m, P), dtype=np.float32)
    for j in range(m):
        out[j] = g.random(P, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    return out


# --------------------------------------------------------------------------
# The five workload configurations.
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    name: str
    dims: Tuple[int, ...]
    loss: str                 # "softmax_ce" | "mse_half"
    has_bias: bool
    gemm_dtype: str           # "fp32" | "bf16"
    m: int
    batch: int
    lr: float
    momentum: float
    n_rows: int
    n_iters: int
    taus: Tuple[int, ...]     # fixed communication periods that are swept
    zero_init: bool
    adacomm_tau0: Optional[int] = None
    adacomm_interval: Optional[int] = None
    seed: int = 20181008


WORKLOADS = {
    # softmax regression, fp32
    "c1_softmax": Workload("c1_softmax", (784, 10), "softmax_ce", True, "fp32", m=4, batch=32, lr=0.05,
                           momentum=0.0, n_rows=65536, n_iters=100, taus=(10,), zero_init=True),
    # ReLU MLP 3072-512-512-10, fp32, momentum 0.9
    "c2_mlp_fp32": Workload("c2_mlp_fp32", (3072, 512, 512, 10), "softmax_ce", True, "fp32", m=8, batch=128,
                            lr=0.05, momentum=0.9, n_rows=50000, n_iters=2000, taus=(1, 5, 20, 100),
                            zero_init=False),
    # ReLU MLP 3072-2048^3-10, bf16 GEMMs, AdaComm
    "c3_mlp_bf16": Workload("c3_mlp_bf16", (3072, 2048, 2048, 2048, 10), "softmax_ce", True, "bf16", m=16,
                            batch=256, lr=0.05, momentum=0.9, n_rows=50000, n_iters=5000, taus=(20,),
                            zero_init=False, adacomm_tau0=20, adacomm_interval=50),
    # least squares y = A x + eps
    "c4_lsq": Workload("c4_lsq", (4096, 1), "mse_half", False, "fp32", m=32, batch=64, lr=1e-4, momentum=0.0,
                       n_rows=8192, n_iters=5000, taus=(50, 1, 10), zero_init=True),
}

# averaging-only sweep: flat vectors of P floats, m replicas, params + momentum
AVERAGING_SWEEP_P = (14_706_698, 23_500_000, 1_000_000_000)
AVERAGING_SWEEP_M = (4, 8, 16)


def make_dataset(w: Workload, n_rows: Optional[int] = None):
    """(X float32 [n][d_in], y) for a workload; y is int32 labels for
    softmax_ce and float32 targets for mse_half.  For a bf16 workload the
    entries of X are already rounded to bf16-representable values."""
    n = int(n_rows if n_rows is not None else w.n_rows)
    if w.loss == "mse_half":
        A, y, _ = least_squares_problem(w.seed, n, w.dims[0])
        return A, y
    X = gaussian_rows(w.seed, n, w.dims[0])
    if w.gemm_dtype == "bf16":
        X = round_to_bf16(X)
    if len(w.dims) == 2:
        y = linear_teacher_labels(w.seed, X, w.dims[1])
    else:
        y = teacher_labels(w.seed, X, w.dims)
    return X, y


def initial_point(w: Workload) -> np.ndarray:
    """x_1, the point every replica starts from (float32, flat)."""
    if w.zero_init:
        return np.zeros(n_params(w.dims, w.has_bias), dtype=np.float32)
    return random_mlp_point(w.seed, w.dims, w.has_bias)
