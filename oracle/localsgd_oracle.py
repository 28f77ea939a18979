"""Plain CPU oracle for periodic-averaging local-update SGD (PASGD) and the
AdaComm communication-period rule.

THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It exists so that the CUDA
library can be checked against an independent, slow, obviously-correct
statement of what the method computes.  Only tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  It shares no code with the CUDA
path and imports nothing from it.

Precision: the paper does not fix one.  All gradient arithmetic here is IEEE
double (numpy float64, matmul as a library step).  Replica state (parameters
and momentum buffers) is *stored* in float32, because the method under test
keeps fp32 master copies and its averaging step is specified to the bit in
fp32 (see `average_replicas`); every update is computed in double and rounded
once on store.

Every function cites the passage of the paper it follows.  Where the paper is
silent the reading taken is stated in the docstring.

Parity pins (tests/test_oracle_*.py): finite-difference gradients, torch's own
SGD(+momentum) optimiser and cross-entropy for m=1 and for tau=1 on the
concatenated batch, closed-form least squares (normal equations, spectral form
of gradient descent), replica equality after averaging, the deviation identity
of the convergence proof, exact-rational means, and a hand-computed tau table.
`run_pasgd` trajectories of ReLU networks beyond a few periods are chaotic:
long free-running trajectories are "parity unpinned" (only their invariants
are checked).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

LOSS_SOFTMAX_CE = "softmax_ce"
LOSS_MSE_HALF = "mse_half"

MOMENTUM_AVERAGE = "average"   # buffers are averaged with the parameters
MOMENTUM_KEEP = "keep"         # each worker keeps its own buffer (the paper's "naive" scheme)
MOMENTUM_RESET = "reset"       # buffers cleared at every period start (local half of block momentum)
MOMENTUM_BLOCK = "block"       # block momentum: reset local buffers + a global momentum on the period's step


@dataclass(frozen=True)
class ModelSpec:
    """A fully connected network x -> W_L relu(... relu(W_1 x + b_1) ...) + b_L.

    dims = (d_in, h_1, ..., d_out).  One layer (len(dims) == 2) is a linear
    model: softmax regression with LOSS_SOFTMAX_CE, least squares with
    LOSS_MSE_HALF (d_out must then be 1).
    Flat parameter layout: for l = 1..L, W_l as [dims[l]][dims[l-1]] row-major
    followed by b_l when has_bias.
    """
    dims: Tuple[int, ...]
    loss: str = LOSS_SOFTMAX_CE
    has_bias: bool = True

    @property
    def n_layers(self) -> int:
        return len(self.dims) - 1

    @property
    def n_params(self) -> int:
        return sum(self.dims[l + 1] * self.dims[l] + (self.dims[l + 1] if self.has_bias else 0)
                   for l in range(self.n_layers))

    def unpack(self, x: np.ndarray) -> List[Tuple[np.ndarray, Optional[np.ndarray]]]:
        """Views (W_l, b_l) into the flat vector x."""
        out = []
        off = 0
        for l in range(self.n_layers):
            n_out, n_in = self.dims[l + 1], self.dims[l]
            W = x[off:off + n_out * n_in].reshape(n_out, n_in)
            off += n_out * n_in
            b = None
            if self.has_bias:
                b = x[off:off + n_out]
                off += n_out
            out.append((W, b))
        assert off == x.shape[0] == self.n_params
        return out


# --------------------------------------------------------------------------
# Objective and stochastic gradient  (Section 2: empirical risk F(x) as the
# mean of per-sample losses f(x; s_i); stochastic gradient g(x; xi) as the
# mean of per-sample gradients over the mini-batch xi)
# --------------------------------------------------------------------------

def forward(spec: ModelSpec, x: np.ndarray, X: np.ndarray):
    """Network outputs for the rows of X.  Returns (Z_L, activations, pre-activations).
    ReLU on every layer but the last."""
    A = np.asarray(X, dtype=np.float64)
    acts = [A]
    pre = []
    layers = spec.unpack(np.asarray(x, dtype=np.float64))
    for l, (W, b) in enumerate(layers):
        Z = A @ W.T
        if b is not None:
            Z = Z + b
        pre.append(Z)
        if l + 1 < len(layers):
            A = np.where(Z > 0.0, Z, 0.0)
            acts.append(A)
    return pre[-1], acts, pre


def per_sample_loss(spec: ModelSpec, Z: np.ndarray, y: np.ndarray) -> np.ndarray:
    """f(x; s_i) for each row: cross-entropy of softmax(z) against label y
    (natural log, max-subtracted log-sum-exp), or (z - y)^2 / 2."""
    if spec.loss == LOSS_SOFTMAX_CE:
        zmax = Z.max(axis=1, keepdims=True)
        lse = zmax[:, 0] + np.log(np.exp(Z - zmax).sum(axis=1))
        return lse - Z[np.arange(Z.shape[0]), np.asarray(y, dtype=np.int64)]
    if spec.loss == LOSS_MSE_HALF:
        r = Z[:, 0] - np.asarray(y, dtype=np.float64)
        return 0.5 * r * r
    raise ValueError(spec.loss)


def batch_loss(spec: ModelSpec, x: np.ndarray, X: np.ndarray, y: np.ndarray) -> float:
    """(1/|xi|) sum_i f(x; s_i): the empirical risk of Section 2 restricted to the rows given."""
    Z, _, _ = forward(spec, x, X)
    return float(per_sample_loss(spec, Z, y).mean())


def loss_and_grad(spec: ModelSpec, x: np.ndarray, X: np.ndarray, y: np.ndarray):
    """Mini-batch loss and the stochastic gradient g(x; xi) = (1/|xi|) sum
    grad f(x; s_i) of Section 2, by back-propagation, in double.
    ReLU'(z) = 1 for z > 0 and 0 otherwise."""
    Bn = X.shape[0]
    Z, acts, pre = forward(spec, x, X)
    loss = float(per_sample_loss(spec, Z, y).mean())
    if spec.loss == LOSS_SOFTMAX_CE:
        zmax = Z.max(axis=1, keepdims=True)
        e = np.exp(Z - zmax)
        dZ = e / e.sum(axis=1, keepdims=True)
        dZ[np.arange(Bn), np.asarray(y, dtype=np.int64)] -= 1.0
        dZ /= Bn
    else:
        dZ = ((Z[:, 0] - np.asarray(y, dtype=np.float64)) / Bn)[:, None]
    layers = spec.unpack(np.asarray(x, dtype=np.float64))
    grads = [None] * spec.n_layers
    for l in range(spec.n_layers - 1, -1, -1):
        W, b = layers[l]
        gW = dZ.T @ acts[l]
        gb = dZ.sum(axis=0) if b is not None else None
        grads[l] = (gW, gb)
        if l > 0:
            dA = dZ @ W
            dZ = np.where(pre[l - 1] > 0.0, dA, 0.0)
    parts = []
    for gW, gb in grads:
        parts.append(gW.reshape(-1))
        if gb is not None:
            parts.append(gb)
    return loss, np.concatenate(parts)


# --------------------------------------------------------------------------
# Local step  (Section 2, mini-batch SGD update x_{k+1} = x_k - eta g(x_k);
# Section 5.3 for momentum: the buffer holds the latest change in x, written
# in the form of the block-momentum equations there, u = beta u + g, x -= eta u)
# --------------------------------------------------------------------------

def sgd_momentum_step(x: np.ndarray, v: np.ndarray, g: np.ndarray, lr: float, mu: float):
    """One local update.  Reading taken where the paper is silent: no
    dampening, no Nesterov, buffer starts at zero, eta multiplies the buffer.
    Inputs may be float32; arithmetic is double; returns double arrays."""
    v_new = mu * np.asarray(v, dtype=np.float64) + g
    x_new = np.asarray(x, dtype=np.float64) - lr * v_new
    return x_new, v_new


# --------------------------------------------------------------------------
# Averaging  (Section 2, PASGD update rule, the case k mod tau = 0; the
# operator J = 1 1^T / m of the convergence proof's notation)
# --------------------------------------------------------------------------

def average_replicas(X: np.ndarray) -> None:
    """Replace every row of the float32 matrix X[m][P] by the mean over rows.

    Specified to the bit: the sum runs over replicas in index order,
    s = x^(0); s = s + x^(j) for j = 1..m-1, each add rounded to fp32, then
    one fp32 division by m.  In place.
    """
    if X.dtype != np.float32:
        raise TypeError("average_replicas is specified on float32 state")
    m = X.shape[0]
    s = X[0].copy()
    for j in range(1, m):
        s = s + X[j]
    mean = s / np.float32(m)
    X[:] = mean[None, :]


def average_replicas_grouped(X: np.ndarray, groups: int) -> None:
    """The same averaging step when the m replicas are spread over `groups` devices (Section 2: the workers'
    models are averaged "by a fusion node or by performing an all-node broadcast"; here one partial sum per
    device is exchanged).  Replicas are dealt out in index order, m / groups consecutive ones per device.
    Specified to the bit, the grouped order:
        partial_g = x^(g*q) + x^(g*q+1) + ... + x^(g*q+q-1)   sequentially in fp32, q = m / groups
        total     = partial_0 + partial_1 + ... + partial_{groups-1}   sequentially in fp32 (device order)
        mean      = total / m   (one fp32 division)
    groups = 1 and groups = m are both the sequential order of average_replicas; anything between is a
    different rounding order (and so a different, equally valid, fp32 mean).  In place.
    """
    if X.dtype != np.float32:
        raise TypeError("average_replicas_grouped is specified on float32 state")
    m = X.shape[0]
    groups = int(groups)
    if groups < 1 or m % groups != 0:
        raise ValueError("the replicas must divide evenly over the groups")
    q = m // groups
    total = None
    for g in range(groups):
        part = X[g * q].copy()
        for j in range(1, q):
            part = part + X[g * q + j]
        total = part if total is None else total + part
    mean = total / np.float32(m)
    X[:] = mean[None, :]


def block_momentum_average(X: np.ndarray, anchor: np.ndarray, u: np.ndarray, lr: float, beta: float) -> None:
    """Averaging step with block momentum (Section 5.3):
        u_j = beta_glob * u_{j-1} + G_j ;   x_{(j+1)tau+1} = x_{j tau+1} - eta_j * u_j
    where x_{j tau+1} is the synchronized model the period started from (`anchor`) and G_j is the
    accumulated step of the period in gradient units.  Reading: G_j = (anchor - mean_i x^(i)) / eta, the
    averaged displacement divided by the learning rate; this equals the paper's sum of averaged
    gradients exactly when the local steps are plain SGD, and is the accumulated "big step" between
    two synchronized models otherwise.
    Specified to the bit in fp32, every operation rounded separately (no fused multiply-add):
        mean as in average_replicas;  d = anchor - mean;  G = d / eta;  t = beta * u;  u' = t + G;
        s = eta * u';  x' = anchor - s.   X rows, anchor <- x';  u <- u'.   In place.
    """
    if X.dtype != np.float32 or anchor.dtype != np.float32 or u.dtype != np.float32:
        raise TypeError("block_momentum_average is specified on float32 state")
    m = X.shape[0]
    s = X[0].copy()
    for j in range(1, m):
        s = s + X[j]
    mean = s / np.float32(m)
    eta, b = np.float32(lr), np.float32(beta)
    d = anchor - mean
    G = d / eta
    t = b * u
    u_new = t + G
    step = eta * u_new
    x_new = anchor - step
    X[:] = x_new[None, :]
    anchor[:] = x_new
    u[:] = u_new


# --------------------------------------------------------------------------
# AdaComm  (Section 4.2, basic update rule)
# --------------------------------------------------------------------------

def adacomm_next_tau(F_t: float, F_0: float, tau_0: int) -> int:
    """tau_l = ceil( sqrt(F_t / F_0) * tau_0 ), with F_inf taken as 0.

    Evaluated literally in IEEE double, no epsilon.  Readings taken where the
    paper is silent: a result below 1 becomes 1; growth above tau_0 is allowed;
    F_0 <= 0, F_t < 0, non-finite input or tau_0 < 1 is an error.
    """
    F_t = float(F_t)
    F_0 = float(F_0)
    if not (math.isfinite(F_t) and math.isfinite(F_0)) or F_0 <= 0.0 or F_t < 0.0 or int(tau_0) < 1:
        raise ValueError("adacomm_next_tau: invalid input")
    t = math.sqrt(F_t / F_0) * float(int(tau_0))
    n = math.ceil(t)
    if n < 1:
        n = 1
    if n > 2**31 - 1:
        raise ValueError("adacomm_next_tau: result does not fit an int")
    return int(n)


def adacomm_next_tau_refined(F_t: float, F_0: float, tau_0: int, tau_prev: int, gamma: float = 0.5,
                             slack: int = 0, lr_0: float = 1.0, lr_l: float = 1.0, lr_changed: bool = False) -> int:
    """The refinements of Section 4.3.

    Candidate (Section 4.3.2, the lr-coupled strategy):
        c = ceil( sqrt( (lr_0 / lr_l) * (F_t / F_0) ) * tau_0 ),  at least 1.
    Faster decay when training saturates (Section 4.3.1, with the slack variable s):
        tau_l = c                        if c + s < tau_{l-1}
                gamma * tau_{l-1}        otherwise.
    Readings taken where the paper is silent: gamma * tau_{l-1} is rounded up and kept at least 1;
    the two rules are combined by using c as the candidate of the first; at the first decision after
    the learning rate changed, c is taken as it is (the saturation test compares periods chosen under
    the same learning rate, and Section 4.3.2 wants the period to grow when the rate drops).
    """
    F_t, F_0, gamma, lr_0, lr_l = float(F_t), float(F_0), float(gamma), float(lr_0), float(lr_l)
    if not all(math.isfinite(v) for v in (F_t, F_0, gamma, lr_0, lr_l)):
        raise ValueError("adacomm_next_tau_refined: invalid input")
    if F_0 <= 0.0 or F_t < 0.0 or int(tau_0) < 1 or int(tau_prev) < 1 or not (0.0 < gamma <= 1.0) or int(slack) < 0 \
            or lr_0 <= 0.0 or lr_l <= 0.0:
        raise ValueError("adacomm_next_tau_refined: invalid input")
    c = math.ceil(math.sqrt((lr_0 / lr_l) * (F_t / F_0)) * float(int(tau_0)))
    if c < 1:
        c = 1
    if c > 2**31 - 1:
        raise ValueError("adacomm_next_tau_refined: result does not fit an int")
    if lr_changed or c + int(slack) < int(tau_prev):
        return int(c)
    n = math.ceil(gamma * float(int(tau_prev)))
    return int(max(1, n))


# --------------------------------------------------------------------------
# PASGD loop  (Section 2, PASGD update rule; Section 4 for the interval scheme)
# --------------------------------------------------------------------------

@dataclass
class PasgdResult:
    params: np.ndarray          # float32 [m][P] at the end
    momentum: np.ndarray        # float32 [m][P]
    loss: np.ndarray            # float64 [K][m] mini-batch loss seen by replica i at iteration k (before its update)
    taus: List[int]             # communication period used by each local-update period
    avg_points: List[int]       # iteration counts k after which an averaging step ran
    F_trace: List[Tuple[int, float, int]]   # AdaComm decisions: (k, F_t, new tau)
    F_0: Optional[float]


def run_pasgd(spec: ModelSpec, x1: np.ndarray, X: np.ndarray, y: np.ndarray, row_offsets: np.ndarray,
              batch: int, lr: float, mu: float, tau: int,
              momentum_mode: str = MOMENTUM_AVERAGE,
              adacomm_interval: Optional[int] = None, probe_rows: int = 0,
              state_hook=None, refined: Optional[dict] = None, block_beta: float = 0.0,
              avg_groups: int = 1) -> PasgdResult:
    """m workers start at the same x_1; each takes local mini-batch steps on its
    own batches; after every tau-th local step (counting from the start of the
    current period) the updated models are replaced by their mean.

    row_offsets[k][i] is the first dataset row of the mini-batch replica i uses
    at iteration k (k = 0..K-1); the batch is rows [off, off + batch).

    Readings taken where the paper is silent, or where this library departs from it (the momentum buffers):
      * the average is taken on the models *after* the tau-th update;
      * momentum buffers follow `momentum_mode`; the default averages them with
        the parameters (which is what makes tau = 1 equal to synchronous
        momentum SGD on the m-fold batch); "keep" is the paper's naive scheme;
      * if K ends inside a period, that period is cut short and averaged;
      * with adacomm_interval = I, the training is cut into intervals of I
        iterations (iteration counts stand in for the paper's wall-clock
        intervals T_0); at the first averaging point with k >= l*I the loss
        F_t of the synchronized model (replica 0) on the first `probe_rows`
        dataset rows is evaluated and tau for the following periods is
        adacomm_next_tau(F_t, F_0, tau_0), where tau_0 = `tau` and F_0 is the
        same loss at x_1.  A period is never cut by an interval boundary.
      * momentum_mode "block" (Section 5.3): the averaging step is block_momentum_average with factor
        `block_beta` on the model the period started from, and the local buffers restart from zero.
      * avg_groups = G > 1: the replicas live on G devices, m / G each, and the averaging step sums in the
        grouped order of average_replicas_grouped (not available with block momentum).
      * refined = {"gamma", "slack", "decay_at": [iterations], "decay_factor"} switches the decision
        to adacomm_next_tau_refined (Section 4.3).  A learning-rate decay scheduled for iteration d
        is applied at the first decision point with k >= d at which the period in force is 1
        (Section 4.3.2: first let the period decay to 1, then decay the rate); one decay per
        decision; the learning rate is kept in float32 as the worker state is.
    """
    K, m = row_offsets.shape
    P = spec.n_params
    xs = np.repeat(np.asarray(x1, dtype=np.float32)[None, :], m, axis=0).copy()
    vs = np.zeros((m, P), dtype=np.float32)
    anchor = np.asarray(x1, dtype=np.float32).copy()       # synchronized model at the period start
    u_glob = np.zeros(P, dtype=np.float32)                  # global block-momentum buffer
    losses = np.zeros((K, m), dtype=np.float64)
    taus: List[int] = []
    avg_points: List[int] = []
    F_trace: List[Tuple[int, float, int]] = []
    F_0 = None
    tau_0 = int(tau)
    cur_tau = int(tau)
    next_interval = 1
    lr_0 = lr
    pending = sorted(int(d) for d in refined.get("decay_at", [])) if refined is not None else []
    lr_trace: List[Tuple[int, float]] = []
    if adacomm_interval is not None:
        F_0 = batch_loss(spec, xs[0], X[:probe_rows], y[:probe_rows])
    k = 0
    while k < K:
        steps = min(cur_tau, K - k)
        taus.append(cur_tau)
        for _ in range(steps):
            for i in range(m):
                r0 = int(row_offsets[k, i])
                loss, g = loss_and_grad(spec, xs[i], X[r0:r0 + batch], y[r0:r0 + batch])
                losses[k, i] = loss
                x_new, v_new = sgd_momentum_step(xs[i], vs[i], g, lr, mu)
                xs[i] = x_new.astype(np.float32)
                vs[i] = v_new.astype(np.float32)
            k += 1
            if state_hook is not None:
                state_hook(k, xs, vs, False)
        if momentum_mode == MOMENTUM_BLOCK and avg_groups > 1:
            raise ValueError("block momentum is defined here on the sequential mean only")
        if momentum_mode == MOMENTUM_BLOCK:
            # Section 5.3: global momentum on the period's accumulated step, local buffers restart
            block_momentum_average(xs, anchor, u_glob, lr, block_beta)
            vs[:] = 0
        elif avg_groups > 1:
            average_replicas_grouped(xs, avg_groups)
            if momentum_mode == MOMENTUM_AVERAGE:
                average_replicas_grouped(vs, avg_groups)
            elif momentum_mode == MOMENTUM_RESET:
                vs[:] = 0
            elif momentum_mode != MOMENTUM_KEEP:
                raise ValueError(momentum_mode)
        else:
            average_replicas(xs)
            if momentum_mode == MOMENTUM_AVERAGE:
                average_replicas(vs)
            elif momentum_mode == MOMENTUM_RESET:
                vs[:] = 0
            elif momentum_mode != MOMENTUM_KEEP:
                raise ValueError(momentum_mode)
        avg_points.append(k)
        if state_hook is not None:
            state_hook(k, xs, vs, True)
        if adacomm_interval is not None and k >= next_interval * adacomm_interval:
            F_t = batch_loss(spec, xs[0], X[:probe_rows], y[:probe_rows])
            if refined is not None:
                changed = False
                if pending and pending[0] <= k and cur_tau == 1:
                    pending.pop(0)
                    lr = float(np.float32(lr * float(refined.get("decay_factor", 0.1))))
                    changed = True
                    lr_trace.append((k, lr))
                cur_tau = adacomm_next_tau_refined(F_t, F_0, tau_0, cur_tau, refined.get("gamma", 0.5),
                                                   refined.get("slack", 0), lr_0, lr, changed)
                F_trace.append((k, F_t, cur_tau))
                next_interval = k // adacomm_interval + 1
                continue
            cur_tau = adacomm_next_tau(F_t, F_0, tau_0)
            F_trace.append((k, F_t, cur_tau))
            next_interval = k // adacomm_interval + 1
    res = PasgdResult(xs, vs, losses, taus, avg_points, F_trace, F_0)
    res.lr_trace = lr_trace
    res.block_u = u_glob
    return res


def tau_schedule_from_trace(F_0: float, tau_0: int, F_values: Sequence[float]) -> List[int]:
    """Recompute the AdaComm decisions from a logged loss trace (Section 4.2)."""
    return [adacomm_next_tau(F, F_0, tau_0) for F in F_values]
