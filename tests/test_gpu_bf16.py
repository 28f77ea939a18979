"""bf16-GEMM path vs the fp64 oracle: loss trajectory within 2e-2 relative over 3 periods
(Section 2 PASGD update rule; rounding points: inputs, weight copies, hidden activations and dZ in
bf16, everything else fp32)."""
import numpy as np
import pytest

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import workloads as wl
from tests.helpers import f32, max_rel_err_per_tensor, small_problem, to_device

pytestmark = pytest.mark.gpu

BF16_LOSS_TOL = 2e-2


def _run_pair(dims, m, B, tau, K, n_rows, seed, mu=0.9, lr=0.05):
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, n_rows, seed, bf16=True)
    offs = wl.batch_row_offsets(seed, K, m, n_rows, B)
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(lr), f32(mu), tau)
    xd, yd = to_device(X, y, bf16=True)
    eng = LocalSGD(m, dims, gemm_dtype="bf16", lr=lr, momentum=mu, batch=B)
    eng.bind_dataset(xd, yd)
    eng.set_params(x1)
    loss = torch.zeros((K, m), device="cuda")
    out = eng.run(K, tau, offs, loss_out=loss)
    eng.sync()
    got = loss.cpu().numpy()
    p, v = eng.state_view()
    assert bool((p[0:1] == p).all()) and bool((v[0:1] == v).all())
    gx, _ = eng.get_all()
    eng.close()
    return got, ref, gx


@pytest.mark.parametrize("dims,m,B", [
    ((256, 256, 128, 10), 2, 128),          # every hidden layer fills tensor-core tiles
    ((200, 136, 72, 10), 3, 48),            # nothing does: CUDA-core kernels with bf16 operands
    ((384, 256, 256, 256, 10), 4, 256),     # the bf16 workload's depth and batch at reduced width
    ((384, 512, 512, 10), 3, 256),          # 512-wide layers, batch 256: forward / backward on CTA pairs
])
def test_loss_trajectory_three_periods(dims, m, B):
    tau, K = 4, 12
    got, ref, gx = _run_pair(dims, m, B, tau, K, 2048, 17)
    rel = np.abs(got - ref.loss) / ref.loss
    assert rel.max() <= BF16_LOSS_TOL, rel.max()
    # parameters stay close too (the bf16 tolerance is stated on the loss only; this is a loose sanity bound)
    assert max_rel_err_per_tensor(gx[0], ref.params[0], dims, True) < 0.25


def test_full_width_layers_short():
    """3072-2048-2048-2048-10, B = 256 (the bf16 workload's shapes), m = 2, 3 periods of 2 steps."""
    dims = wl.WORKLOADS["c3_mlp_bf16"].dims
    got, ref, _ = _run_pair(dims, 2, 256, 2, 6, 1024, 23)
    rel = np.abs(got - ref.loss) / ref.loss
    assert rel.max() <= BF16_LOSS_TOL, rel.max()


def test_eval_loss_bf16():
    from paper_1810_08313_b200.binding import LocalSGD
    dims = (256, 128, 10)
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 5, bf16=True)
    xd, yd = to_device(X, y, bf16=True)
    eng = LocalSGD(2, dims, gemm_dtype="bf16", lr=0.05, momentum=0.0, batch=128)
    eng.bind_dataset(xd, yd); eng.set_params(x1)
    F = eng.eval_loss(1, 0, 512)
    want = orc.batch_loss(spec, x1, X[:512], y[:512])
    assert abs(F - want) / want <= BF16_LOSS_TOL
    eng.close()


def test_eval_loss_bf16_wide_layers():
    """Forward-only pass through the CTA-pair kernels (512-wide layers, batch 256) with shared weights."""
    from paper_1810_08313_b200.binding import LocalSGD
    dims = (384, 512, 512, 10)
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 7, bf16=True)
    xd, yd = to_device(X, y, bf16=True)
    eng = LocalSGD(3, dims, gemm_dtype="bf16", lr=0.05, momentum=0.9, batch=256)
    eng.bind_dataset(xd, yd); eng.set_params(x1)
    for rows in (256, 768):
        F = eng.eval_loss(2, 0, rows)
        want = orc.batch_loss(spec, x1, X[:rows], y[:rows])
        assert abs(F - want) / want <= BF16_LOSS_TOL, (rows, F, want)
    eng.close()


def _one_step_gradients(dims, m, B, seed=29):
    """Momentum buffers after one step from v = 0 (they equal the stochastic gradient) vs the oracle's gradient."""
    from paper_1810_08313_b200.binding import LocalSGD
    import torch
    from tests.helpers import tensor_slices
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, seed, bf16=True)
    offs = wl.batch_row_offsets(7, 1, m, 1024, B)
    rng = np.random.default_rng(1)
    xs = np.stack([x1 + 0.01 * rng.standard_normal(x1.size).astype(np.float32) for _ in range(m)])
    xd, yd = to_device(X, y, bf16=True)
    eng = LocalSGD(m, dims, gemm_dtype="bf16", lr=0.05, momentum=0.9, batch=B)
    eng.bind_dataset(xd, yd)
    for i in range(m):
        eng.set_state(i, xs[i], np.zeros_like(xs[i]))
    ld = torch.zeros((1, m), device="cuda")
    eng.local_steps(1, offs, ld)
    eng.sync()
    _, gv = eng.get_all()
    eng.close()
    out = []
    for i in range(m):
        r0 = int(offs[0, i])
        loss, g = orc.loss_and_grad(spec, xs[i], X[r0:r0 + B], y[r0:r0 + B])
        assert abs(float(ld[0, i]) - loss) / loss < 5e-3
        for name, s in tensor_slices(dims, True):
            want = g[s]; got = gv[i][s].astype(np.float64)
            err = np.max(np.abs(got - want)) / np.max(np.abs(want))
            cos = float(got @ want / (np.linalg.norm(got) * np.linalg.norm(want)))
            out.append((i, name, err, cos))
    return out


def test_tensor_core_update_kernel_tight():
    """One linear layer 256 -> 128 classes, B = 128: the weight gradient runs on the tensor-core update
    kernel with nothing but bf16 rounding of dZ between it and the oracle, so a tight bound holds.
    (A wrong tile, operand orientation or replica index is off by O(1).)"""
    for i, name, err, cos in _one_step_gradients((256, 128), 3, 128):
        assert err < 1e-2 and cos > 0.99995, (i, name, err, cos)


@pytest.mark.parametrize("dims,m,B", [((256, 256, 128, 10), 2, 128), ((384, 256, 256, 256, 10), 3, 256),
                                      ((256, 128, 128), 2, 128),
                                      ((384, 512, 1024, 10), 3, 256),      # CTA pairs, two and four column tiles
                                      ((256, 512, 512, 10), 2, 512),       # CTA pairs, two row tiles per replica
                                      ((512, 512, 256, 10), 3, 256),       # update on CTA pairs: fewer units than pairs
                                      ((1024, 1024, 10), 5, 256)])         # update on CTA pairs: 80 units, left-over strips
def test_single_step_gradients_through_relu(dims, m, B):
    """All three tensor-core kernels in one step.  bf16 rounding flips a few ReLU masks, which moves single
    entries by O(10 %) of the largest one; the direction of every tensor's gradient is what is checked."""
    for i, name, err, cos in _one_step_gradients(dims, m, B):
        assert cos > 0.995 and err < 0.5, (i, name, err, cos)


@pytest.mark.parametrize("dims,m,B", [((512, 512, 1024, 10), 3, 256), ((1024, 1024, 10), 5, 256)])
def test_cta_pair_kernels_match_one_cta_kernels(dims, m, B, monkeypatch):
    """The CTA-pair GEMM and update kernels against the one-CTA kernels they replace (LS_DISABLE_PAIR=1), one
    step from the same state: the same products in the same order, so weights and their momentum must agree far
    more tightly than either agrees with the fp64 oracle.  (The bias gradient of a hidden layer is summed from
    the bf16-rounded dZ in the pair kernel and from the unrounded values in the one-CTA kernel: biases get a
    looser bound.)"""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    from tests.helpers import tensor_slices
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 31, bf16=True)
    offs = wl.batch_row_offsets(9, 1, m, 1024, B)
    xd, yd = to_device(X, y, bf16=True)
    out = {}
    for tag, val in (("pair", "0"), ("one", "1")):
        monkeypatch.setenv("LS_DISABLE_PAIR", val)
        eng = LocalSGD(m, dims, gemm_dtype="bf16", lr=0.05, momentum=0.9, batch=B)
        eng.bind_dataset(xd, yd); eng.set_params(x1)
        ld = torch.zeros((1, m), device="cuda")
        eng.local_steps(1, offs, ld)
        eng.sync()
        out[tag] = eng.get_all() + (ld.cpu().numpy(),)
        eng.close()
    (px, pv, pl), (ox, ov, ol) = out["pair"], out["one"]
    assert np.max(np.abs(pl - ol) / np.abs(ol)) < 1e-5
    for i in range(m):
        for name, sl in tensor_slices(dims, True):
            tol = 2e-2 if name.startswith("b") else 1e-5
            for a, b in ((px[i][sl], ox[i][sl]), (pv[i][sl], ov[i][sl])):
                err = np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30)
                assert err < tol, (i, name, err)



@pytest.mark.parametrize("dims,m,B,has_bias,mu", [
    ((512, 512, 1024, 10), 3, 256, True, 0.9), ((256, 384, 10), 5, 64, True, 0.9), ((384, 2048, 10), 2, 32, True, 0.9),
    ((256, 128, 10), 17, 256, True, 0.9),
    ((256, 512, 10), 3, 256, False, 0.9),         # no biases: nothing to finish for them
    ((256, 512, 10), 3, 128 + 64, True, 0.0),     # no momentum buffers; 24 rows per CTA
])
def test_one_launch_output_layer_matches_two_kernels(dims, m, B, has_bias, mu, monkeypatch):
    """The output layer of a training step as one launch (clusters of four CTAs, two per replica) against the
    forward + backward kernels it replaces (LS_DISABLE_HEAD_STEP=1), three steps from the same state.  Both
    compute the same fp32 products; only the order of the sums differs, so the output layer's weights, both
    biases and the first loss agree to fp32 rounding; dZ of the layer below is stored in bf16, where a different
    last bit of a sum can flip a rounding, so the layers below (and, from the second step on, everything) get the
    bound of one bf16 step on a few elements.
    Shapes: 32, 8 and 4 rows per CTA, one and several column groups per thread, more replicas than fit one round."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    from tests.helpers import tensor_slices
    spec, X, y, x1 = small_problem(dims, "softmax_ce", has_bias, 1024, 37, bf16=True)
    steps = 3
    offs = wl.batch_row_offsets(11, steps, m, 1024, B)
    xd, yd = to_device(X, y, bf16=True)
    out = {}
    for tag, val in (("one", "0"), ("two", "1")):
        monkeypatch.setenv("LS_DISABLE_HEAD_STEP", val)
        eng = LocalSGD(m, dims, has_bias=has_bias, gemm_dtype="bf16", lr=0.05, momentum=mu, batch=B)
        eng.bind_dataset(xd, yd); eng.set_params(x1)
        ld = torch.zeros((steps, m), device="cuda")
        n0 = eng.launch_count()
        eng.local_steps(steps, offs, ld)
        eng.sync()
        out[tag] = eng.get_all() + (ld.cpu().numpy(), eng.launch_count() - n0)
        eng.close()
    (px, pv, pl, pn), (ox, ov, ol, on) = out["one"], out["two"]
    assert pn < on, (pn, on)                      # the one-launch path really ran: fewer launches per step
    assert np.max(np.abs(pl[0] - ol[0]) / np.abs(ol[0])) < 1e-5     # first step: the same inputs, fp32 sums
    assert np.max(np.abs(pl - ol) / np.abs(ol)) < 2e-3
    L = len(dims) - 1
    for i in range(m):
        for name, sl in tensor_slices(dims, has_bias):
            tol = 2e-3 if name in (f"W{L}", f"b{L}") else 2e-2
            for a, b in ((px[i][sl], ox[i][sl]), (pv[i][sl], ov[i][sl])):
                err = np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30)
                assert err < tol, (i, name, err)
