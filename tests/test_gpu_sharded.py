"""Averaging of a job whose replicas are spread over several GPUs (Section 2; grouped summation order), on ONE
GPU: the two kernels on raw buffers, the handle path, and two ranks emulated by two handles whose partial sums
are put side by side by the test (no kernel waits on another, so running them one after the other is the same
computation)."""
import numpy as np
import pytest

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import workloads as wl
from tests.helpers import f32, max_rel_err_per_tensor, small_problem, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,G", [(4, 1), (4, 2), (8, 2), (8, 4), (16, 4), (16, 16), (6, 3), (24, 2)])
@pytest.mark.parametrize("P", [100_003, 4096, 5])
def test_flat_kernels_match_the_grouped_order_bit_for_bit(m, G, P):
    import torch
    from paper_1810_08313_b200 import binding
    stride = (P + 63) // 64 * 64
    X = wl.uniform_flat(3, m, P)
    want = X.copy(); orc.average_replicas_grouped(want, G)
    q = m // G
    buf = torch.full((m, stride), 7.0, dtype=torch.float32, device="cuda")       # padding must stay untouched
    buf[:, :P] = torch.from_numpy(X).cuda()
    parts = torch.full((G, stride), -3.0, dtype=torch.float32, device="cuda")
    for g in range(G):                                                           # "rank" g: its own replicas only
        binding.partial_sum_flat(buf[g * q:(g + 1) * q].view(-1), q, P, parts[g], stride)
    for g in range(G):
        binding.combine_partials_flat(parts.view(-1), G, stride, m, P, buf[g * q:(g + 1) * q].view(-1), q, stride)
    torch.cuda.synchronize()
    got = buf.cpu().numpy()
    assert np.array_equal(got[:, :P].view(np.uint32), want.view(np.uint32))
    assert np.all(got[:, P:] == 7.0) and bool((parts[:, P:] == -3.0).all())


def test_flat_argument_checks():
    import torch
    from paper_1810_08313_b200 import binding
    lib = binding._lib()
    t = torch.zeros(1024, device="cuda")
    assert lib.ls_partial_sum_flat(None, 2, 8, 8, t.data_ptr(), None) == binding.LS_ERR_INVALID_ARG
    assert lib.ls_partial_sum_flat(t.data_ptr(), 0, 8, 8, t.data_ptr(), None) == binding.LS_ERR_INVALID_ARG
    assert lib.ls_partial_sum_flat(t.data_ptr(), 2, 8, 4, t.data_ptr(), None) == binding.LS_ERR_INVALID_ARG      # stride < P
    assert lib.ls_partial_sum_flat(t.data_ptr() + 4, 2, 8, 8, t.data_ptr(), None) == binding.LS_ERR_INVALID_ARG  # alignment
    assert lib.ls_combine_partials_flat(t.data_ptr(), 2, 8, 1, 8, t.data_ptr(), 2, 8, None) == binding.LS_ERR_INVALID_ARG


@pytest.mark.parametrize("gemm,mode,mu", [("fp32", "average", 0.9), ("bf16", "average", 0.9), ("fp32", "keep", 0.9),
                                          ("fp32", "reset", 0.9), ("fp32", "average", 0.0)])
def test_one_gpu_share_equals_the_plain_average(gemm, mode, mu):
    """n_gpus = 1 is the sequential order: ls_average() on a handle declared as the only share of its job gives
    the bits of the plain averaging kernel, for parameters, momentum and the bf16 copies (seen through a loss)."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B = (256, 128, 10), 4, 128
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 9, bf16=(gemm == "bf16"))
    xd, yd = to_device(X, y, bf16=(gemm == "bf16"))
    st = wl.uniform_flat(8, 2 * m, spec.n_params) * np.float32(0.1)
    res = []
    for shard in (False, True):
        eng = LocalSGD(m, dims, gemm_dtype=gemm, lr=0.05, momentum=mu, batch=B, momentum_mode=mode)
        eng.bind_dataset(xd, yd)
        for i in range(m):
            eng.set_state(i, st[i], st[m + i])
        if shard:
            eng.set_shard(1, m, torch.zeros(eng.shard_buffer_floats(), device="cuda"))
        eng.average()
        eng.sync()
        px, pv = eng.get_all()
        res.append((px, pv, eng.eval_loss(m - 1, 0, 2 * B)))
        eng.close()
    assert np.array_equal(res[0][0].view(np.uint32), res[1][0].view(np.uint32))
    assert np.array_equal(res[0][1].view(np.uint32), res[1][1].view(np.uint32))
    assert res[0][2] == res[1][2]


def test_block_momentum_is_refused_on_several_gpus():
    import torch
    from paper_1810_08313_b200 import binding
    from paper_1810_08313_b200.binding import LocalSGD, LsError
    eng = LocalSGD(2, (16, 8), batch=8, momentum_mode="block", block_momentum=0.3)
    with pytest.raises(LsError) as e:
        eng.set_shard(1, 2, torch.zeros(eng.shard_buffer_floats(), device="cuda"))
    assert e.value.code == binding.LS_ERR_UNSUPPORTED
    eng.close()
    eng = LocalSGD(2, (16, 8), batch=8)
    with pytest.raises(LsError):
        eng.set_shard(2, 5, torch.zeros(eng.shard_buffer_floats(), device="cuda"))      # m_total != n_gpus * m
    with pytest.raises(LsError):
        eng.set_shard(2, 4, torch.zeros(eng.shard_buffer_floats(), device="cuda"))      # two GPUs need an exchange
    eng.close()


@pytest.mark.parametrize("gemm", ["fp32", "bf16"])
def test_exchange_callback_inside_the_averaging_step(gemm):
    """The callback path of ls_set_shard with n_gpus = 2: this handle is rank 0 of a two-rank job; the test's
    callback plays the all-gather and supplies rank 1's partial sums from replicas it made up.  The result is
    the oracle's grouped mean over all four replicas, bit for bit, through ls_average and ls_local_steps_avg."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m, B = (256, 128, 10), 2, 128
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 9, bf16=(gemm == "bf16"))
    xd, yd = to_device(X, y, bf16=(gemm == "bf16"))
    P = spec.n_params
    st = wl.uniform_flat(18, 4 * m, P) * np.float32(0.1)       # params of ranks 0, 1 then momentum of ranks 0, 1
    eng = LocalSGD(m, dims, gemm_dtype=gemm, lr=0.05, momentum=0.9, batch=B)
    eng.bind_dataset(xd, yd)
    for i in range(m):
        eng.set_state(i, st[i], st[2 * m + i])
    n = eng.shard_buffer_floats()
    stride = n // 2
    partial = torch.zeros(n, device="cuda")
    gathered = torch.zeros(2 * n, device="cuda")
    # rank 1's partial sums, in the padded device layout, taken from a scratch handle holding rank 1's replicas
    other = LocalSGD(m, dims, gemm_dtype=gemm, lr=0.05, momentum=0.9, batch=B)
    for i in range(m):
        other.set_state(i, st[m + i], st[3 * m + i])
    other_partial = torch.zeros(n, device="cuda")
    other.shard_partial_sum(other_partial)
    other.sync()
    calls = []

    def fake_all_gather(partial_ptr, gathered_ptr, nbytes, n_gpus):
        calls.append((partial_ptr == partial.data_ptr(), gathered_ptr == gathered.data_ptr(), nbytes, n_gpus))
        with torch.cuda.stream(eng.stream):
            gathered[:n].copy_(partial); gathered[n:].copy_(other_partial)
        return 0

    eng.set_shard(2, 2 * m, partial, gathered, fake_all_gather)
    eng.average()
    eng.sync()
    assert calls == [(True, True, n * 4, 2)]
    wx = np.ascontiguousarray(st[:2 * m]); wv = np.ascontiguousarray(st[2 * m:])
    orc.average_replicas_grouped(wx, 2); orc.average_replicas_grouped(wv, 2)
    gx, gv = eng.get_all()
    for i in range(m):
        assert np.array_equal(gx[i].view(np.uint32), wx[0].view(np.uint32))
        assert np.array_equal(gv[i].view(np.uint32), wv[0].view(np.uint32))
    # a whole period in one call goes through the same exchange
    eng.local_steps(2, wl.batch_row_offsets(1, 2, m, 1024, B), average=True)
    eng.sync()
    assert len(calls) == 2
    # a failing exchange is reported, not swallowed
    from paper_1810_08313_b200 import binding
    eng.set_shard(2, 2 * m, partial, gathered, lambda *a: 1)
    with pytest.raises(binding.LsError) as e:
        eng.average()
    assert e.value.code == binding.LS_ERR_EXCHANGE
    eng.set_shard(0, 0)
    eng.average(); eng.sync()
    eng.close(); other.close()


@pytest.mark.parametrize("G", [2, 4])
def test_two_and_four_emulated_ranks_follow_the_oracle(G):
    """G handles on one GPU stand for G ranks (m_total / G replicas each).  Every period: local steps on each,
    partial sums of each, the gathered buffer filled in rank order, the combining kernel on each.  Against
    run_pasgd(avg_groups=G): all replicas of all handles bitwise equal after every average, parameters and
    momentum within the free-running bound, losses per step."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    dims, m_total, B, tau, K = (96, 64, 48, 10), 8, 32, 3, 9
    spec, X, y, x1 = small_problem(dims, "softmax_ce", True, 1024, 23)
    offs = wl.batch_row_offsets(6, K, m_total, 1024, B)
    ref = orc.run_pasgd(spec, x1, X, y, offs, B, f32(0.05), f32(0.9), tau, avg_groups=G)
    xd, yd = to_device(X, y)
    q = m_total // G
    engs = []
    for g in range(G):
        e = LocalSGD(q, dims, lr=0.05, momentum=0.9, batch=B); e.bind_dataset(xd, yd); e.set_params(x1)
        engs.append(e)
    n = engs[0].shard_buffer_floats()
    gathered = torch.zeros(G * n, device="cuda")
    losses = [torch.zeros((K, q), device="cuda") for _ in range(G)]
    for k0 in range(0, K, tau):
        for g, e in enumerate(engs):
            e.local_steps(tau, np.ascontiguousarray(offs[k0:k0 + tau, g * q:(g + 1) * q]), losses[g][k0:k0 + tau])
        for g, e in enumerate(engs):
            e.shard_partial_sum(gathered[g * n:(g + 1) * n])
        torch.cuda.synchronize()
        for e in engs:
            e.shard_average(gathered, G, m_total)
        torch.cuda.synchronize()
        views = [e.state_view() for e in engs]
        p0, v0 = views[0][0][0], views[0][1][0]
        for p, v in views:
            assert bool((p == p0[None]).all()) and bool((v == v0[None]).all())
    for g, e in enumerate(engs):
        gx, gv = e.get_all()
        for i in range(q):
            assert max_rel_err_per_tensor(gx[i], ref.params[g * q + i], dims, True) <= 1e-4
            assert max_rel_err_per_tensor(gv[i], ref.momentum[g * q + i], dims, True) <= 1e-3
        got = losses[g].cpu().numpy()
        want = ref.loss[:, g * q:(g + 1) * q]
        assert np.max(np.abs(got - want) / want) <= 1e-4
        e.close()
