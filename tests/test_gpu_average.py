"""Averaging kernel vs the oracle: bit-exact (Section 2, PASGD update rule, case k mod tau = 0)."""
import numpy as np
import pytest

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run(m, P, stride=None, seed=1, offset_floats=0):
    import torch
    from paper_1810_08313_b200 import binding
    stride = P if stride is None else stride
    host = wl.uniform_flat(seed, m, stride)
    want = host[:, :P].copy()
    orc.average_replicas(want)
    raw = torch.zeros(m * stride + offset_floats + 8, dtype=torch.float32, device="cuda")
    buf = raw[offset_floats:offset_floats + m * stride]
    buf.copy_(torch.from_numpy(host.reshape(-1)))
    binding.average_flat(buf, m, P, stride)
    torch.cuda.synchronize()
    got = buf.cpu().numpy().reshape(m, stride)
    assert np.array_equal(got[:, :P].view(np.uint32), want.view(np.uint32))
    # padding between vectors is untouched
    assert np.array_equal(got[:, P:].view(np.uint32), host[:, P:].view(np.uint32))


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 8, 16, 17, 32, 64])
def test_bit_exact_all_replica_counts(m):
    _run(m, 100_003)


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 7, 1023, 1024, 1025, 262_147])
def test_ragged_sizes(P):
    _run(4, P)


def test_empty_is_a_no_op():
    _run(4, 0, stride=8)


def test_strided_and_padded_replicas():
    _run(8, 1000, stride=1024)
    _run(8, 1001, stride=1028)


def test_unaligned_buffers_take_the_scalar_path():
    _run(4, 1001, stride=1001)            # stride not a multiple of 4
    _run(4, 1000, stride=1000, offset_floats=1)   # base not 16-byte aligned


def test_several_tiles_per_thread():
    # more float4 columns than one pass of the grid covers
    _run(16, 148 * 4 * 256 * 4 * 3 + 2)


def test_model_sized_vector_with_tail():
    # P of the 3072-2048-2048-2048-10 network: P mod 4 == 2
    P = 14_706_698
    assert P % 4 == 2
    _run(4, P)


def test_invalid_arguments():
    import torch
    from paper_1810_08313_b200 import binding
    buf = torch.zeros(64, dtype=torch.float32, device="cuda")
    lib = binding._lib()
    assert lib.ls_average_flat(None, 4, 16, 16, None) == binding.LS_ERR_INVALID_ARG
    assert lib.ls_average_flat(buf.data_ptr(), 0, 16, 16, None) == binding.LS_ERR_INVALID_ARG
    assert lib.ls_average_flat(buf.data_ptr(), 4, 16, 8, None) == binding.LS_ERR_INVALID_ARG
    assert lib.ls_average_flat(buf.data_ptr(), 4, -1, 16, None) == binding.LS_ERR_INVALID_ARG


def test_full_size_sampled_columns():
    """Largest sweep point that fits comfortably: m = 16, P = 23.5 M (1.5 GB), checked on sampled columns."""
    import torch
    from paper_1810_08313_b200 import binding
    m, P = 16, 23_500_000
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    buf = torch.rand((m, P), generator=g, device="cuda", dtype=torch.float32) * 2 - 1
    idx = np.unique(np.concatenate([np.arange(0, 64), np.arange(P - 64, P),
                                    np.random.default_rng(0).integers(0, P, 4096)]))
    before = buf[:, torch.from_numpy(idx).cuda()].cpu().numpy().copy()
    binding.average_flat(buf, m, P)
    torch.cuda.synchronize()
    after = buf[:, torch.from_numpy(idx).cuda()].cpu().numpy()
    want = np.ascontiguousarray(before)
    orc.average_replicas(want)
    assert np.array_equal(after.view(np.uint32), want.view(np.uint32))
    # property at full size: all replicas equal
    assert bool((buf[0:1] == buf).all())


# ---- block momentum (Section 5.3): the same pass with the period-start model and the global buffer ----

def _run_block(m, P, stride=None, seed=3, offset_floats=0, lr=0.05, beta=0.3):
    import torch
    from paper_1810_08313_b200 import binding
    stride = P if stride is None else stride
    host = wl.uniform_flat(seed, m, stride)
    extra = wl.uniform_flat(seed + 100, 2, max(P, 1))
    anchor, u = extra[0, :P].copy(), extra[1, :P].copy()
    want, want_a, want_u = host[:, :P].copy(), anchor.copy(), u.copy()
    orc.block_momentum_average(want, want_a, want_u, float(np.float32(lr)), float(np.float32(beta)))
    raw = torch.zeros(m * stride + offset_floats + 8, dtype=torch.float32, device="cuda")
    buf = raw[offset_floats:offset_floats + m * stride]
    buf.copy_(torch.from_numpy(host.reshape(-1)))
    a_raw = torch.zeros(P + offset_floats + 8, dtype=torch.float32, device="cuda")
    u_raw = torch.zeros(P + offset_floats + 8, dtype=torch.float32, device="cuda")
    a_dev, u_dev = a_raw[offset_floats:offset_floats + P], u_raw[offset_floats:offset_floats + P]
    a_dev.copy_(torch.from_numpy(anchor)); u_dev.copy_(torch.from_numpy(u))
    # an empty slice has no address: hand the (unused) allocation over instead
    binding.block_average_flat(buf, a_dev if P else a_raw, u_dev if P else u_raw, m, P, lr, beta, stride)
    torch.cuda.synchronize()
    got = buf.cpu().numpy().reshape(m, stride)
    assert np.array_equal(got[:, :P].view(np.uint32), want.view(np.uint32))
    assert np.array_equal(got[:, P:].view(np.uint32), host[:, P:].view(np.uint32))
    assert np.array_equal(a_dev.cpu().numpy().view(np.uint32), want_a.view(np.uint32))
    assert np.array_equal(u_dev.cpu().numpy().view(np.uint32), want_u.view(np.uint32))
    # nothing written past the vectors
    assert float(a_raw[offset_floats + P:].abs().sum()) == 0.0 and float(u_raw[offset_floats + P:].abs().sum()) == 0.0


@pytest.mark.parametrize("m", [1, 2, 3, 4, 8, 16, 17, 64])
def test_block_momentum_bit_exact_all_replica_counts(m):
    _run_block(m, 100_003)


@pytest.mark.parametrize("P", [1, 3, 4, 7, 8, 9, 1025, 262_147])
def test_block_momentum_ragged_sizes(P):
    _run_block(4, P)


def test_block_momentum_alignment_paths_and_factors():
    _run_block(8, 1000, stride=1024)                      # 256-bit path, padded
    _run_block(8, 1004, stride=1028)                      # 128-bit path
    _run_block(4, 1001, stride=1001)                      # scalar path
    _run_block(4, 1000, stride=1000, offset_floats=1)     # unaligned bases
    _run_block(4, 4096, beta=0.0)
    _run_block(4, 4096, lr=0.4, beta=0.9)
    _run_block(4, 0, stride=8)


def test_block_momentum_invalid_arguments():
    import torch
    from paper_1810_08313_b200 import binding
    buf = torch.zeros(64, dtype=torch.float32, device="cuda")
    a = torch.zeros(16, dtype=torch.float32, device="cuda")
    lib = binding._lib()
    bad = binding.LS_ERR_INVALID_ARG
    assert lib.ls_block_average_flat(buf.data_ptr(), None, a.data_ptr(), 4, 16, 16, 0.1, 0.3, None) == bad
    assert lib.ls_block_average_flat(buf.data_ptr(), a.data_ptr(), a.data_ptr(), 4, 16, 16, 0.0, 0.3, None) == bad
    assert lib.ls_block_average_flat(buf.data_ptr(), a.data_ptr(), a.data_ptr(), 4, 16, 16, 0.1, -0.5, None) == bad
    assert lib.ls_block_average_flat(buf.data_ptr(), a.data_ptr(), a.data_ptr(), 4, 16, 8, 0.1, 0.3, None) == bad
