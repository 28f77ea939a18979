"""Host side of a job spread over several GPUs (Section 2: m workers, one exchange per averaging step): which
replicas a rank owns and the rank-ordered exchange of partial sums, run as two gloo ranks on the CPU.  The
arithmetic on either side of the exchange is the oracle's here (the CUDA kernels are checked in
tests/test_gpu_sharded.py)."""
import os

import numpy as np
import pytest

from oracle import localsgd_oracle as orc
from paper_1810_08313_b200 import sharded
from paper_1810_08313_b200 import workloads as wl


def test_shard_range():
    assert [sharded.shard_range(16, 4, r) for r in range(4)] == [(0, 4), (4, 4), (8, 4), (12, 4)]
    assert sharded.shard_range(8, 1, 0) == (0, 8) and sharded.shard_range(8, 8, 7) == (7, 1)
    for bad in [(6, 4, 0), (4, 2, 2), (4, 0, 0), (2, 4, 0), (4, 2, -1)]:
        with pytest.raises(ValueError):
            sharded.shard_range(*bad)


def test_exchange_without_a_process_group_is_the_one_rank_case():
    import torch
    t = torch.arange(6, dtype=torch.float32).view(2, 3)
    g = sharded.exchange_partials(t)
    assert g.shape == (1, 2, 3) and torch.equal(g[0], t)


def _rank_main(rank, world, port, m, P, out):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X = wl.uniform_flat(77, m, P)                       # every rank can regenerate the whole job's state
    first, q = sharded.shard_range(m, world, rank)
    part = X[first].copy()                              # this rank's partial sum, index order, fp32
    for j in range(1, q):
        part = part + X[first + j]
    gathered = sharded.exchange_partials(torch.from_numpy(part)).numpy()
    total = gathered[0].copy()                          # rank order
    for g in range(1, world):
        total = total + gathered[g]
    mean = total / np.float32(m)
    out.put((rank, mean.view(np.uint32).copy(), gathered.shape))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("m", [4, 16])
def test_two_ranks_over_gloo_reach_the_grouped_mean_bit_for_bit(m):
    import torch.multiprocessing as mp
    P, world = 1003, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29600 + (os.getpid() % 2000) + m
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, m, P, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=120) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = wl.uniform_flat(77, m, P)
    orc.average_replicas_grouped(want, world)
    for rank, bits, shape in got:
        assert shape == (world, P)
        assert np.array_equal(bits, want[0].view(np.uint32)), rank      # same bits on every rank
