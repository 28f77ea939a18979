"""One local-update SGD job whose replicas are spread over several GPUs, one process per GPU.

The m replicas of the job are dealt out in index order, m / G consecutive ones per rank (Section 2 of the paper:
m workers whose models are averaged by an all-node exchange).  Local steps need no communication; each averaging
step exchanges ONE partial sum per rank (an all-gather over the process group: NCCL on GPUs) and is finished by the
library's kernels in a fixed, rank-ordered summation, so every rank holds the same bits afterwards.

This module is plumbing only: which replicas a rank owns, and the all-gather that the library calls back into.
All arithmetic runs in the CUDA library (ls_set_shard / ls_shard_partial_sum / ls_shard_average).
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import numpy as np


def shard_range(m_total: int, n_ranks: int, rank: int) -> Tuple[int, int]:
    """(first replica, number of replicas) of `rank`: consecutive blocks of m_total / n_ranks replicas."""
    m_total, n_ranks, rank = int(m_total), int(n_ranks), int(rank)
    if n_ranks < 1 or not (0 <= rank < n_ranks) or m_total < n_ranks or m_total % n_ranks != 0:
        raise ValueError("the replicas must divide evenly over the ranks")
    q = m_total // n_ranks
    return rank * q, q


def exchange_partials(local, gathered=None, group=None):
    """All-gather of one tensor per rank, in rank order: returns a tensor [world][...local.shape] in which entry g
    is rank g's `local` (this rank's own included).  `gathered` may be a preallocated output.  Works on CUDA
    tensors over NCCL and on CPU tensors over gloo; without an initialised process group it is the one-rank case."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        out = local.unsqueeze(0).clone() if gathered is None else gathered
        if gathered is not None:
            out.view(1, *local.shape).copy_(local.unsqueeze(0))
        return out.view(1, *local.shape)
    world = dist.get_world_size(group)
    if gathered is None:
        gathered = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    flat = gathered.view(world, -1)
    if local.is_cuda:
        dist.all_gather_into_tensor(flat.view(-1), local.contiguous().view(-1), group=group)
    else:
        parts = [flat[g] for g in range(world)]
        dist.all_gather(parts, local.contiguous().view(-1), group=group)
    return gathered.view(world, *local.shape)


class ShardedLocalSGD:
    """This rank's share of a job of m_total replicas.  Same calls as LocalSGD; row offsets are given for the
    whole job ([.][m_total]) and every rank uses its own columns.  Every rank must make the same calls in the
    same order (the averaging step is collective)."""

    def __init__(self, m_total: int, dims: Sequence[int], loss: str = "softmax_ce", has_bias: bool = True,
                 gemm_dtype: str = "fp32", lr: float = 0.05, momentum: float = 0.0, batch: int = 32,
                 momentum_mode: str = "average", device: Optional[str] = None, group=None):
        import torch
        import torch.distributed as dist
        from .binding import LocalSGD
        self._torch = torch
        self.group = group
        on = dist.is_available() and dist.is_initialized()
        self.world = dist.get_world_size(group) if on else 1
        self.rank = dist.get_rank(group) if on else 0
        self.m_total = int(m_total)
        self.first, self.m = shard_range(m_total, self.world, self.rank)
        if device is None:
            device = f"cuda:{torch.cuda.current_device()}"
        self.eng = LocalSGD(self.m, dims, loss, has_bias, gemm_dtype, lr=lr, momentum=momentum, batch=batch,
                            momentum_mode=momentum_mode, device=device)
        n = self.eng.shard_buffer_floats()
        # 256-byte aligned device buffers (torch's caching allocator returns 512-byte aligned blocks)
        self.partial = torch.zeros(n, dtype=torch.float32, device=device)
        self.gathered = torch.zeros(self.world * n, dtype=torch.float32, device=device) if self.world > 1 else None
        self.eng.set_shard(self.world, self.m_total, self.partial, self.gathered,
                           self._exchange if self.world > 1 else None)

    def _exchange(self, partial_ptr, gathered_ptr, nbytes, n_gpus) -> int:
        """Called by the library inside an averaging step, after it has enqueued the partial-sum kernel."""
        try:
            torch = self._torch
            n = nbytes // 4
            # the collective is enqueued relative to the handle's stream: NCCL waits for the work already on the
            # current stream and the current stream waits for the collective
            with torch.cuda.stream(self.eng.stream):
                exchange_partials(self.partial[:n], self.gathered[:n_gpus * n].view(n_gpus, n), self.group)
            return 0
        except Exception:           # never let an exception cross the C boundary
            return 1

    def _mine(self, row_offsets: np.ndarray) -> np.ndarray:
        offs = np.asarray(row_offsets, dtype=np.int64)
        if offs.ndim != 2 or offs.shape[1] != self.m_total:
            raise ValueError("row_offsets must be [steps][m_total]")
        return np.ascontiguousarray(offs[:, self.first:self.first + self.m])

    def bind_dataset(self, x, y):
        self.eng.bind_dataset(x, y)

    def set_params(self, x1):
        self.eng.set_params(x1)

    def local_steps(self, tau: int, row_offsets, loss_out=None, average: bool = False):
        self.eng.local_steps(tau, self._mine(row_offsets), loss_out, average=average)

    def average(self):
        self.eng.average()

    def eval_loss(self, replica: int, row_offset: int, n_rows: int) -> float:
        return self.eng.eval_loss(replica, row_offset, n_rows)

    def run(self, K: int, tau_0: int, row_offsets, interval: int = 0, probe_rows: int = 0, loss_out=None):
        """The native run loop on this rank's share; every rank reaches the same AdaComm decisions because every
        rank evaluates the same synchronized model on the same probe rows."""
        return self.eng.run(K, tau_0, self._mine(row_offsets), interval=interval, probe_rows=probe_rows,
                            loss_out=loss_out)

    def sync(self):
        self.eng.sync()

    def get_state(self, replica: int):
        return self.eng.get_state(replica)

    def close(self):
        self.eng.close()
