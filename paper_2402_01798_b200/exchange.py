"""Host-side plumbing for running the path with the N workers spread over several GPUs.

In a data-parallel job GPU r holds the gradients of some of the N workers (Algorithm 1's clients).  Each
rank compresses its own workers' rows; the one exchange step of the path is that every rank then needs
all N packed rows and all N parameter records to form the averaged update (Algorithm 1, aggregation
step).  This module holds what that needs on the host and nothing of the method's arithmetic:

  * which workers a rank owns (``worker_slice``);
  * the all-gather of the small parameter records and of the packed rows through ``torch.distributed``
    (NCCL on GPUs, gloo in the CPU tests) -- the gathered rows land in local memory and the ordinary
    ``tq_decompress_aggregate`` runs on them;
  * ``PeerRows``: the packed rows placed in symmetric memory so that every rank can hand the peers' row
    ADDRESSES to ``tq_decompress_aggregate_rows``; the aggregation kernel then pulls each row over NVLink
    while it aggregates and no gathered copy of the rows is ever written.  Every rank issues its own plain loads.

Rows are always presented to the aggregation in global worker order, so the result does not depend on
how many ranks there are.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def worker_slice(rank: int, world: int, n_workers: int) -> Tuple[int, int]:
    """(first worker, count) of the contiguous block of workers that `rank` owns; blocks differ by at most one."""
    if not (0 <= rank < world) or n_workers < 0:
        raise ValueError("rank outside the world, or a negative worker count")
    base, extra = divmod(n_workers, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def all_worker_slices(world: int, n_workers: int) -> List[Tuple[int, int]]:
    return [worker_slice(r, world, n_workers) for r in range(world)]


def gather_worker_rows(local: torch.Tensor, n_workers: int, group=None) -> torch.Tensor:
    """All-gather of per-worker rows.  `local` is [count, width] (this rank's workers, any dtype, CPU or CUDA);
    returns [n_workers, width] in global worker order on every rank.  Ranks may own different counts."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    slices = all_worker_slices(world, n_workers)
    first, count = slices[rank]
    if local.dim() != 2 or local.shape[0] != count:
        raise ValueError(f"rank {rank} owns {count} workers but passed {tuple(local.shape)}")
    most = max(c for _, c in slices)
    width = local.shape[1]
    padded = local.new_zeros((most, width))
    padded[:count] = local
    parts = [local.new_empty((most, width)) for _ in range(world)]
    dist.all_gather(parts, padded.contiguous(), group=group)
    out = local.new_empty((n_workers, width))
    for r, (f, c) in enumerate(slices):
        out[f:f + c] = parts[r][:c]
    return out


class PeerRows:
    """This rank's packed rows in symmetric memory, and the addresses of every rank's rows.

    GPU only (NCCL process group, peer access between the GPUs).  ``local`` is where ``tq_compress`` writes
    this rank's rows; ``row_addresses()`` lists all N rows' device addresses in global worker order for
    ``tq_decompress_aggregate_rows``.  ``ready()`` must separate the writes of a round from the peers' reads,
    and ``done()`` the reads from the next round's writes (both are barriers across the group).
    """

    def __init__(self, n_workers: int, words: int, device, group=None):
        import torch.distributed._symmetric_memory as symm
        self.group = group if group is not None else dist.group.WORLD
        self.world = dist.get_world_size(self.group)
        self.rank = dist.get_rank(self.group)
        self.n_workers, self.words = n_workers, words
        self.slices = all_worker_slices(self.world, n_workers)
        most = max(c for _, c in self.slices)
        self.buffer = symm.empty((most, words), dtype=torch.int32, device=device)
        self.handle = symm.rendezvous(self.buffer, self.group.group_name)
        self.local = self.buffer[: self.slices[self.rank][1]]

    def row_addresses(self) -> List[int]:
        row_bytes = self.words * 4
        out = []
        for r, (_, c) in enumerate(self.slices):
            base = int(self.handle.buffer_ptrs[r])
            out.extend(base + k * row_bytes for k in range(c))
        return out

    def ready(self):
        self.handle.barrier()

    def done(self):
        self.handle.barrier()
