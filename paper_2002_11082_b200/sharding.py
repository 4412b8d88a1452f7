"""Host-side logic for running the path on several GPUs.

Two ways to use more than one GPU, both without any arithmetic here:

* replicas (weak scaling, what ``bench.py --gpus N`` times): every rank quantizes its own workers'
  buckets and the ranks only meet for timing (``worker_ids``, ``max_over_ranks``,
  ``aggregate_throughput``);
* data parallelism as in Algorithm 2 (each rank is one worker): because every worker has its own
  levels, codes cannot be added in transit, so the exchange is an all-gather of the packed codes and
  the level tables into every rank's own memory (``CodeExchange``), followed by a local
  ``ogq_unpack_sum`` over the gathered buffers.  The gathered data is read from local HBM by ordinary
  loads; nothing here reads a peer's memory from a kernel.

Everything works with any torch.distributed backend, which lets the CPU tests cover it with gloo.
"""
from __future__ import annotations

from typing import List, Tuple


def worker_ids(rank: int, workers_per_rank: int) -> List[int]:
    """Global ids (= data seeds) of the simulated workers that `rank` owns; disjoint across ranks."""
    return [rank * workers_per_rank + k for k in range(workers_per_rank)]


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's value (a step time): what a multi-GPU throughput has to be computed from."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(bytes_per_rank: float, ms_per_step_max: float, world_size: int) -> float:
    """Whole-job GB/s: every rank moved `bytes_per_rank` in the time of the slowest rank."""
    return world_size * bytes_per_rank / (ms_per_step_max * 1e-3) / 1e9


class CodeExchange:
    """Receive buffers and bookkeeping of the all-gather of Algorithm 2's "encode ... send / receive and
    decode" step: after ``gather`` every rank holds all ranks' packed words and level tables, rank k's
    at row k, and ``pointer_rows`` gives the per-worker addresses ``ogq_unpack_sum`` takes.

    packed_words: words of one worker's packed buffer (ogq_packed_layout(...)[-1]); num_tensors, levels:
    shape of one worker's level table.  Bytes each rank receives per step: ``recv_bytes``.
    """

    def __init__(self, world_size: int, packed_words: int, num_tensors: int, levels: int, device=None):
        import torch

        self.world = int(world_size)
        self.packed_words = int(packed_words)
        self.level_count = int(num_tensors) * int(levels)
        self.all_packed = torch.zeros((self.world, max(self.packed_words, 1)), dtype=torch.int32, device=device)
        self.all_levels = torch.zeros((self.world, max(self.level_count, 1)), dtype=torch.float32, device=device)

    @property
    def recv_bytes(self) -> int:
        return (self.world - 1) * 4 * (self.packed_words + self.level_count)

    def gather(self, dist, packed, levels) -> None:
        """All-gathers this rank's packed words and level table (contiguous tensors on the exchange's
        device) into the receive buffers.  With one rank it is a local copy."""
        if self.world == 1 or dist is None or not dist.is_initialized():
            self.all_packed[0, : self.packed_words].copy_(packed.reshape(-1)[: self.packed_words])
            self.all_levels[0, : self.level_count].copy_(levels.reshape(-1)[: self.level_count])
            return
        if self.packed_words:
            dist.all_gather_into_tensor(self.all_packed.view(-1), packed.reshape(-1)[: self.packed_words].contiguous())
        if self.level_count:
            dist.all_gather_into_tensor(self.all_levels.view(-1), levels.reshape(-1)[: self.level_count].contiguous())

    def pointer_rows(self) -> Tuple[List[int], List[int]]:
        """Addresses of every worker's packed words and level table inside the receive buffers."""
        pk = [self.all_packed.data_ptr() + k * self.all_packed.stride(0) * 4 for k in range(self.world)]
        lv = [self.all_levels.data_ptr() + k * self.all_levels.stride(0) * 4 for k in range(self.world)]
        return pk, lv
