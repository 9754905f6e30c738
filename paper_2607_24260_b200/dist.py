"""Multi-GPU plumbing for the benchmark: one process per GPU, every rank runs its own batch of
sequences (the path shards by sequence with no data-path collective), so all that is exchanged is
a barrier and the max / sum of a few host scalars.  Uses torch.distributed (NCCL on GPUs, gloo on
CPU for the tests)."""
from __future__ import annotations

import os


class Group:
    def __init__(self, backend: str = "nccl", device: str = "cpu"):
        import torch
        import torch.distributed as dist
        self.torch, self.dist, self.device = torch, dist, device
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if not dist.is_initialized():
            dist.init_process_group(backend=backend)
        self.rank, self.world = dist.get_rank(), dist.get_world_size()

    def barrier(self):
        self.dist.barrier()

    def _reduce(self, x: float, op):
        t = self.torch.tensor([float(x)], dtype=self.torch.float64, device=self.device)
        self.dist.all_reduce(t, op=op)
        return float(t.item())

    def max_float(self, x: float) -> float:
        return self._reduce(x, self.dist.ReduceOp.MAX)

    def sum_float(self, x: float) -> float:
        return self._reduce(x, self.dist.ReduceOp.SUM)

    def close(self):
        if self.dist.is_initialized():
            self.dist.destroy_process_group()


def shard_units(n_units: int, rank: int, world: int):
    """Contiguous share of `n_units` independent units (sequences) for `rank`."""
    base, rem = divmod(n_units, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def aggregate_throughput(units_per_rank: float, elapsed_s_local: float, group: Group) -> float:
    """Whole-job throughput: all ranks' units / the slowest rank's time."""
    return group.sum_float(units_per_rank) / group.max_float(elapsed_s_local)
