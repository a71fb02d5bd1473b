"""Rank plumbing for the multi-GPU benchmark: one process per GPU, no data-path collective.

The MSD path shards only trivially (independent GEMM / attention problems), so the ranks run replicas of the workload
and meet only to line up the timed region and to combine its timing: a barrier on both sides, the MAX over ranks of
the device time, and the SUM over ranks of the units processed.  The same code runs over NCCL on GPUs and over gloo in
the CPU tests.
"""
import os

import torch
import torch.distributed as dist


class Ranks:
    def __init__(self, backend, device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device if device is not None else torch.device("cpu")
        self._owns_group = False
        if self.world > 1 and not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            kwargs = {"device_id": self.device} if backend == "nccl" else {}
            dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kwargs)
            self._owns_group = True

    @property
    def is_root(self):
        return self.rank == 0

    def barrier(self):
        if self.world > 1:
            dist.barrier()

    def _reduce(self, value, op):
        if self.world == 1:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=op)
        return float(t.item())

    def max_over_ranks(self, value):
        """The slowest rank's time is the job's time."""
        return self._reduce(value, dist.ReduceOp.MAX)

    def sum_over_ranks(self, value):
        return self._reduce(value, dist.ReduceOp.SUM)

    def job_throughput(self, units_this_rank, ms_this_rank):
        """Whole-job units per second: all ranks' units over the slowest rank's time (also returns that time in ms)."""
        ms = self.max_over_ranks(ms_this_rank)
        units = self.sum_over_ranks(units_this_rank)
        return units / (ms * 1e-3), ms

    def close(self):
        if self._owns_group and dist.is_initialized():
            dist.destroy_process_group()
