"""Host-side plumbing for running independent replicas, one process per GPU.

The recurrence has no exchange step, so several GPUs simply evaluate independent
problems; the only cross-rank operations are a barrier around the timed region and
the maximum of the per-rank times (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os


class Replicas:
    """Process-group wrapper that degrades to a single process when WORLD_SIZE is 1 or unset."""

    def __init__(self, backend: str = "nccl", device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            kwargs = {}
            if backend == "nccl" and device is not None:
                kwargs["device_id"] = device
            if not dist.is_initialized():
                dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kwargs)
            self.dist = dist

    def barrier(self) -> None:
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank decides: max of a per-rank time."""
        if self.dist is None:
            return float(value)
        import torch
        t = torch.tensor([float(value)], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def aggregate_throughput(self, units_per_replica: float, seconds_local: float) -> float:
        """Whole-job throughput: every replica processed `units_per_replica` in at most the slowest rank's time."""
        return self.world * units_per_replica / self.max_over_ranks(seconds_local)

    def close(self) -> None:
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None
