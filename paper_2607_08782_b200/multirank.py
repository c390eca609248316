"""Plumbing for running independent replicas of the layer on several GPUs of one node.

The path has no inter-GPU exchange (the expert-parallel ranks are logical partitions of one GPU), so N GPUs
run N replicas; `torch.distributed` is used only to line the replicas up (barrier) and to combine their
timings (max over ranks) into a whole-job throughput."""
from __future__ import annotations

import os


class Ranks:
    """Process-group handle read from the torchrun environment (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_*).
    With WORLD_SIZE absent or 1 every method is a local no-op."""

    def __init__(self, backend: str = "nccl", device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend
        self.device = device
        self._dist = None
        if self.world > 1:
            import torch
            import torch.distributed as dist
            kwargs = {}
            if backend == "nccl" and device is not None:
                kwargs["device_id"] = torch.device(device)
            dist.init_process_group(backend, **kwargs)
            self._dist = dist

    def barrier(self):
        if self._dist is not None:
            self._dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank's value: whole-job time of a step that every replica runs once."""
        if self._dist is None:
            return float(value)
        import torch
        dev = self.device if self.backend == "nccl" else "cpu"
        t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
        self._dist.all_reduce(t, op=self._dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, seconds_local: float) -> float:
        """Aggregate throughput: units processed by all ranks divided by the slowest rank's time (weak scaling)."""
        return self.world * units_per_rank / self.max_over_ranks(seconds_local)

    def close(self):
        if self._dist is not None:
            self._dist.destroy_process_group()
            self._dist = None
