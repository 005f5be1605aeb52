"""Host-side plumbing for running N independent replicas of the layer step, one process
per GPU.  The path itself never communicates between GPUs; torch.distributed is used only
to line the ranks up around the timed region and to take the slowest rank's time."""
from __future__ import annotations

import os
from typing import Optional

import torch


def env_ranks():
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


class Replicas:
    def __init__(self, backend: Optional[str] = None, device: Optional[torch.device] = None):
        self.rank, self.local_rank, self.world = env_ranks()
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                kw = {}
                if backend == "nccl" and device is not None:
                    kw["device_id"] = device
                dist.init_process_group(backend or "gloo", **kw)
            self.dist = dist

    def barrier(self):
        if self.device is not None and self.device.type == "cuda":
            torch.cuda.synchronize(self.device)
        if self.dist is not None:
            self.dist.barrier()
            if self.device is not None and self.device.type == "cuda":
                torch.cuda.synchronize(self.device)

    def max_over_ranks(self, value: float) -> float:
        if self.dist is None:
            return float(value)
        t = torch.tensor([float(value)], dtype=torch.float64,
                         device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_throughput(self, units_per_rank: float, ms: float) -> float:
        """Whole-job units per second: every rank processed `units_per_rank` in the time of
        the slowest rank."""
        return self.world * units_per_rank / (self.max_over_ranks(ms) * 1e-3)

    def close(self):
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
