"""Host-side plumbing for running independent replicas of the prefill path, one process per GPU.

The path has no inter-GPU exchange (Eq. 4's softmax and every TopK are global over one prompt's candidates),
so more GPUs means one independent prompt per rank.  The process group is used for two things only: a barrier
around the timed region and the maximum of the per-rank times.  Backend "nccl" on GPUs, "gloo" in CPU tests."""
from __future__ import annotations

import os
from typing import Optional

import torch


class Replicas:
    def __init__(self, backend: Optional[str] = None, device: Optional[torch.device] = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
            kw = {}
            if backend == "nccl" and device is not None:
                kw["device_id"] = device
            if not dist.is_initialized():
                dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        """Device sync, then a barrier over the ranks, then a device sync again."""
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
                         device=self.device if self.device is not None and self.device.type == "cuda" else "cpu")
        if t.is_cuda:
            t = t.float()
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_throughput(self, units_per_rank: float, ms: float) -> float:
        """Whole-job units per second: every rank processed `units_per_rank` in the slowest rank's `ms`."""
        return units_per_rank * self.world / (self.max_over_ranks(ms) * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.barrier()
            self.dist.destroy_process_group()
            self.dist = None
