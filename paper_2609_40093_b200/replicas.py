"""One process per GPU, independent replicas: the only multi-GPU plumbing this path needs.

The routing-aware dispatch/combine path is defined on one GPU with logical ranks, so
N GPUs run N independent copies of the workload. There is no data-path collective;
torch.distributed carries only the barrier around the timed region and the
max-over-ranks of the measured time. The backend is NCCL on GPUs and gloo on CPU
(tests).
"""
from __future__ import annotations

import os

import torch


class Replicas:
    def __init__(self, backend: str | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.cuda = torch.cuda.is_available() and backend != "gloo"
        self.backend = backend or ("nccl" if self.cuda else "gloo")
        if self.cuda:
            torch.cuda.set_device(self.local if self.world > 1 else 0)
        if self.world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29511")
            if self.backend == "nccl":
                dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
            else:
                dist.init_process_group("gloo")

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        if self.cuda:
            torch.cuda.synchronize()

    def max_over_ranks(self, value: float) -> float:
        if self.world == 1:
            return float(value)
        import torch.distributed as dist
        t = torch.tensor([value], dtype=torch.float64, device="cuda" if self.cuda else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, seconds_this_rank: float) -> float:
        """Units all ranks processed divided by the slowest rank's time."""
        return self.world * units_per_rank / self.max_over_ranks(seconds_this_rank)

    def close(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
