"""Rank plumbing of the benchmark: one process per GPU, independent batches per rank (weak scaling).

The chains' rows and images are independent problems, so ranks exchange no data; the process group
only serves the barrier around the timed region and the max-over-ranks of the device time."""
from __future__ import annotations

import os

import torch


class Ranks:
    def __init__(self, backend: str = "nccl"):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            kw = {}
            if backend == "nccl":
                kw["device_id"] = torch.device("cuda", self.local_rank)
            dist.init_process_group(backend, **kw)
            self.dist = dist

    @property
    def device(self):
        return torch.device("cuda", self.local_rank) if self.backend == "nccl" else torch.device("cpu")

    def batch_seed(self, base_seed: int = 0) -> int:
        """Every rank draws its own batch of the same shape."""
        return base_seed + self.rank

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        if self.backend == "nccl":
            torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        if self.dist is None:
            return float(x)
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def aggregate(self, units_per_rank: float, ms_per_step_max: float) -> float:
        """Whole-job throughput: all ranks' units over the slowest rank's time."""
        return self.world * units_per_rank / (ms_per_step_max * 1e-3)

    def finish(self):
        if self.dist is not None:
            self.dist.barrier()
            self.dist.destroy_process_group()
