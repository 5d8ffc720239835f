"""Multi-GPU plumbing: independent replicas, one process per GPU.

The prover and the distance kernels have no exchange step (every proof and every logit row is an
independent unit), so N GPUs run N replicas of the workload on different seeded inputs and no
collective touches the data.  ``torch.distributed`` is used for exactly two things: a barrier on
both sides of the timed region and the maximum over ranks of the device-timed duration.
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def env() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment (1 process: 0, 0, 1)."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


class Replicas:
    """Process group of the replicas (``backend`` nccl on GPUs, gloo in CPU tests); a single
    process needs no group and every method degenerates."""

    def __init__(self, backend: str = "nccl", device: Optional[torch.device] = None):
        self.rank, self.local_rank, self.world = env()
        self.device = device if device is not None else torch.device("cpu")
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                kwargs = {"device_id": self.device} if backend == "nccl" else {}
                dist.init_process_group(backend, **kwargs)
            self.dist = dist

    def seed(self, base: int) -> int:
        """Data seed of this replica: replicas work on different inputs."""
        return base + self.rank

    def barrier(self) -> None:
        if self.device.type == "cuda":
            torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            if self.device.type == "cuda":
                torch.cuda.synchronize()

    def max_over_ranks(self, value: float) -> float:
        """The slowest replica's figure (a duration): what the whole job took."""
        if self.dist is None:
            return float(value)
        t = torch.tensor([value], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_replica: float, seconds: float) -> float:
        """Aggregate throughput: every replica's units over the slowest replica's time."""
        return units_per_replica * self.world / self.max_over_ranks(seconds)

    def close(self) -> None:
        if self.dist is not None and self.dist.is_initialized():
            self.dist.destroy_process_group()
            self.dist = None
