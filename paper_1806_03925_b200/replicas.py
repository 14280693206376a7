"""Host-side plumbing for running independent replicas of the step, one process per GPU.

On one GPU the path has no exchange step, so N GPUs run N replicas (own tables, own batches); the only things the
ranks share are a barrier around the timed region, the maximum of their device-measured times and the sum of the
page views they processed.  Nothing here touches the data path; the backend is NCCL on GPUs and gloo in the CPU
tests.
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Optional


@dataclass
class Replicas:
    rank: int
    world: int
    local_rank: int
    backend: Optional[str] = None

    @staticmethod
    def from_env() -> "Replicas":
        return Replicas(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                        int(os.environ.get("LOCAL_RANK", "0")))

    def init(self, backend: str, device=None) -> None:
        """Joins the process group (no-op for a single process)."""
        if self.world <= 1:
            return
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kw)
        self.backend = backend

    @property
    def seed(self) -> int:
        """Every replica draws its own tables and batches."""
        return self.rank

    def barrier(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max_over_ranks(self, value: float, device="cpu") -> float:
        """The slowest rank's figure (a timed region ends when the last replica is done)."""
        if self.world <= 1:
            return float(value)
        import torch
        import torch.distributed as dist
        t = torch.tensor([float(value)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, ms_max: float) -> float:
        """Units per second over all replicas: every rank processed units_per_rank in at most ms_max."""
        return units_per_rank * self.world / (ms_max * 1e-3)

    def close(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            if dist.is_initialized():
                dist.destroy_process_group()
