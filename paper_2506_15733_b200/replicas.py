"""Rank plumbing for running independent replicas of the scoring step, one process per GPU.

The path shards by rows / problems with no exchange step (candidates are drawn independently and
SubSample works per problem), so ranks never exchange data: the only collectives are the barrier
around a timed region and the MAX of the ranks' elapsed times.  ``torch.distributed`` carries both
(NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Optional


@dataclass
class Replicas:
    rank: int
    local_rank: int
    world: int
    backend: Optional[str] = None      # None: single process, torch.distributed unused

    @classmethod
    def from_env(cls) -> "Replicas":
        """Rank layout as torch.distributed.run exports it (a plain launch is a world of one)."""
        return cls(int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
                   int(os.environ.get("WORLD_SIZE", "1")))

    def init(self, backend: str, device=None) -> None:
        """Join the process group (rendezvous from MASTER_ADDR / MASTER_PORT); no-op for one rank."""
        if self.world == 1:
            return
        import torch.distributed as dist
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kw)
        self.backend = backend

    def _device(self):
        import torch
        return torch.device("cuda", self.local_rank) if self.backend == "nccl" else torch.device("cpu")

    def barrier(self) -> None:
        if self.backend is not None:
            import torch.distributed as dist
            dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank's figure: a multi-GPU time is the maximum over ranks."""
        if self.backend is None:
            return float(value)
        import torch
        import torch.distributed as dist
        t = torch.tensor([float(value)], dtype=torch.float64, device=self._device())
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_rate(self, units_per_rank: float, elapsed_s: float) -> float:
        """Units all ranks processed divided by the slowest rank's time (weak scaling: same work per rank)."""
        return units_per_rank * self.world / self.max_over_ranks(elapsed_s)

    def shutdown(self) -> None:
        if self.backend is not None:
            import torch.distributed as dist
            dist.destroy_process_group()
            self.backend = None
