"""Multi-process plumbing for running independent replicas of the step, one process per GPU.

The path does not shard across GPUs (all simulated workers live on one device and the method has no
exchange step at this level), so N GPUs run N replicas: no data-path collective.  The only
communication is a barrier around the timed region and a max-over-ranks of the measured time.
Backend "nccl" on GPUs; "gloo" lets the same logic be tested on CPU.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


class Replicas:
    def __init__(self, backend: str = "nccl", device: torch.device | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device if device is not None else torch.device("cpu")
        self.owns_group = False
        if self.world > 1 and not dist.is_initialized():
            kw = {"device_id": self.device} if backend == "nccl" else {}
            dist.init_process_group(backend, **kw)
            self.owns_group = True

    def barrier(self) -> None:
        if self.world > 1:
            dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        """The slowest rank's time: what a whole-job throughput has to be divided by."""
        if self.world == 1:
            return float(value)
        t = torch.tensor([value], dtype=torch.float64, device=self.device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_value(self, units_per_rank_per_step: float, ms_per_step_local: float) -> tuple[float, float]:
        """(value, ms_per_step): units all ranks processed per second, on the slowest rank's clock."""
        ms = self.max_over_ranks(ms_per_step_local)
        return self.world * units_per_rank_per_step / (ms * 1e-3), ms

    def replica_seed_offset(self) -> int:
        """Replicas draw different gradients: their workload seeds are offset by this."""
        return 100 * self.rank

    def close(self) -> None:
        if self.owns_group and dist.is_initialized():
            dist.destroy_process_group()
