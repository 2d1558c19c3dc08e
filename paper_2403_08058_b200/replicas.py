"""Multi-GPU plumbing of the benchmark: independent replicas, one process per GPU.

The clustered-attention path has no exchange step (every request-layer is independent), so ranks
never trade data: each rank runs the same workload on its own GPU.  The only communication is a
barrier around the timed region and the reduction of the per-rank timings (maximum) and work
(sum) into the whole-job figure.  The same code runs on CPU with the gloo backend in the tests.
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass
class Ranks:
    rank: int
    local_rank: int
    world: int
    dist: object = None      # torch.distributed when world > 1
    device: object = None    # device used for the reduction tensors

    def barrier(self) -> None:
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, values):
        """Element-wise maximum of a list of floats over all ranks (time-like quantities)."""
        return self._reduce(values, "max")

    def sum_over_ranks(self, values):
        """Element-wise sum of a list of floats over all ranks (work-like quantities)."""
        return self._reduce(values, "sum")

    def _reduce(self, values, how):
        values = [float(v) for v in values]
        if self.dist is None:
            return values
        t = torch.tensor(values, dtype=torch.float64, device=self.device)
        op = self.dist.ReduceOp.MAX if how == "max" else self.dist.ReduceOp.SUM
        self.dist.all_reduce(t, op=op)
        return [float(x) for x in t.cpu()]

    def close(self) -> None:
        if self.dist is not None:
            self.dist.barrier()
            self.dist.destroy_process_group()


def init_ranks(backend: str = "nccl", device=None) -> Ranks:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE (torchrun) and joins the process group if there is one."""
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return Ranks(rank, local_rank, 1, None, device)
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    kwargs = {}
    if backend == "nccl" and device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend, rank=rank, world_size=world, **kwargs)
    return Ranks(rank, local_rank, world, dist, device if backend == "nccl" else torch.device("cpu"))


def whole_job_throughput(ranks: Ranks, units_local: float, seconds_local: float) -> dict:
    """Aggregate of independent replicas: units of all ranks / slowest rank's time."""
    (seconds,) = ranks.max_over_ranks([seconds_local])
    (units,) = ranks.sum_over_ranks([units_local])
    return dict(units=units, seconds=seconds, value=units / seconds if seconds > 0 else 0.0)
