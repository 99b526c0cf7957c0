"""Independent replicas: the only multi-GPU form of this path.

Every GPU owns its KV pools, its block tables and its host link; nothing crosses GPUs (the paper's
multi-instance deployment is replicas behind a router, Section 4.4).  One process per GPU runs the
same workload on its own seeded data; the only communication is the measurement itself: a barrier on
both sides of the timed region and a max-over-ranks of the device times, through torch.distributed
(NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple


def env() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment (1 process = rank 0 of 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own KV contents; shapes, context lengths and victims are the workload's."""
    return base_seed + 1000 * rank


class Group:
    """Process group of the replicas (a no-op for one process)."""

    def __init__(self, backend: str, device=None):
        import torch
        import torch.distributed as dist
        self.rank, self.world, self.local_rank = env()
        self.dist = dist
        self.torch = torch
        self.device = device if device is not None else torch.device("cpu")
        self.active = self.world > 1
        if self.active and not dist.is_initialized():
            kw = {}
            if backend == "nccl":
                kw["device_id"] = self.device
            dist.init_process_group(backend, **kw)

    def barrier(self) -> None:
        if self.active:
            self.dist.barrier()

    def max_over_ranks(self, values: Sequence[float]) -> List[float]:
        """Element-wise maximum over the replicas (timings: the slowest replica defines the step)."""
        if not self.active:
            return [float(v) for v in values]
        t = self.torch.tensor(list(values), dtype=self.torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return [float(v) for v in t.tolist()]

    def sum_over_ranks(self, values: Sequence[float]) -> List[float]:
        """Element-wise sum over the replicas (units processed: the whole job's work)."""
        if not self.active:
            return [float(v) for v in values]
        t = self.torch.tensor(list(values), dtype=self.torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return [float(v) for v in t.tolist()]

    def close(self) -> None:
        if self.active and self.dist.is_initialized():
            self.dist.barrier()
            self.dist.destroy_process_group()


def whole_job_rate(group: Group, units_local: float, ms_local: float) -> Tuple[float, float]:
    """(units of all replicas per second, max-over-ranks milliseconds)."""
    (ms,) = group.max_over_ranks([ms_local])
    (units,) = group.sum_over_ranks([units_local])
    return units / (ms * 1e-3), ms
