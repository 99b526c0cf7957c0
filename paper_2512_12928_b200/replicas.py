"""Independent replicas: the only multi-GPU form of this path.

Every GPU owns its KV pools, its block tables and its host link; nothing crosses GPUs (the paper's
multi-instance deployment is replicas behind a router, Section 4.4).  One process per GPU runs the
same workload on its own seeded data; the only communication is the measurement itself: a barrier on
both sides of the timed region and a max-over-ranks of the device times, through torch.distributed
(NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Optional, Sequence, Tuple


def env() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment (1 process = rank 0 of 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def spawn(argv: Sequence[str], n: int, stdout=None) -> List[int]:
    """Starts n replicas of a command on this node, one process per GPU, with the environment a launcher would
    give them (RANK = LOCAL_RANK = 0..n-1, WORLD_SIZE = n, rendezvous on 127.0.0.1 at a free port), waits for
    all of them and returns their exit codes.  What `bench.py --gpus N` does when it was not started by a
    launcher."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env, stdout=stdout))
    return [p.wait() for p in procs]


def numa_cpus_of_gpu(local_rank: int, sysfs: str = "/sys") -> Optional[List[int]]:
    """CPUs of the NUMA node the GPU's PCIe slot hangs off, from sysfs, or None when the box does not say
    (pinned host pools allocated by a process bound to these CPUs land in the memory nearest to the GPU's link)."""
    try:
        import torch
        p = torch.cuda.get_device_properties(local_rank)
        bus = f"{p.pci_domain_id:04x}:{p.pci_bus_id:02x}:{p.pci_device_id:02x}.0"
        node = int(open(os.path.join(sysfs, "bus/pci/devices", bus, "numa_node")).read())
        if node < 0:
            return None
        return parse_cpulist(open(os.path.join(sysfs, "devices/system/node", f"node{node}", "cpulist")).read())
    except Exception:
        return None


def parse_cpulist(text: str) -> List[int]:
    """'0-3,8,10-11' -> [0, 1, 2, 3, 8, 10, 11]."""
    cpus: List[int] = []
    for part in text.strip().split(","):
        if not part:
            continue
        lo, _, hi = part.partition("-")
        cpus.extend(range(int(lo), int(hi or lo) + 1))
    return cpus


def bind_near_gpu(local_rank: int) -> bool:
    """Restricts this process to the CPUs near its GPU, if the box exposes them and they are allowed."""
    cpus = numa_cpus_of_gpu(local_rank)
    if not cpus:
        return False
    allowed = sorted(set(cpus) & os.sched_getaffinity(0))
    if not allowed:
        return False
    os.sched_setaffinity(0, allowed)
    return True


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
