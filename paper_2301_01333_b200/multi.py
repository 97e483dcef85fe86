"""Rank plumbing for runs with one process per GPU.

The path shards with no exchange step: every output row of an MLP chain depends only on the same input row (the
outer parallel loop over the batch, Section V "coarse-grain fusion") and every (batch, head) unit of the attention
block is independent (Section VII "MHA").  So the only communication a multi-GPU run needs is for timing: a barrier
on both sides of the timed region and the maximum of the ranks' times.  Everything here takes the backend as a
parameter ("nccl" on GPUs, "gloo" for the CPU tests) and holds none of the method's arithmetic.
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Callable, Dict, Optional, Tuple


@dataclass
class Ranks:
    rank: int
    world: int
    local: int
    backend: Optional[str]          # None: single process, no process group

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def init_ranks(backend: str = "nccl", device: Optional[str] = None) -> Ranks:
    """Read RANK / WORLD_SIZE / LOCAL_RANK (as torchrun sets them) and join the process group when there is more
    than one rank.  `device` ("cuda:3") binds an NCCL group to this rank's GPU."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch
        import torch.distributed as dist
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = torch.device(device)
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
        return Ranks(rank, world, local, backend)
    return Ranks(rank, world, local, None)


def barrier(r: Ranks) -> None:
    if r.world > 1:
        import torch.distributed as dist
        dist.barrier()


def _reduce(r: Ranks, x: float, op_name: str, device: Optional[str]) -> float:
    if r.world == 1:
        return float(x)
    import torch
    import torch.distributed as dist
    dev = device if (r.backend == "nccl" and device is not None) else "cpu"
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return float(t.item())


def max_over_ranks(r: Ranks, x: float, device: Optional[str] = None) -> float:
    """The slowest rank's value: a multi-GPU step is as long as its slowest GPU."""
    return _reduce(r, x, "MAX", device)


def sum_over_ranks(r: Ranks, x: float, device: Optional[str] = None) -> float:
    """Whole-job totals (units processed by all ranks)."""
    return _reduce(r, x, "SUM", device)


def build_on_local_root(r: Ranks, build: Callable[[], object]) -> None:
    """One rank per node compiles the in-tree library, the others wait for it."""
    if r.local == 0:
        build()
    barrier(r)


def finish(r: Ranks) -> None:
    if r.world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def split_units(total: int, world: int, rank: int) -> Tuple[int, int]:
    """Even split of `total` independent units over `world` ranks: (first unit, count) of `rank`.  The first
    total % world ranks take one unit more; the shares tile [0, total) in rank order."""
    base, extra = divmod(total, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def timed_region(r: Ranks, run_steps: Callable[[], float], device: Optional[str] = None) -> float:
    """Barrier, this rank's timed steps (`run_steps` returns its own device time in ms), barrier, and the maximum
    over ranks of that time."""
    barrier(r)
    ms = run_steps()
    barrier(r)
    return max_over_ranks(r, ms, device)


def job_line_fields(r: Ranks, units_this_rank: float, ms: float, device: Optional[str] = None) -> Dict[str, float]:
    """Whole-job aggregate: the units all ranks processed divided by the slowest rank's time."""
    total = sum_over_ranks(r, units_this_rank, device)
    return {"units_total": total, "ms": ms, "units_per_s": total / (ms * 1e-3) if ms > 0 else 0.0}
