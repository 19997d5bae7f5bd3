"""Rank plumbing for multi-GPU runs of the benchmark.

The activation pass has no exchange step: with N GPUs every rank runs the same
work on its own device (replicas, weak scaling) and the data path contains no
collective.  torch.distributed is used for exactly two things: a barrier
around the timed region and the maximum over ranks of the device time.  The
backend is NCCL on GPUs and gloo on CPU (the latter is what the tests use).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class World:
    rank: int
    local_rank: int
    size: int

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def world_from_env() -> World:
    return World(int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
                 int(os.environ.get("WORLD_SIZE", "1")))


def init(w: World, backend: str, device=None) -> None:
    """Joins the process group named by MASTER_ADDR / MASTER_PORT (a no-op for one rank)."""
    if w.size > 1 and not dist.is_initialized():
        kwargs = {}
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend, rank=w.rank, world_size=w.size, **kwargs)


def finish(w: World) -> None:
    if w.size > 1 and dist.is_initialized():
        dist.destroy_process_group()


def barrier(w: World, cuda: bool) -> None:
    if w.size > 1:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(w: World, value: float, device="cpu") -> float:
    """The slowest rank's time: what a whole-job throughput must be divided by."""
    if w.size == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(w: World, units_per_rank_per_step: float, steps: int, ms_slowest: float) -> float:
    """Units per second over all ranks: every rank processed its own units in the slowest rank's time."""
    return w.size * units_per_rank_per_step * steps / (ms_slowest / 1e3)
