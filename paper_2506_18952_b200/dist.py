"""Multi-GPU plumbing for the benchmark: the verify step shards by sequence, so N GPUs run N independent
replicas (each holds all of W_lm and its own batch); there is no data-path collective.  torch.distributed is
used only for the start/stop barrier, the max-over-ranks time and the sum of per-rank counters."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when not launched by one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str) -> tuple[int, int, int]:
    rank, world, local = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29531")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def barrier():
    if dist.is_initialized():
        dist.barrier()


def _reduce(value: float, op, device) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def rank_seed_offset(rank: int) -> int:
    """Each replica verifies its own batch: same recipe, different seed."""
    return 1000003 * rank


def aggregate_throughput(units_this_rank: float, ms_this_rank: float, device="cpu") -> tuple[float, float]:
    """Whole-job units/s = units over all ranks / slowest rank's time.  Returns (units_per_s, max_ms)."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
