"""Multi-process plumbing for the benchmark: one process per GPU, the path shards
by sequence (sequences are independent: routing is per token, pruning per sequence),
so ranks run replicas of the workload on their own token batches and exchange nothing
on the data path.  The only communication is the barrier around the timed region and
the max-over-ranks of the measured time."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def token_seed_for_rank(base_seed: int, rank: int) -> int:
    """Each rank draws its own token batch (weak scaling: fixed work per GPU)."""
    return base_seed + 7919 * rank


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device: str = "cpu") -> Tuple[float, float]:
    """Whole-job throughput = units all ranks processed / slowest rank's time."""
    t = max_over_ranks(seconds_this_rank, device)
    u = sum_over_ranks(units_this_rank, device)
    return u / t, t


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
