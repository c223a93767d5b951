"""Multi-process plumbing for the benchmark: the layer does not shard (one GPU holds every
expert, no inter-GPU exchange step), so N processes are N independent replicas of the same
workload on different seeds.  Only the timing is reduced across ranks."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment (single process: 0,0,1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str):
    rank, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29531")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def replica_seed(base_seed: int, rank: int) -> int:
    """Every replica draws its own activations; the weights' seed is shared."""
    return base_seed + 7907 * rank


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's value (the job finishes when the last replica does)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, elapsed_ms_this_rank: float, device="cpu"):
    """Whole-job throughput: units all ranks processed / slowest rank's time.
    Returns (units_per_second, ms)."""
    total_units = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(elapsed_ms_this_rank, device)
    return total_units / (ms * 1e-3), ms


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
