"""Multi-GPU plumbing: the path shards over the batch only (images / GEMM rows are independent and
the packed weights are replicated), so ranks are replicas with no data-path collective.  The only
communication is the barrier around the timed region and the max-over-ranks of the step time."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str):
    """Initialise the default process group from the torchrun environment (no-op for one rank)."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The job's step time is that of the slowest replica."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_batch(n_items: int, rank: int, world: int):
    """Contiguous [lo, hi) share of a batch for strong-scaling splits of one batch."""
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def whole_job_throughput(units_per_rank_step: float, steps: int, ms_local: float, device="cpu"):
    """(aggregate units/s over all ranks, ms per step) with the time taken as the max over ranks."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_per_rank_step, device)
    return units * steps / (ms * 1e-3), ms / steps
