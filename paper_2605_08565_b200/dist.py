"""Process-group plumbing for the benchmark: one process per GPU, no data-path collective.

Blocks are independent, so the path shards by giving every rank its own tensors (weak scaling).
The only exchanges are a barrier around the timed region and two scalar reductions (MAX of the
elapsed time, SUM of the elements processed) used to form the whole-job throughput.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None) -> tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def _device():
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def reduce_max(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(local_units: float, local_seconds: float) -> tuple[float, float]:
    """(units of all ranks / max-over-ranks time, that time)."""
    total = reduce_sum(local_units)
    t = reduce_max(local_seconds)
    return (total / t if t > 0 else 0.0), t


def rank_seed(base_seed: int, rank: int, index: int = 0) -> int:
    """Distinct, reproducible seed per (rank, tensor index): ranks never share a tensor."""
    return int(base_seed) * 1_000_003 + int(rank) * 1009 + int(index)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
