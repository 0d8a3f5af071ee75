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


# ------------------------------------------------------------------------------------------------
# One tensor sharded by rows over the ranks (blocks are independent, so whole rows of blocks go to
# one rank).  Only hierarchical scaling and the tensor MSE need an exchange: one MAX all-reduce of
# the tensor abs-max (exact, order-free) and one gather of the per-rank SSE sums, added in rank
# order in binary64 so that the result does not depend on arrival order.
# ------------------------------------------------------------------------------------------------
def row_shard(n_rows: int, rank: int, world: int) -> tuple[int, int]:
    """[first, last) rows of `rank` when n_rows are dealt out in contiguous, nearly equal ranges."""
    return n_rows * rank // world, n_rows * (rank + 1) // world


def _all_reduce_max(t: torch.Tensor) -> None:
    """In-place MAX all-reduce; a CUDA tensor under the gloo backend goes through a host copy."""
    if dist.get_backend() == "gloo" and t.is_cuda:
        h = t.cpu()
        dist.all_reduce(h, op=dist.ReduceOp.MAX)
        t.copy_(h)
    else:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)


def global_amax(local_amax: torch.Tensor) -> torch.Tensor:
    """MAX all-reduce of a one-element float32 tensor holding this rank's abs-max (in place).  The
    maximum is exact and order-free, so every rank ends with the same bits."""
    if dist.is_initialized():
        _all_reduce_max(local_amax)
    return local_amax


def global_mse(local_sse_sum, n_total: int) -> float:
    """Tensor MSE from the per-rank sums of block SSE (a float, or a one-element float64 tensor on any
    device): the sums are gathered and added in rank order in binary64, then divided once by the
    element count of the whole tensor, so the result does not depend on arrival order."""
    mine = torch.as_tensor(local_sse_sum, dtype=torch.float64).reshape(1)
    if not dist.is_initialized():
        return float(mine.item()) / n_total
    if dist.get_backend() == "gloo":
        mine = mine.cpu()
    parts = [torch.zeros_like(mine) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, mine)
    total = 0.0
    for v in torch.cat(parts).cpu().tolist():     # rank order
        total += v
    return total / n_total


def sharded_hierarchical_quantize(x_local: torch.Tensor, n_total: int, block_size: int, scale_fmt: int, recipe: int):
    """Quantize this rank's rows of a tensor that is sharded by rows, with ONE tensor scale
    g = amax_of_the_whole_tensor / (6 * 448) shared by all ranks.  Returns (codes, scales, block_sse,
    g tensor on the device, tensor MSE of the whole tensor).  Every rank reads only its own memory.

    Only argument marshalling and the two exchanges happen here: the abs-max, g, the quantization and
    this rank's binary64 sum of block SSEs (the library's fixed tree, called with the divisor 1, so
    that the quotient is the sum itself) are computed by the library on the device; the only host
    read is the final one of the gathered sums."""
    from . import binding as mxq
    n = x_local.numel()
    dev = x_local.device
    amax = torch.empty(1, dtype=torch.float32, device=dev)
    mxq.mxq_tensor_amax(x_local, n, amax)
    global_amax(amax)
    # g from the all-reduced abs-max, on the device: the abs-max of the one-element tensor `amax` is itself
    amax_all = torch.empty(1, dtype=torch.float32, device=dev)
    dg = torch.empty(1, dtype=torch.float32, device=dev)
    mxq.mxq_tensor_amax(amax, 1, amax_all, dg)
    codes, scales, sse = mxq.quantize(x_local, block_size, scale_fmt, recipe, 1.0, dg)
    local_sum = mxq.tensor_mse(sse, 1)
    mse = global_mse(local_sum, n_total)
    return codes, scales, sse, dg, mse


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
