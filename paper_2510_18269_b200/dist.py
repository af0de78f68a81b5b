"""Process-group plumbing for multi-GPU runs (one process per GPU).

The OQM path has no exchange step: every layer, and every video stream, is
independent, so ranks never communicate on the data path.  torch.distributed
is used only for the barrier around the timed region and for reducing the
per-rank timings (max) and unit counts (sum).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init_from_env(n_gpus: int, backend: str | None = None):
    """Returns (rank, world, local_rank).  Single-process runs do not create a process group."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def _device():
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float) -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float) -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_layers(n_layers: int, rank: int, world: int):
    """Contiguous layer range [begin, begin+count) owned by `rank` when one stream is split by layer."""
    base, rem = divmod(n_layers, world)
    begin = rank * base + min(rank, rem)
    return begin, base + (1 if rank < rem else 0)


def finish():
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
