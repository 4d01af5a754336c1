"""Multi-GPU plumbing (one process per GPU, torch.distributed).

The path shards without any data-path collective: BASP groups are independent units (each
group's all-to-all stays inside the group), so different GPUs take different groups -- or,
for weak scaling, different micro-batches -- and only timing is reduced across ranks.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment (1 process -> 0, 0, 1)."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def init(backend: str | None = None) -> tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        kw = {}
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
            kw["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    """Slowest rank's value (how every multi-GPU time is reported)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def groups_of_gpu(num_groups: int, world: int, rank: int) -> range:
    """Contiguous block of BASP groups that physical GPU `rank` of `world` hosts when ONE
    micro-batch is spread over several GPUs (virtual rank r -> GPU floor(r * world / N), the
    contiguous assignment of the paper's Section IV-A).  Needs world to divide num_groups."""
    if num_groups % world != 0:
        raise ValueError("the number of groups must be a multiple of the number of GPUs "
                         "(a group split across GPUs would need a real all-to-all)")
    per = num_groups // world
    return range(rank * per, (rank + 1) * per)


def finalize():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
