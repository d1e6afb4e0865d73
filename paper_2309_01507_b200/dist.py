"""Multi-process plumbing: one process per GPU, no data-path collective.

The optimizer step treats tensors independently (Sec. 2.1: the step is applied layer by layer), so
several GPUs shard it at tensor granularity and exchange nothing inside the step. This module holds
the rendezvous helpers the benchmark uses (barrier, max-over-ranks timing) and the byte-balanced
tensor partition for a tensor-granular (ZeRO-1 style) ownership split.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when not launched by it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None) -> bool:
    """Joins the process group when WORLD_SIZE > 1. Returns True if a group is active."""
    _, _, world = env()
    if world <= 1:
        return False
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return True


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def _reduce(value: float, op, device) -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def shutdown() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def partition_by_bytes(numels, world: int):
    """Tensor-granular ownership: assigns tensor indices to `world` ranks, largest first onto the
    least-loaded rank. Returns a list of index lists (each sorted), covering every tensor once."""
    if world < 1:
        raise ValueError("world must be >= 1")
    load = [0] * world
    owned = [[] for _ in range(world)]
    for i in sorted(range(len(numels)), key=lambda k: (-numels[k], k)):
        r = min(range(world), key=lambda k: (load[k], k))
        owned[r].append(i)
        load[r] += numels[i]
    return [sorted(o) for o in owned]
