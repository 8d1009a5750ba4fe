"""Process-group plumbing for multi-GPU runs (one process per GPU, launched by torchrun).

Encode and decode have no collective inside them: layers (or whole gradients) are independent units.  The one
exchange step of data-parallel training is between them: an all-gather of the fixed-capacity payload buffers
(`all_gather_bytes`), after which every rank averages all payloads with `atomo_decode_average`.
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment (1-process defaults)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
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


def shard_units(costs: Sequence[float], world: int) -> List[List[int]]:
    """Greedy longest-first partition of independent units (layers) by cost; deterministic."""
    order = sorted(range(len(costs)), key=lambda i: (-costs[i], i))
    loads = [0.0] * world
    parts: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (loads[k], k))
        parts[r].append(i)
        loads[r] += costs[i]
    return [sorted(p) for p in parts]


def all_gather_bytes(buf: torch.Tensor) -> List[torch.Tensor]:
    """The exchange step of data-parallel training: every rank contributes its payload buffer (uint8, the same
    fixed capacity on every rank) and receives all of them, as views of one gathered buffer in rank order.
    Without a process group the list holds the caller's own buffer."""
    if buf.dtype != torch.uint8 or buf.dim() != 1:
        raise ValueError("payload buffers are flat uint8 tensors")
    if not dist.is_initialized():
        return [buf]
    world = dist.get_world_size()
    gathered = torch.empty(world * buf.numel(), dtype=torch.uint8, device=buf.device)
    dist.all_gather_into_tensor(gathered, buf.contiguous())
    return list(gathered.view(world, buf.numel()).unbind(0))


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
