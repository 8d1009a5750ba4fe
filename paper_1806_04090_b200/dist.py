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


class PeerPayloads:
    """Payload buffers that every rank of one node can read in place (CUDA peer access over NVLink through
    torch's symmetric memory).  Each rank encodes into `self.buf`; after `publish()` the averaging decode is
    given `self.views()` -- tensors that alias the peers' buffers -- so ONE kernel both fetches every
    worker's payload over NVLink (plain loads, a few hundred KB) and forms the averaged gradient: there is no
    separate collective and no staging copy.  `release()` keeps a rank from overwriting its buffer while a
    peer may still be reading it.  Without a process group (or without symmetric memory) the object holds a
    plain local buffer and `views()` is just that buffer.
    Not exercised on more than one GPU in this build (one GPU available): the single-rank path and the gloo
    fallback are what the tests cover."""

    def __init__(self, nbytes: int, device: torch.device):
        self.handle = None
        self.world = dist.get_world_size() if dist.is_initialized() else 1
        self.nbytes = int(nbytes)
        if self.world > 1 and device.type == "cuda":
            import torch.distributed._symmetric_memory as symm_mem
            self.buf = symm_mem.empty(self.nbytes, dtype=torch.uint8, device=device)
            self.handle = symm_mem.rendezvous(self.buf, dist.group.WORLD)
        else:
            self.buf = torch.empty(self.nbytes, dtype=torch.uint8, device=device)

    def publish(self) -> None:
        """Call after encode has been enqueued: when it returns, every rank's payload of this step is complete
        and visible to the kernels enqueued next on the current stream."""
        if self.handle is not None:
            self.handle.barrier(channel=0)
        elif self.world > 1:
            dist.barrier()

    def views(self) -> List[torch.Tensor]:
        if self.handle is None:
            return [self.buf] if self.world == 1 else all_gather_bytes(self.buf)
        return [self.handle.get_buffer(r, (self.nbytes,), torch.uint8) for r in range(self.world)]

    def release(self) -> None:
        """Call after the averaging decode has been enqueued: no rank starts the next encode (which rewrites its
        buffer) before every rank has finished reading."""
        if self.handle is not None:
            self.handle.barrier(channel=1)
        elif self.world > 1:
            dist.barrier()


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
