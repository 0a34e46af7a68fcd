"""Multi-GPU plumbing of the benchmark: one process per GPU, independent shards, no data-path
collective.  Output channels (and layers) are independent sub-problems, so ranks only meet at
the timing barrier and for a MAX / SUM reduce of scalars."""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def init_from_env(expected_world: int = 1, backend: str | None = None) -> Tuple[int, int, int]:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_* (torchrun) if there is
    one.  Returns (rank, world_size, local_rank)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if backend == "nccl":
            torch.cuda.set_device(local)
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    if expected_world not in (1, world) and rank == 0:
        print(f"warning: --gpus {expected_world} but WORLD_SIZE={world}", flush=True)
    return rank, world, local


def _device() -> torch.device:
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def shard_channels(shapes: Sequence[Sequence[int]], rank: int, world: int) -> List[Tuple[int, int, int]]:
    """Strong-scaling split of a model: (layer, first_channel, n_channels) pieces for `rank`.
    Every layer's output channels are cut into `world` contiguous ranges of near-equal size, so
    each rank gets the same mix of layer shapes and no piece needs data from another."""
    out = []
    for i, s in enumerate(shapes):
        m = int(s[0])
        lo, hi = m * rank // world, m * (rank + 1) // world
        if hi > lo:
            out.append((i, lo, hi - lo))
    return out


def finish() -> None:
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
