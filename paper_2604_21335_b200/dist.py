"""Multi-process plumbing: one process per GPU, problems sharded with no exchange.

Every (batch, kv head) problem of the path is independent (metadata, selection,
routing budget and attention are all per problem), so ranks never communicate
on the data path.  torch.distributed is used only for the start/stop barriers
and the max-over-ranks reduction of the measured time.
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import List, Tuple

import torch
import torch.distributed as dist


@dataclass
class Rank:
    rank: int = 0
    world: int = 1
    local_rank: int = 0
    backend: str = ""

    @property
    def is_main(self) -> bool:
        return self.rank == 0


def init_from_env(backend: str | None = None) -> Rank:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_* (torchrun);
    a plain `python` launch is a world of one and creates no group."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world == 1:
        return Rank()
    rank = int(os.environ["RANK"])
    local = int(os.environ.get("LOCAL_RANK", rank))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    if backend == "nccl":
        torch.cuda.set_device(local)
    dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return Rank(rank, world, local, backend)


def shutdown(r: Rank) -> None:
    if r.world > 1 and dist.is_initialized():
        dist.destroy_process_group()


def shard_range(n_items: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced split of n_items independent units: [begin, end)."""
    base, extra = divmod(n_items, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_problems(batch: int, n_kv_heads: int, rank: int, world: int) -> List[Tuple[int, int]]:
    """(batch, kv head) problems owned by `rank` when all problems are split evenly."""
    b, e = shard_range(batch * n_kv_heads, rank, world)
    return [(p // n_kv_heads, p % n_kv_heads) for p in range(b, e)]


def barrier(r: Rank) -> None:
    if r.world > 1:
        dist.barrier()


def max_over_ranks(r: Rank, value: float) -> float:
    if r.world == 1:
        return float(value)
    dev = "cuda" if r.backend == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(r: Rank, value: float) -> float:
    if r.world == 1:
        return float(value)
    dev = "cuda" if r.backend == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
