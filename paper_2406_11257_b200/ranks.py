"""One process per GPU: the host-side plumbing of a multi-rank run.

Tensors are compressed independently of one another (Algorithm 1 works per tensor), so the path
shards by tensor with NO data-path collective: a rank compresses its own tensors and writes its own
records.  What crosses ranks is bookkeeping only: a barrier around the timed region, the maximum of
the ranks' device times, and, when one checkpoint is partitioned, the list of who owns which tensor.
Everything here works on CPU tensors with the gloo backend as well as on CUDA tensors with NCCL.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def rank_info() -> tuple[int, int, int]:
    """(rank, world size, local rank) as the launcher exports them; (0, 1, 0) for a plain process."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Weak scaling: every rank compresses a checkpoint of its own, generated from its own seed."""
    return base_seed + rank


def partition_tensors(numels, world: int) -> list[list[int]]:
    """Strong scaling: the tensors of ONE checkpoint dealt to `world` ranks, balanced by element count
    (largest first, each to the rank with the least so far; ties to the lower rank, so every rank
    computes the same answer without talking).  Returns, per rank, the tensor indices in ascending
    order.  A tensor is never split: its statistics and its codebooks are per tensor."""
    if world < 1:
        raise ValueError("world size")
    load = [0] * world
    owned: list[list[int]] = [[] for _ in range(world)]
    for i in sorted(range(len(numels)), key=lambda i: (-int(numels[i]), i)):
        r = min(range(world), key=lambda r: (load[r], r))
        owned[r].append(i)
        load[r] += int(numels[i])
    return [sorted(o) for o in owned]


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's time: what a multi-rank number is quoted on."""
    if world == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device="cpu") -> float:
    if world == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_all_ranks: float, ms_slowest: float) -> float:
    """Units per second of the whole job: everything all ranks processed over the slowest rank's time."""
    return units_all_ranks / (ms_slowest * 1e-3)
