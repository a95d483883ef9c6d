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


def gather_objects(obj, world: int) -> list:
    """Every rank's `obj`, in rank order, on every rank (host-side bookkeeping; not on the data path)."""
    if world == 1:
        return [obj]
    out = [None] * world
    dist.all_gather_object(out, obj)
    return out


def assemble_offsets(numels, shares, local_offsets_by_rank):
    """The checkpoint-wide table of one partitioned checkpoint.

    shares[r] = tensor indices rank r compressed (ascending); local_offsets_by_rank[r] = that rank's
    offsets list (len(shares[r]) + 1) into its own blob.  Returns (table, offsets): table[i] =
    (owner rank, offset in the owner's blob, record bytes) for tensor i of the checkpoint; offsets =
    where record i starts if the records are laid back to back in checkpoint order (len n + 1), i.e.
    the tensor_offsets a single-process compress of the whole list returns."""
    n = len(numels)
    table = [None] * n
    for r, (idx, offs) in enumerate(zip(shares, local_offsets_by_rank)):
        if len(offs) != len(idx) + 1:
            raise ValueError(f"rank {r}: {len(idx)} tensors but {len(offs)} offsets")
        for k, i in enumerate(idx):
            if table[i] is not None:
                raise ValueError(f"tensor {i} compressed twice")
            table[i] = (r, int(offs[k]), int(offs[k + 1] - offs[k]))
    if any(t is None for t in table):
        raise ValueError("a tensor was compressed by no rank")
    offsets = [0]
    for _, _, nbytes in table:
        offsets.append(offsets[-1] + nbytes)
    return table, offsets


def compress_partitioned(compress_share, numels, world: int, rank: int):
    """One checkpoint compressed by `world` ranks, each on its own GPU (strong scaling).

    The tensor list is dealt by partition_tensors; this rank calls compress_share(indices), which
    compresses those tensors into the rank's own blob with their checkpoint-wide indices (so the
    records are the ones a single process writes) and returns the offsets into that blob.  The ranks
    then exchange only those offsets (host objects) and every rank assembles the same table.  No
    tensor data, record or statistic crosses ranks.  Returns (my indices, table, offsets) as in
    assemble_offsets."""
    shares = partition_tensors(numels, world)
    mine = shares[rank]
    local = [int(o) for o in compress_share(mine)]
    table, offsets = assemble_offsets(numels, shares, gather_objects(local, world))
    return mine, table, offsets


def assemble_blob(table, blobs_by_rank) -> bytes:
    """The single checkpoint blob (records in checkpoint order) from the ranks' blobs; host bytes."""
    return b"".join(bytes(blobs_by_rank[r][off:off + nbytes]) for r, off, nbytes in table)
