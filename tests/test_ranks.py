"""The multi-rank plumbing on CPU: two gloo ranks.  The path shards by tensor with no data-path
collective, so what is checked is the bookkeeping: the partition of a tensor list, the barrier and
the slowest-rank time, the whole-job rate, and that the ranks' records together are exactly the
records of a single process (here produced by the oracle, since there is no GPU)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import ranks, synth


def test_partition_covers_every_tensor_once_and_balances():
    numels = [n for _, n in synth.tensor_list(synth.CONFIG_SHAPES["llama-7b"])]
    for world in (1, 2, 3, 8):
        parts = ranks.partition_tensors(numels, world)
        assert len(parts) == world
        flat = sorted(i for p in parts for i in p)
        assert flat == list(range(len(numels)))
        loads = [sum(numels[i] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(numels)              # greedy largest-first bound
        assert all(p == sorted(p) for p in parts)
    assert ranks.partition_tensors([], 2) == [[], []]
    assert ranks.partition_tensors([5, 5, 5], 2) == [[0, 2], [1]]  # ties go to the lower rank
    with pytest.raises(ValueError):
        ranks.partition_tensors([1], 0)


def test_single_process_defaults():
    assert ranks.max_over_ranks(3.5, 1) == 3.5 and ranks.sum_over_ranks(2.0, 1) == 2.0
    assert ranks.whole_job_rate(1000, 500.0) == 2000.0
    assert ranks.rank_seed(1000, 3) == 1003
    ranks.barrier(1)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert ranks.rank_info() == (rank, world, rank)
        shapes = synth.tensor_list(synth.CONFIG_SHAPES["tiny"])[:10]
        numels = [n for _, n in shapes]
        mine = ranks.partition_tensors(numels, world)[rank]
        p = orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL, kmeans_iters=2)
        recs = {}
        for i in mine:                                             # tensor i keeps its checkpoint-wide index
            q = synth.make_quad(numels[i], 77, i, device="cpu")
            blob, _ = orc.compress_tensor(*(t.numpy() for t in q), p, tensor_index=i)
            recs[i] = blob
        ranks.barrier(world)
        slow = ranks.max_over_ranks(10.0 + 5.0 * rank, world)      # rank 1 is the slow one
        total = ranks.sum_over_ranks(float(sum(numels[i] for i in mine)), world)
        gathered = [None] * world
        dist.all_gather_object(gathered, {i: len(b) for i, b in recs.items()})
        out[rank] = dict(slow=slow, total=total, sizes=gathered, recs=recs, seed=ranks.rank_seed(1000, rank))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_tensor_and_agree_on_the_timing():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    shapes = synth.tensor_list(synth.CONFIG_SHAPES["tiny"])[:10]
    numels = [n for _, n in shapes]
    assert res[0]["slow"] == res[1]["slow"] == 15.0                # every rank reports the slowest rank's time
    assert res[0]["total"] == res[1]["total"] == float(sum(numels))
    assert ranks.whole_job_rate(res[0]["total"], res[0]["slow"]) == sum(numels) / 15e-3
    assert res[0]["seed"] != res[1]["seed"]
    # the two ranks' records together = the records of one process, tensor by tensor
    p = orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL, kmeans_iters=2)
    merged = {**res[0]["recs"], **res[1]["recs"]}
    assert sorted(merged) == list(range(len(numels))) and not set(res[0]["recs"]) & set(res[1]["recs"])
    for i, n in enumerate(numels):
        q = synth.make_quad(n, 77, i, device="cpu")
        want, _ = orc.compress_tensor(*(t.numpy() for t in q), p, tensor_index=i)
        assert merged[i] == want
    sizes = {}
    for d in res[0]["sizes"]:
        sizes.update(d)
    assert sizes == {i: len(b) for i, b in merged.items()}


def _part_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        numels = [n for _, n in synth.tensor_list(synth.CONFIG_SHAPES["tiny"])]
        blob = bytearray()

        def compress_share(indices):                               # stub records: the tensor's index and size, repeated
            offs = [0]
            for i in indices:
                blob.extend(_stub_record(i, numels[i]))
                offs.append(len(blob))
            return offs

        mine, table, offsets = ranks.compress_partitioned(compress_share, numels, world, rank)
        out[rank] = dict(mine=mine, table=table, offsets=offsets, blob=bytes(blob))
    finally:
        dist.destroy_process_group()


def _stub_record(i, numel):
    return (i.to_bytes(4, "little") + numel.to_bytes(8, "little")) * (1 + numel % 7) + bytes(4)   # 16-byte multiples


def test_two_gloo_ranks_compress_one_partitioned_checkpoint():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_part_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    numels = [n for _, n in synth.tensor_list(synth.CONFIG_SHAPES["tiny"])]
    assert res[0]["table"] == res[1]["table"] and res[0]["offsets"] == res[1]["offsets"]
    assert sorted(res[0]["mine"] + res[1]["mine"]) == list(range(len(numels)))
    whole = b"".join(_stub_record(i, n) for i, n in enumerate(numels))          # what one process writes
    assert ranks.assemble_blob(res[0]["table"], [res[0]["blob"], res[1]["blob"]]) == whole
    offs = res[0]["offsets"]
    assert offs[-1] == len(whole)
    for i, n in enumerate(numels):
        assert whole[offs[i]:offs[i + 1]] == _stub_record(i, n)
        r, off, nbytes = res[0]["table"][i]
        assert i in res[r]["mine"] and res[r]["blob"][off:off + nbytes] == _stub_record(i, n)


def test_assemble_offsets_refuses_inconsistent_shares():
    with pytest.raises(ValueError):
        ranks.assemble_offsets([4, 4], [[0], [0]], [[0, 16], [0, 16]])          # tensor 0 twice, tensor 1 never
    with pytest.raises(ValueError):
        ranks.assemble_offsets([4, 4], [[0], []], [[0, 16], [0]])               # tensor 1 by nobody
    with pytest.raises(ValueError):
        ranks.assemble_offsets([4], [[0]], [[0]])                               # offsets too short
    table, offs = ranks.assemble_offsets([4, 8, 4], [[1], [0, 2]], [[0, 32], [0, 16, 48]])
    assert table == [(1, 0, 16), (0, 0, 32), (1, 16, 32)] and offs == [0, 16, 48, 80]
