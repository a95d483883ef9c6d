"""Parity at the full benchmark size, in the launch configuration bench.py times: the LLaMA-7B-shaped
list (291 tensors, 6.74 G parameters, 108 GB of inputs), one excp_compress_checkpoint with the
benchmark's parameters and workspace.  The oracle cannot run the whole workload in seconds, so:
  * four tensors are compared record for record with the oracle run in full (worker processes, one
    tensor each): the 131 M embedding (the largest tensor of the workload), a 45 M MLP matrix, a
    16.8 M attention matrix and a 4096-element norm; for the two largest also Algorithm 2 on the GPU
    against the oracle's on the same record;
  * every record's header and size against its counts."""
import struct

import numpy as np
import pytest
import torch

import oracle_pool
from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding, synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def test_llama7b_checkpoint_in_the_benchmark_configuration():
    free, _ = torch.cuda.mem_get_info()
    if free < 150e9:
        pytest.skip("needs about 150 GB of free device memory")
    shapes = synth.tensor_list(synth.CONFIG_SHAPES["llama-7b"])
    n_tot = sum(n for _, n in shapes)
    quads = [synth.make_quad(n, 1000, i, device=DEV) for i, (_, n) in enumerate(shapes)]
    big = max(range(len(shapes)), key=lambda i: shapes[i][1])      # the 131 M embedding
    mlp = [i for i, (_, n) in enumerate(shapes) if n == 4096 * 11008][5]
    attn = [i for i, (_, n) in enumerate(shapes) if n == 4096 * 4096][3]
    small = [i for i, (_, n) in enumerate(shapes) if n == 4096][0]
    oparams = dict(kmeans_iters=10, median_source=orc.MEDIAN_ABS_RESIDUAL)
    jobs = {i: oracle_pool.submit_compress(tuple(t.cpu().numpy() for t in quads[i]), oparams, i, want_decode=i in (big, mlp))
            for i in (big, mlp, attn, small)}                      # the longest first
    h = binding.Handle(workspace_numel=1_800_000_000)
    try:
        p = binding.Params(kmeans_iters=10, median_source=binding.MEDIAN_ABS_RESIDUAL)
        blob = torch.empty(int(0.80 * n_tot) + 4096 * len(shapes) + (1 << 20), dtype=torch.uint8, device=DEV)
        offs, stats = h.compress_checkpoint(p, quads, blob)

        def rec(i):
            return blob[offs[i]:offs[i + 1]].cpu().numpy().tobytes()

        # every record: header fields and size against the counts
        for i, (_, n) in enumerate(shapes):
            head = struct.unpack("<IIQQQIIIIQQ", blob[offs[i]:offs[i] + 64].cpu().numpy().tobytes())
            want = orc.record_bytes(n, stats[i].nnz_w, stats[i].nnz_o, 4)
            assert head == (orc.MAGIC, 1, n, stats[i].nnz_w, stats[i].nnz_o, 4, 15, 256, 0, want, 0), i
            assert offs[i + 1] - offs[i] == want and stats[i].nnz_o <= stats[i].nnz_w <= n
        assert 0.4 < sum(s.nnz_w for s in stats) / n_tot < 0.65

        for i, job in jobs.items():                                # whole records against the oracle
            want = job.get(1500)
            assert (stats[i].nnz_w, stats[i].nnz_o) == (want["nnz_w"], want["nnz_o"]), shapes[i]
            assert np.float32(stats[i].median).view(np.uint32) == want["median"].view(np.uint32), shapes[i]
            assert np.float32(stats[i].mean_abs_ea).view(np.uint32) == want["mean_abs_ea"].view(np.uint32), shapes[i]
            assert stats[i].thr_w == want["thr_w"] and stats[i].thr_o == want["thr_o"], shapes[i]
            assert rec(i) == want["record"], shapes[i]
            if "decoded" in want:
                w_out, ea_out, eas_out = (torch.empty_like(quads[i][1]) for _ in range(3))
                h.decompress_tensor(blob[offs[i]:], offs[i + 1] - offs[i], quads[i][1], w_out, ea_out, eas_out)
                for got, exp in zip((w_out, ea_out, eas_out), want["decoded"]):
                    assert np.array_equal(got.cpu().numpy().view(np.uint32), exp.view(np.uint32)), shapes[i]
                del w_out, ea_out, eas_out
    finally:
        h.close()
        oracle_pool.shutdown()
        del quads
        torch.cuda.empty_cache()                                   # hand the 108 GB back before the next test module
