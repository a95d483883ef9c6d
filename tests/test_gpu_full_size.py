"""Parity at the full benchmark size, in the launch configuration bench.py times: the LLaMA-7B-shaped
list (291 tensors, 6.74 G parameters, 108 GB of inputs), one excp_compress_checkpoint with the
benchmark's parameters and workspace.  The oracle cannot run the whole workload in seconds, so:
  * two tensors (a 16.8 M attention matrix, a 4096-element norm) are compared record for record;
  * the largest tensors (the 131 M embedding, a 45 M MLP matrix) are checked through what holds at any
    size and the oracle's vectorised pieces compute quickly: the exact median and mean, both
    thresholds, both bitmaps in full, every code against the record's own centres (nearest centre by
    the mid-point rule), sorted centres, and Algorithm 2 on the GPU against the oracle's on the record;
  * every record's header and size against its counts."""
import struct

import numpy as np
import pytest
import torch

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
    h = binding.Handle(workspace_numel=1_200_000_000)
    try:
        p = binding.Params(kmeans_iters=10, median_source=binding.MEDIAN_ABS_RESIDUAL)
        op = orc.Params(kmeans_iters=10, median_source=orc.MEDIAN_ABS_RESIDUAL)
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

        by_name = {name: i for i, (name, _) in enumerate(shapes)}
        small = [i for i, (_, n) in enumerate(shapes) if n == 4096][0]
        attn = [i for i, (_, n) in enumerate(shapes) if n == 4096 * 4096][3]
        for i in (small, attn):                                    # whole records against the oracle
            q = tuple(t.cpu().numpy() for t in quads[i])
            want, info = orc.compress_tensor(*q, op, tensor_index=i)
            assert rec(i) == want, shapes[i]
            assert np.float32(stats[i].median).view(np.uint32) == np.float32(info["median"]).view(np.uint32)

        big = max(range(len(shapes)), key=lambda i: shapes[i][1])  # the 131 M embedding
        mlp = [i for i, (_, n) in enumerate(shapes) if n == 4096 * 11008][5]
        for i in (big, mlp):
            w_t, w_prev, ea, eas = (t.cpu().numpy() for t in quads[i])
            n = w_t.size
            dw = orc.residual(w_t, w_prev)
            med = orc.lower_median_abs(dw)
            mean = orc.exact_mean_abs(ea)
            assert np.float32(stats[i].median).view(np.uint32) == med.view(np.uint32)
            assert np.float32(stats[i].mean_abs_ea).view(np.uint32) == mean.view(np.uint32)
            m_w, thr_w = orc.weight_mask(dw, eas, op.alpha, med)
            m_o, thr_o = orc.moment_mask(ea, m_w, op.beta, mean)
            assert stats[i].thr_w == thr_w and stats[i].thr_o == thr_o
            r = orc.parse_record(rec(i))                           # checks sizes, populations, code range
            assert np.array_equal(r["m_w"], m_w) and np.array_equal(r["m_o"], m_o)
            for c, codes, s in ((r["c_w"], r["codes_w"], dw[m_w]), (r["c_ea"], r["codes_ea"], ea[m_o]),
                                (r["c_eas"], r["codes_eas"], eas[m_o])):
                assert np.all(np.diff(c) >= 0)
                assert np.array_equal(codes.astype(np.int64) - 1, orc.assign(s, c))   # nearest centre, mid-points down
                assert s.min() <= c[0] <= c[-1] <= s.max()                           # centres are means of members
            w_out, ea_out, eas_out = (torch.empty_like(quads[i][1]) for _ in range(3))
            h.decompress_tensor(blob[offs[i]:], offs[i + 1] - offs[i], quads[i][1], w_out, ea_out, eas_out)
            w_hat, ea_hat, eas_hat = orc.decompress_tensor(rec(i), w_prev)
            for got, want in ((w_out, w_hat), (ea_out, ea_hat), (eas_out, eas_hat)):
                assert np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))
            # the reconstruction error of a kept weight is at most the distance to the outermost centre gap
            err = np.abs(w_hat.astype(np.float64) - w_t)[m_w].max()
            assert err <= np.abs(dw).max()
            del w_out, ea_out, eas_out
    finally:
        h.close()
        del quads
        torch.cuda.empty_cache()                                   # hand the 108 GB back before the next test module
