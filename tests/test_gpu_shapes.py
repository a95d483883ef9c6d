"""Parity at the stated shapes of the workload configurations, whole records against the oracle:

  * the Pythia-410M-shaped checkpoint pair in full (292 tensors, 405 M parameters), with the median
    of Eq. (rw) taken over |dW| and over |W_t|;
  * the threshold-stress distribution (1 % of the residual at 10x) on the two largest kinds of
    tensor of the Pythia-1.4B shape (the 103 M embedding, a 16.8 M MLP matrix);
  * Section 3.4 / Algorithm 3: a chain of 8 checkpoints over a 410M-shaped subset that contains its
    largest tensor, every residual taken against the previous reconstruction, every step's records
    and the final reconstruction equal to the oracle's chain bit for bit (drift zero), then the
    whole chain decompressed again from the initial weights;
  * code widths 2 and 8 and an ablation combination on a 17 M tensor (many blocks share it).

The oracle runs in worker processes (tests/oracle_pool.py), one tensor per worker; everything is
submitted up front, the longest job (the chain of the 51.5 M embedding) first."""
import numpy as np
import pytest
import torch

import oracle_pool
from paper_2406_11257_b200 import binding, synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
CHAIN_STEPS = 8
PARAMS_RES = dict(kmeans_iters=10, median_source=1)
PARAMS_W = dict(kmeans_iters=10, median_source=0)


def cpu(t):
    return t.detach().cpu().numpy()


def same_bits(a, b):
    return np.array_equal(np.asarray(a).view(np.uint32), np.asarray(b).view(np.uint32))


@pytest.fixture(scope="module")
def work():
    """Generates the inputs of the chain, the outlier tensors and the wide/narrow-code tensor on the GPU, keeps
    them there, and starts the oracle on all of them."""
    free, _ = torch.cuda.mem_get_info()
    if free < 40e9:
        pytest.skip("needs about 40 GB of free device memory")
    out = {}
    # ---- the chain: embedding + the first layer of the 410M shape -------------------------------
    shapes = synth.tensor_list(synth.CONFIG_SHAPES["pythia-410m"])[:13]
    w0 = [synth.make_quad(n, 77, i, device=DEV)[1] for i, (_, n) in enumerate(shapes)]
    steps, w_true = [], w0
    for k in range(CHAIN_STEPS):
        quads = [synth.make_quad(n, 77, i, device=DEV, step=k + 1, w_prev=w_true[i]) for i, (_, n) in enumerate(shapes)]
        steps.append([(q[0], q[2], q[3]) for q in quads])          # W_(k+1) = W_k + delta_k, fresh moments
        w_true = [q[0] for q in quads]
    out["chain"] = dict(shapes=shapes, w0=w0, steps=steps,
                        jobs=[oracle_pool.submit_chain(cpu(w0[i]), [tuple(cpu(t) for t in steps[k][i]) for k in range(CHAIN_STEPS)],
                                                       PARAMS_RES, i) for i in range(len(shapes))])
    # ---- threshold stress: 1 % of the residual at 10x, Pythia-1.4B-shaped tensors --------------
    s14 = synth.tensor_list(synth.CONFIG_SHAPES["pythia-1.4b"])
    picks = [0, next(i for i, (name, _) in enumerate(s14) if name.endswith("fc1.w"))]
    quads = [synth.make_quad(s14[i][1], 5, i, device=DEV, outlier_frac=0.01) for i in picks]
    out["outliers"] = dict(quads=quads, jobs=[oracle_pool.submit_compress(tuple(cpu(t) for t in q), PARAMS_RES, j, True)
                                              for j, q in enumerate(quads)])
    # ---- 2- and 8-bit codes, an ablation combination, on one 17 M tensor ------------------------
    n = 17_000_005
    q = synth.make_quad(n, 9, 0, device=DEV)
    variants = [dict(bits=2, kmeans_iters=10, median_source=1, seed=4),
                dict(bits=8, kmeans_iters=2, median_source=1, seed=4),
                dict(bits=4, kmeans_iters=10, median_source=1, seed=4, flags=binding.FLAG_NO_W2M | binding.FLAG_NO_M2W)]
    out["variants"] = dict(quad=q, params=variants,
                           jobs=[oracle_pool.submit_compress(tuple(cpu(t) for t in q), v, 0) for v in variants])
    yield out
    oracle_pool.shutdown()


def test_pythia410m_checkpoint_in_full_with_both_medians(work):
    shapes = synth.tensor_list(synth.CONFIG_SHAPES["pythia-410m"])
    n_tot = sum(n for _, n in shapes)
    quads = [synth.make_quad(n, 1000, i, device=DEV) for i, (_, n) in enumerate(shapes)]
    jobs = [oracle_pool.submit_compress(tuple(cpu(t) for t in q), [PARAMS_RES, PARAMS_W], i, want_decode=(i < 14))
            for i, q in enumerate(quads)]
    h = binding.Handle(workspace_numel=150_000_000)               # three groups of tensors
    try:
        blob = torch.empty(sum(binding.compress_bound(n) for _, n in shapes), dtype=torch.uint8, device=DEV)
        got = {}
        for mode in (1, 0):
            offs, stats = h.compress_checkpoint(binding.Params(kmeans_iters=10, median_source=mode), quads, blob)
            raw = blob[:offs[-1]].cpu().numpy().tobytes()
            got[mode] = ([raw[offs[i]:offs[i + 1]] for i in range(len(shapes))], stats, offs[-1])
            if mode == 1:                                          # Algorithm 2 on the leading tensors
                w_out = [q[1].clone() for q in quads[:14]]
                ea_out = [torch.empty_like(q[1]) for q in quads[:14]]
                eas_out = [torch.empty_like(q[1]) for q in quads[:14]]
                h.decompress_checkpoint(blob, offs[:15], w_out, w_out, ea_out, eas_out)
                decoded = [tuple(cpu(t) for t in trio) for trio in zip(w_out, ea_out, eas_out)]
        for i, job in enumerate(jobs):
            res = job.get(900)
            for mode, want in ((1, res[0]), (0, res[1])):
                recs, stats, _ = got[mode]
                tag = f"tensor {i} {shapes[i]}, median source {mode}"
                assert (stats[i].nnz_w, stats[i].nnz_o) == (want["nnz_w"], want["nnz_o"]), tag
                assert same_bits(np.float32(stats[i].median), want["median"]), tag
                assert same_bits(np.float32(stats[i].mean_abs_ea), want["mean_abs_ea"]), tag
                assert recs[i] == want["record"], tag
            if i < 14:
                for a, b in zip(decoded[i], res[0]["decoded"]):
                    assert same_bits(a, b), f"decoded tensor {i}"
        # the sizes the two readings of Eq. (rw) give on this distribution
        assert 15 < 12 * n_tot / got[1][2] < 30
        assert 45 < 12 * n_tot / got[0][2] <= 48                    # the literal median keeps almost nothing: two bitmaps = 12 B / 48
    finally:
        h.close()


def test_outlier_residuals_on_the_largest_14b_shaped_tensors(work):
    quads = work["outliers"]["quads"]
    h = binding.Handle(workspace_numel=max(q[0].numel() for q in quads))
    try:
        blob = torch.empty(sum(binding.compress_bound(q[0].numel()) for q in quads), dtype=torch.uint8, device=DEV)
        offs, stats = h.compress_checkpoint(binding.Params(kmeans_iters=10, median_source=1), quads, blob)
        w_out = [q[1].clone() for q in quads]
        ea_out = [torch.empty_like(q[1]) for q in quads]
        eas_out = [torch.empty_like(q[1]) for q in quads]
        h.decompress_checkpoint(blob, offs, w_out, w_out, ea_out, eas_out)
        for j, job in enumerate(work["outliers"]["jobs"]):
            want = job.get(900)
            assert (stats[j].nnz_w, stats[j].nnz_o) == (want["nnz_w"], want["nnz_o"])
            assert blob[offs[j]:offs[j + 1]].cpu().numpy().tobytes() == want["record"], j
            for a, b in zip((w_out[j], ea_out[j], eas_out[j]), want["decoded"]):
                assert same_bits(cpu(a), b)
            assert 0.4 < stats[j].nnz_w / quads[j][0].numel() < 0.65    # the median shrugs the outliers off
    finally:
        h.close()


def test_code_widths_and_switches_on_a_17m_tensor(work):
    q = work["variants"]["quad"]
    n = q[0].numel()
    h = binding.Handle(workspace_numel=n)
    try:
        blob = torch.empty(binding.compress_bound(n, 8), dtype=torch.uint8, device=DEV)
        for v, job in zip(work["variants"]["params"], work["variants"]["jobs"]):
            nbytes, st = h.compress_tensor(binding.Params(**v), *q, blob)
            want = job.get(900)
            assert (st.nnz_w, st.nnz_o) == (want["nnz_w"], want["nnz_o"]), v
            assert blob[:nbytes].cpu().numpy().tobytes() == want["record"], v
    finally:
        h.close()


def test_chain_of_eight_checkpoints_has_no_drift(work):
    ch = work["chain"]
    shapes, w0, steps = ch["shapes"], ch["w0"], ch["steps"]
    nt = len(shapes)
    h = binding.Handle(workspace_numel=sum(n for _, n in shapes) + 4096 * nt)
    try:
        p = binding.Params(kmeans_iters=10, median_source=1)
        cap = sum(binding.compress_bound(n) for _, n in shapes)
        w_hat = [w.clone() for w in w0]
        ea_out = [torch.empty_like(w) for w in w0]
        eas_out = [torch.empty_like(w) for w in w0]
        blobs = []
        for k in range(CHAIN_STEPS):                               # Algorithm 1 against the last reconstruction, then Algorithm 2 in place
            blob = torch.empty(cap, dtype=torch.uint8, device=DEV)
            quads = [(steps[k][i][0], w_hat[i], steps[k][i][1], steps[k][i][2]) for i in range(nt)]
            offs, _ = h.compress_checkpoint(p, quads, blob)
            h.decompress_checkpoint(blob, offs, w_hat, w_hat, ea_out, eas_out)
            blobs.append((blob[:offs[-1]].clone(), offs))
            del blob
        # Algorithm 3: the whole chain again from the initial weights
        w_again = [w.clone() for w in w0]
        for blob, offs in blobs:
            h.decompress_checkpoint(blob, offs, w_again, w_again, ea_out, eas_out)
        for i, job in enumerate(ch["jobs"]):
            want = job.get(1500)
            for k, (blob, offs) in enumerate(blobs):
                assert blob[offs[i]:offs[i + 1]].cpu().numpy().tobytes() == want["records"][k], (i, k)
            assert same_bits(cpu(w_hat[i]), want["w_hat"]) and same_bits(cpu(w_again[i]), want["w_hat"]), i
            assert same_bits(cpu(ea_out[i]), want["ea_hat"]) and same_bits(cpu(eas_out[i]), want["eas_hat"]), i
    finally:
        h.close()
