"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs.  Masks, bitmaps, counts, codes and whole records must
be bit-identical; centres and reconstructions are held to 1e-6 * max|dW| (and
are expected to be identical too)."""
import math

import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding, synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(workspace_numel=6_000_000)
    h.set_report_sse(True)
    yield h
    h.close()


def to_dev(quads):
    return [tuple(torch.as_tensor(a).to(DEV).contiguous() for a in q) for q in quads]


def to_np(quads):
    return [tuple(a.detach().cpu().numpy() for a in q) for q in quads]


def oparams(p: binding.Params) -> orc.Params:
    return orc.Params(alpha=p.alpha, beta=p.beta, bits=p.bits, kmeans_iters=p.kmeans_iters, seed=p.seed,
                      median_source=p.median_source, flags=p.flags)


def gpu_compress(h, p, dquads, capacity=None):
    bound = sum(binding.compress_bound(q[0].numel()) for q in dquads) if capacity is None else capacity
    blob = torch.full((max(bound, 16),), 0xAB, dtype=torch.uint8, device=DEV)   # dirty on purpose
    offs, stats = h.compress_checkpoint(p, dquads, blob)
    return blob, offs, stats


def check_against_oracle(p, quads_np, blob_t, offs, stats, first_index=0):
    raw = blob_t.cpu().numpy().tobytes()
    for i, (w_t, w_prev, ea, eas) in enumerate(quads_np):
        want, info = orc.compress_tensor(w_t, w_prev, ea, eas, oparams(p), tensor_index=first_index + i)
        st = stats[i]
        tag = f"tensor {i} (numel {w_t.size})"
        assert np.float32(st.median).view(np.uint32) == np.float32(info["median"]).view(np.uint32), tag
        assert np.float32(st.mean_abs_ea).view(np.uint32) == np.float32(info["mean_abs_ea"]).view(np.uint32), tag
        assert st.thr_w == info["thr_w"] and st.thr_o == info["thr_o"], tag
        assert (st.nnz_w, st.nnz_o) == (info["nnz_w"], info["nnz_o"]), tag
        for got_sse, want_sse in ((st.sse_w, info["sse_w"]), (st.sse_ea, info["sse_ea"]), (st.sse_eas, info["sse_eas"])):
            assert math.isclose(got_sse, want_sse, rel_tol=1e-5, abs_tol=0.0), tag    # a diagnostic: fp32 squares, sums in another order
        got = raw[offs[i]:offs[i + 1]]
        assert len(got) == len(want) == st.blob_bytes, tag
        rec = orc.parse_record(got)
        np.testing.assert_array_equal(rec["m_w"], info["m_w"], err_msg=tag)
        np.testing.assert_array_equal(rec["m_o"], info["m_o"], err_msg=tag)
        tol = 1e-6 * (float(np.abs(info["dw"]).max()) if w_t.size else 0.0)
        for c, s in (("c_w", "s_w"), ("c_ea", "s_ea"), ("c_eas", "s_eas")):
            scale = float(np.abs(info[s]).max()) if info[s].size else 0.0
            assert np.abs(rec[c].astype(np.float64) - info[c]).max() <= max(tol, 1e-6 * scale), (tag, c)
            np.testing.assert_array_equal(rec[c].view(np.uint32), info[c].view(np.uint32), err_msg=f"{tag} {c}")
        for c in ("codes_w", "codes_ea", "codes_eas"):
            np.testing.assert_array_equal(rec[c], info[c], err_msg=f"{tag} {c}")
        assert got == want, tag


def rand_quad_np(n, seed, scale_ea=1e-4):
    rng = np.random.default_rng(seed)
    w_prev = (rng.standard_normal(n) * 0.02).astype(np.float32)
    dw = (rng.standard_t(3, n) * 1e-4 / math.sqrt(3)).astype(np.float32)
    w_t = (w_prev + dw).astype(np.float32)
    ea = (rng.standard_normal(n) * scale_ea).astype(np.float32)
    eas = ((np.abs(rng.standard_normal(n)) * 1e-4) ** 2 + 1e-12).astype(np.float32)
    return w_t, w_prev, ea, eas


# ------------------------------------------------------------------ compress
@pytest.mark.parametrize("mode", [binding.MEDIAN_ABS_WEIGHT, binding.MEDIAN_ABS_RESIDUAL])
def test_hand_example(handle, mode):
    g = {}
    import os
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "hand_example.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split(":", 1)
            g[k.strip()] = v.split()
    f = lambda k: np.array([float(x) for x in g[k]], np.float32)
    q = [(f("w_t"), f("w_prev"), f("ea"), f("eas"))]
    p = binding.Params(alpha=0.25, beta=0.5, median_source=mode)
    blob, offs, stats = gpu_compress(handle, p, to_dev(q))
    check_against_oracle(p, q, blob, offs, stats)
    tag = "abs_weight" if mode == 0 else "abs_residual"
    raw = blob.cpu().numpy()
    assert raw[256] == int(g["bitmap_w_" + tag][0], 16) and raw[272] == int(g["bitmap_o_" + tag][0], 16)


@pytest.mark.parametrize("n", [0, 1, 3, 31, 32, 33, 127, 129, 4095, 4096, 4097, 10007, 3 * 4096 + 5, 100003])
def test_edge_sizes_residual_median(handle, n):
    q = [rand_quad_np(n, 100 + n)]
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=n)
    blob, offs, stats = gpu_compress(handle, p, to_dev(q))
    check_against_oracle(p, q, blob, offs, stats)


@pytest.mark.parametrize("n", [1, 33, 4097, 50001])
def test_edge_sizes_weight_median(handle, n):
    # the literal reading keeps almost nothing on these distributions; alpha is lowered so
    # that the quantiser still sees survivors
    q = [rand_quad_np(n, 200 + n)]
    p = binding.Params(alpha=2e-7, median_source=binding.MEDIAN_ABS_WEIGHT)
    blob, offs, stats = gpu_compress(handle, p, to_dev(q))
    check_against_oracle(p, q, blob, offs, stats)
    if n > 1000:
        assert stats[0].nnz_w > n // 10


def test_tiny_checkpoint_both_modes(handle):
    ck = synth.make_checkpoint("tiny", global_seed=3, device=DEV)
    dquads = [c[1:] for c in ck]
    quads = to_np(dquads)
    for mode in (binding.MEDIAN_ABS_RESIDUAL, binding.MEDIAN_ABS_WEIGHT):
        p = binding.Params(median_source=mode, seed=11)
        blob, offs, stats = gpu_compress(handle, p, dquads)
        assert offs[0] == 0 and all(b - a == s.blob_bytes for a, b, s in zip(offs, offs[1:], stats))
        check_against_oracle(p, quads, blob, offs, stats)


def test_many_groups_and_tensor_index(handle):
    """A workspace smaller than the checkpoint splits it into groups; records,
    offsets and the per-tensor start samples must not notice."""
    sizes = [5000, 0, 70000, 1, 4096, 130000, 33, 8192, 99999]
    quads = [rand_quad_np(n, 300 + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=5)
    small = binding.Handle(workspace_numel=140_000)
    small.set_report_sse(True)
    try:
        blob, offs, stats = gpu_compress(small, p, dquads)
        check_against_oracle(p, quads, blob, offs, stats)
        blob2, offs2, _ = gpu_compress(handle, p, dquads)
        assert offs == offs2 and torch.equal(blob[:offs[-1]], blob2[:offs2[-1]])
    finally:
        small.close()


def test_outlier_residuals_and_run_to_run_determinism(handle):
    dq = [synth.make_quad(300_000, 9, 0, device=DEV, outlier_frac=0.01),
          synth.make_quad(50_000, 9, 1, device=DEV, outlier_frac=0.01)]
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL)
    blob, offs, stats = gpu_compress(handle, p, dq)
    check_against_oracle(p, to_np(dq), blob, offs, stats)
    for _ in range(3):
        b2, o2, _ = gpu_compress(handle, p, dq)
        assert o2 == offs and torch.equal(b2[:offs[-1]], blob[:offs[-1]])


def test_centres_do_not_depend_on_which_cells_were_gathered(handle):
    """The K-means iterations read only the value cells their thresholds fall into.  Whatever the first
    round gathers (nothing: margin -1, so every stream takes the complete second round; only the
    predicted cells: 0; more: 1, 5), the records are the oracle's plain Lloyd iterations."""
    n = 2_000_000
    dq = [synth.make_quad(n, 21, 0, device=DEV), synth.make_quad(70_000, 21, 1, device=DEV, outlier_frac=0.01)]
    h = binding.Handle(workspace_numel=n + 80_000)
    h.set_report_sse(True)
    try:
        for bits in (4, 2):
            p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, bits=bits, seed=5)
            ref = None
            for margin in (1, -1, 0, 5):
                h.set_kmeans_margin(margin)
                bound = sum(binding.compress_bound(q[0].numel(), bits) for q in dq)
                blob = torch.full((bound,), 0xCD, dtype=torch.uint8, device=DEV)
                offs, stats = h.compress_checkpoint(p, dq, blob)
                if ref is None:
                    check_against_oracle(p, to_np(dq), blob, offs, stats)
                    ref = (blob[:offs[-1]].clone(), offs)
                else:
                    assert offs == ref[1] and torch.equal(blob[:offs[-1]], ref[0]), (bits, margin)
        with pytest.raises(binding.ExcpError):
            h.set_kmeans_margin(-2)
    finally:
        h.close()


def test_degenerate_value_patterns(handle):
    n = 20000
    base = rand_quad_np(n, 400)
    cases = []
    w_t, w_prev, ea, eas = (a.copy() for a in base)                # all residuals equal in magnitude
    w_prev[:] = 0.0; w_t[:] = 0.125; w_t[::2] = -0.125; eas[:] = 1.0
    cases.append((w_t, w_prev, ea, eas))
    w_t, w_prev, ea, eas = (a.copy() for a in base)                # nothing changed: all pruned
    cases.append((w_prev.copy(), w_prev, ea, eas))
    w_t, w_prev, ea, eas = (a.copy() for a in base)                # ea over a huge exponent range
    ea[::3] *= np.float32(1e-30); ea[1::3] *= np.float32(1e20); ea[5] = 0.0; ea[7] = 1e-45
    cases.append((w_t, w_prev, ea, eas))
    w_t, w_prev, ea, eas = (a.copy() for a in base)                # zeros in the second moment, constant ea
    eas[::2] = 0.0; ea[:] = 3e-4; ea[::5] = -3e-4
    cases.append((w_t, w_prev, ea, eas))
    w_t, w_prev, ea, eas = (a.copy() for a in base)                # fewer survivors than centres
    w_t[:] = w_prev; w_t[[5, 77, 4099, 19999]] += np.float32([0.5, -0.25, 0.125, 1.0])
    cases.append((w_t, w_prev, ea, eas))
    for mode in (0, 1):
        p = binding.Params(median_source=mode, beta=0.5)
        blob, offs, stats = gpu_compress(handle, p, to_dev(cases))
        check_against_oracle(p, cases, blob, offs, stats)


def test_median_when_the_sample_misleads(handle):
    """The median is bracketed from 65536 evenly spaced elements.  Here every 16th element (the
    ones a 2^20-element tensor's sample takes) is large, so the bracket misses the true median
    and the histogram path has to find it; a second tensor is exactly as large as the sample."""
    n = 1 << 20
    w_t, w_prev, ea, eas = rand_quad_np(n, 450)
    w_t[::16] = w_prev[::16] + np.float32(0.5)
    w_prev2 = rand_quad_np(65536, 451)
    cases = [(w_t, w_prev, ea, eas), w_prev2, rand_quad_np(65537, 452)]
    for mode in (0, 1):
        p = binding.Params(median_source=mode, alpha=2e-7 if mode == 0 else 5e-5)
        if mode == 0:
            cases[0][0][::16] = np.float32(7.0)
        blob, offs, stats = gpu_compress(handle, p, to_dev(cases))
        check_against_oracle(p, cases, blob, offs, stats)


def test_zero_kmeans_iterations_and_other_hyperparameters(handle):
    q = [rand_quad_np(60000, 500)]
    for p in (binding.Params(kmeans_iters=0, median_source=1), binding.Params(kmeans_iters=3, median_source=1, seed=99),
              binding.Params(alpha=0.0, beta=0.0, median_source=1), binding.Params(alpha=1e9, median_source=1)):
        blob, offs, stats = gpu_compress(handle, p, to_dev(q))
        check_against_oracle(p, q, blob, offs, stats)


# ---------------------------------------------------------------- decompress
def gpu_decompress(h, blob, offs, dquads, in_place=False):
    w_prev = [q[1].clone() for q in dquads]
    w_out = w_prev if in_place else [torch.full_like(t, 7.0) for t in w_prev]
    ea_out = [torch.full_like(t, 7.0) for t in w_prev]
    eas_out = [torch.full_like(t, 7.0) for t in w_prev]
    h.decompress_checkpoint(blob, offs, w_prev, w_out, ea_out, eas_out)
    return w_out, ea_out, eas_out


def test_decompress_matches_oracle_and_in_place(handle):
    sizes = [0, 1, 33, 4097, 70001, 12288]
    quads = [rand_quad_np(n, 600 + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL)
    blob, offs, stats = gpu_compress(handle, p, dquads)
    raw = blob.cpu().numpy().tobytes()
    for in_place in (False, True):
        w_out, ea_out, eas_out = gpu_decompress(handle, blob, offs, dquads, in_place)
        for i, q in enumerate(quads):
            w_hat, ea_hat, eas_hat = orc.decompress_tensor(raw[offs[i]:offs[i + 1]], q[1])
            np.testing.assert_array_equal(w_out[i].cpu().numpy().view(np.uint32), w_hat.view(np.uint32))
            np.testing.assert_array_equal(ea_out[i].cpu().numpy().view(np.uint32), ea_hat.view(np.uint32))
            np.testing.assert_array_equal(eas_out[i].cpu().numpy().view(np.uint32), eas_hat.view(np.uint32))


def test_gpu_decodes_a_record_written_by_the_oracle(handle):
    q = rand_quad_np(33333, 700)
    want_blob, info = orc.compress_tensor(*q, orc.Params(median_source=1, seed=4))
    blob = torch.frombuffer(bytearray(want_blob), dtype=torch.uint8).to(DEV)
    w_prev = torch.as_tensor(q[1]).to(DEV)
    outs = [torch.empty_like(w_prev) for _ in range(3)]
    handle.decompress_tensor(blob, len(want_blob), w_prev, *outs)
    for got, want in zip(outs, orc.decompress_tensor(want_blob, q[1])):
        np.testing.assert_array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_chain_of_checkpoints_has_no_drift(handle):
    """Eight steps, each residual against the previous RECONSTRUCTION (Section 3.4,
    Algorithm 3's loop): the GPU chain and the oracle chain stay identical."""
    n, steps = 150_000, 8
    w_true = synth.make_quad(n, 21, 0, device=DEV)[1]
    w_hat_gpu = w_true.clone()
    w_hat_cpu = w_true.cpu().numpy().copy()
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=2)
    blob = torch.empty(binding.compress_bound(n), dtype=torch.uint8, device=DEV)
    for k in range(steps):
        w_next, _, ea, eas = synth.make_quad(n, 21, 0, device=DEV, step=k + 1, w_prev=w_true)
        nbytes, st = handle.compress_tensor(p, w_next, w_hat_gpu, ea, eas, blob)
        want, info = orc.compress_tensor(w_next.cpu().numpy(), w_hat_cpu, ea.cpu().numpy(), eas.cpu().numpy(), oparams(p))
        assert blob[:nbytes].cpu().numpy().tobytes() == want, f"step {k}"
        ea_o, eas_o = torch.empty_like(ea), torch.empty_like(ea)
        handle.decompress_tensor(blob, nbytes, w_hat_gpu, w_hat_gpu, ea_o, eas_o)     # in place
        w_hat_cpu, ea_c, eas_c = orc.decompress_tensor(want, w_hat_cpu)
        np.testing.assert_array_equal(w_hat_gpu.cpu().numpy().view(np.uint32), w_hat_cpu.view(np.uint32))
        np.testing.assert_array_equal(ea_o.cpu().numpy(), ea_c)
        assert float((w_next - w_hat_gpu).abs().max()) <= float(np.abs(info["dw"]).max())
        w_true = w_next


# -------------------------------------------------------------------- errors
def test_error_codes(handle):
    q = rand_quad_np(5000, 800)
    dq = to_dev([q])
    p = binding.Params(median_source=1)
    blob = torch.empty(binding.compress_bound(5000), dtype=torch.uint8, device=DEV)
    for k in range(4):                                       # NaN / Inf anywhere, negative second moment
        bad = [t.clone() for t in dq[0]]
        bad[k][1234] = float("nan") if k % 2 else float("inf")
        with pytest.raises(binding.ExcpError) as e:
            handle.compress_tensor(p, *bad, blob)
        assert e.value.status == -6
    bad = [t.clone() for t in dq[0]]
    bad[3][17] = -1e-9
    with pytest.raises(binding.ExcpError) as e:
        handle.compress_tensor(p, *bad, blob)
    assert e.value.status == -6
    with pytest.raises(binding.ExcpError) as e:              # record does not fit
        handle.compress_tensor(p, *dq[0], blob[:512])
    assert e.value.status == -3
    with pytest.raises(binding.ExcpError) as e:              # misaligned input
        handle.compress_tensor(p, dq[0][0][1:], dq[0][1][1:], dq[0][2][1:], dq[0][3][1:], blob)
    assert e.value.status == -1
    for bits, code in ((5, -1), (16, -1)):                   # widths other than 2, 4, 8
        with pytest.raises(binding.ExcpError) as e:
            handle.compress_tensor(binding.Params(bits=bits), *dq[0], blob)
        assert e.value.status == code
    with pytest.raises(binding.ExcpError) as e:              # tensor larger than the workspace
        big = torch.zeros(7_000_000, device=DEV)
        handle.compress_tensor(p, big, big, big, big, torch.empty(binding.compress_bound(7_000_000), dtype=torch.uint8, device=DEV))
    assert e.value.status == -1
    nbytes, _ = handle.compress_tensor(p, *dq[0], blob)      # the handle still works afterwards
    assert nbytes > 0


def test_corrupt_records_are_refused_without_faulting(handle):
    q = rand_quad_np(9000, 900)
    dq = to_dev([q])[0]
    p = binding.Params(median_source=1)
    blob = torch.empty(binding.compress_bound(9000), dtype=torch.uint8, device=DEV)
    nbytes, st = handle.compress_tensor(p, *dq, blob)
    outs = [torch.empty_like(dq[1]) for _ in range(3)]
    codes_w = 256 + 2 * orc.bitmap_bytes(9000)
    assert st.nnz_w > 16
    for pos, flip in ((0, 1), (4, 3), (8, 1), (16, 0x80), (24, 0x80), (32, 12), (48, 0x10), (256, 1), (codes_w + 3, None)):
        bad = blob.clone()
        bad[pos] = 0 if flip is None else (int(bad[pos]) ^ flip)
        with pytest.raises(binding.ExcpError) as e:
            handle.decompress_tensor(bad, nbytes, dq[1], *outs)
        assert e.value.status == -5, pos
    with pytest.raises(binding.ExcpError) as e:              # truncated
        handle.decompress_tensor(blob, nbytes - 16, dq[1], *outs)
    assert e.value.status == -5
    handle.decompress_tensor(blob, nbytes, dq[1], *outs)     # the intact record still decodes
    # A bit set past the last element, with the populations kept equal to the header's counts (a kept weight whose
    # moments are pruned is cleared in exchange): only the rule "no bit at or past numel" catches it; the oracle
    # refuses the same bytes.
    raw = bytearray(blob[:nbytes].cpu().numpy().tobytes())
    r = orc.parse_record(bytes(raw))
    victim = int(np.flatnonzero(r["m_w"] & ~r["m_o"])[-1])
    raw[256 + victim // 8] ^= 1 << (victim % 8)
    stray = 9000 + 5                                          # 9000 = 281 * 32 + 8: bit 13 of the last word
    raw[256 + stray // 8] |= 1 << (stray % 8)
    with pytest.raises(orc.CorruptBlob):
        orc.parse_record(bytes(raw))
    bad = torch.frombuffer(raw, dtype=torch.uint8).to(DEV)
    with pytest.raises(binding.ExcpError) as e:
        handle.decompress_tensor(bad, nbytes, dq[1], *outs)
    assert e.value.status == -5


# ----------------------------------------------------------------- host path
def test_host_buffer_path_gives_the_same_records(handle):
    sizes = [5000, 0, 70000, 1, 4096, 130000, 33, 8192, 99999, 64000]
    quads = [rand_quad_np(n, 1000 + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=8)
    blob, offs, stats = gpu_compress(handle, p, dquads)
    small = binding.Handle(workspace_numel=140_000)          # several groups: both staging slots reused
    try:
        hquads = [tuple(torch.as_tensor(a).pin_memory() for a in q) for q in quads]
        hblob = torch.full((offs[-1] + 64,), 0xCD, dtype=torch.uint8).pin_memory()
        for _ in range(2):
            hoffs, hstats = small.compress_checkpoint_host(p, hquads, hblob)
            assert hoffs == offs
            assert bytes(hblob[:offs[-1]].numpy()) == blob[:offs[-1]].cpu().numpy().tobytes()
            assert [s.nnz_w for s in hstats] == [s.nnz_w for s in stats]
        with pytest.raises(binding.ExcpError) as e:
            small.compress_checkpoint_host(p, hquads, hblob[:offs[-1] - 16])
        assert e.value.status == -3
    finally:
        small.close()


def test_host_buffer_path_with_wide_codes_and_every_element_kept():
    """Records far larger than 4-bit ones (8-bit codes, nothing pruned) through the host-buffer entry point: the
    device staging grows with the code width, the records equal the device path's, and a host buffer that is too
    small is refused with status -3 before anything is copied past the staging."""
    sizes = [70000, 4096, 130000, 33, 64000]
    quads = [rand_quad_np(n, 1100 + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    small = binding.Handle(workspace_numel=140_000)
    try:
        hquads = [tuple(torch.as_tensor(a).pin_memory() for a in q) for q in quads]
        p4 = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=8)
        cap4 = sum(binding.compress_bound(n) for n in sizes)
        small.compress_checkpoint_host(p4, hquads, torch.empty(cap4, dtype=torch.uint8).pin_memory())   # staging sized for 4 bits
        p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=8, bits=8, kmeans_iters=3,
                           flags=binding.FLAG_NO_PRUNE)
        cap = sum(binding.compress_bound(n, 8) for n in sizes)
        blob = torch.full((cap,), 0xAB, dtype=torch.uint8, device=DEV)
        offs, stats = small.compress_checkpoint(p, dquads, blob)
        assert [s.nnz_w for s in stats] == sizes and offs[-1] > cap4
        hblob = torch.full((cap,), 0xCD, dtype=torch.uint8).pin_memory()
        hoffs, hstats = small.compress_checkpoint_host(p, hquads, hblob)
        assert hoffs == offs
        assert bytes(hblob[:offs[-1]].numpy()) == blob[:offs[-1]].cpu().numpy().tobytes()
        with pytest.raises(binding.ExcpError) as e:
            small.compress_checkpoint_host(p, hquads, hblob[:offs[-1] - 16])
        assert e.value.status == -3
        hoffs, _ = small.compress_checkpoint_host(p, hquads, hblob)              # the handle is still usable
        assert hoffs == offs
    finally:
        small.close()


def test_a_share_of_a_checkpoint_gives_the_whole_lists_records(handle):
    """excp_compress_checkpoint_indexed: the tensors dealt to two ranks, each share compressed on its own with the
    tensors' checkpoint-wide indices, give together exactly the records (and, assembled, the blob and the offsets)
    of one call over the whole list."""
    from paper_2406_11257_b200 import ranks
    sizes = [30000, 5000, 70000, 0, 4096, 130000, 33, 8192, 99999]
    dquads = to_dev([rand_quad_np(n, 1300 + i) for i, n in enumerate(sizes)])
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=21)
    blob, offs, _ = gpu_compress(handle, p, dquads)
    whole = blob[:offs[-1]].cpu().numpy().tobytes()
    shares = ranks.partition_tensors(sizes, 2)
    blobs, local = [], []
    for idx in shares:
        b = torch.empty(sum(binding.compress_bound(sizes[i]) for i in idx) + 16, dtype=torch.uint8, device=DEV)
        o, _ = handle.compress_checkpoint(p, [dquads[i] for i in idx], b, tensor_indices=idx)
        blobs.append(b[:o[-1]].cpu().numpy().tobytes())
        local.append(o)
    table, goffs = ranks.assemble_offsets(sizes, shares, local)
    assert goffs == offs
    assert ranks.assemble_blob(table, blobs) == whole


def test_a_wait_that_runs_out_comes_back_as_status_minus_7(handle):
    """The bounded waits: a barrier that nothing completes makes the wait run out after the given time (no copy is
    in flight, nothing faults); a whole compress call whose waits are given no time at all returns -7 after every
    warp has let its own copies land, the later kernels of the call do nothing, and the handle works afterwards."""
    import time
    t0 = time.time()
    assert handle.selftest_wait_timeout(5_000_000) == -7          # 5 ms
    assert time.time() - t0 < 10
    assert handle.selftest_wait_timeout(0) == -7
    q = rand_quad_np(300_000, 1400)
    dq = to_dev([q])
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=2)
    blob = torch.empty(binding.compress_bound(300_000), dtype=torch.uint8, device=DEV)
    handle.set_wait_limit(0)
    try:
        with pytest.raises(binding.ExcpError) as e:
            handle.compress_tensor(p, *dq[0], blob)
        assert e.value.status == -7
    finally:
        handle.set_wait_limit(2_000_000_000)
    blob2, offs, stats = gpu_compress(handle, p, dq)
    check_against_oracle(p, [q], blob2, offs, stats)


def test_profile_counts_launches_and_times_stages(handle):
    dq = [synth.make_quad(200_000, 3, 0, device=DEV)]
    blob = torch.empty(binding.compress_bound(200_000), dtype=torch.uint8, device=DEV)
    handle.profile_enable(True)
    try:
        handle.compress_tensor(binding.Params(median_source=1, kmeans_iters=10), *dq[0], blob)
        ms, launches = handle.profile_read()
        # statistics, mask sweep, scan + layout, K-means (start, 2 counting sweeps, plan, 2 gathers, iterations,
        # the second and third rounds' 4 each), header + edges, 2 packing sweeps, bitmaps
        assert launches == 11 + 1 + 2 + (1 + 2 + 1 + 2 + 1 + 4 + 4) + 2 + 2 + 1
        assert ms["mask_compact"] > 0 and ms["kmeans_iterate"] > 0 and ms["decode"] == 0
    finally:
        handle.profile_enable(False)
