"""GPU parity for weights stored as float16 / bfloat16 (Section 4.3 notes float16 weights): the
record is byte for byte the oracle's (= that of the widened tensors) and Algorithm 2's weights are
the oracle's 16-bit patterns."""
import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding
from test_gpu_parity import DEV, rand_quad_np

pytestmark = pytest.mark.gpu

FMT = {binding.WEIGHTS_F16: (torch.float16, orc.WEIGHTS_F16), binding.WEIGHTS_BF16: (torch.bfloat16, orc.WEIGHTS_BF16)}


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(workspace_numel=700_000)
    yield h
    h.close()


def make(n, seed, fmt, scale=30.0):
    """Weights a 16-bit format can hold, with residuals that survive its rounding."""
    w_t, w_prev, ea, eas = rand_quad_np(n, seed)
    ofmt = FMT[fmt][1]
    wp16 = orc.narrow_weights(w_prev, ofmt)
    wt16 = orc.narrow_weights((orc.widen_weights(wp16, ofmt) + (w_t - w_prev) * np.float32(scale)).astype(np.float32), ofmt)
    return wt16, wp16, ea, eas


def dev16(a, fmt):
    t = torch.as_tensor(a.view(np.int16) if a.dtype != np.float32 else a).to(DEV)
    return t.view(FMT[fmt][0]) if a.dtype != np.float32 else t


def bits16(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("fmt", [binding.WEIGHTS_F16, binding.WEIGHTS_BF16])
@pytest.mark.parametrize("mode", [binding.MEDIAN_ABS_WEIGHT, binding.MEDIAN_ABS_RESIDUAL])
def test_sixteen_bit_weights_match_the_oracle(handle, fmt, mode):
    sizes = [0, 1, 7, 8, 9, 33, 4095, 4097, 70001, 12288, 300000, 65536, 65537, 100003]   # ragged tails of every residue
    quads = [make(n, 4000 + i, fmt) for i, n in enumerate(sizes)]
    dquads = [(dev16(q[0], fmt), dev16(q[1], fmt), torch.as_tensor(q[2]).to(DEV), torch.as_tensor(q[3]).to(DEV)) for q in quads]
    p = binding.Params(alpha=5e-5 if mode == 1 else 6e-6, median_source=mode, kmeans_iters=4)
    blob = torch.full((sum(binding.compress_bound(n) for n in sizes),), 0xAB, dtype=torch.uint8, device=DEV)
    offs, stats = handle.compress_checkpoint(p, dquads, blob, weight_format=fmt)
    raw = blob.cpu().numpy().tobytes()
    op = orc.Params(alpha=p.alpha, median_source=mode, kmeans_iters=4)
    kept = 0
    for i, q in enumerate(quads):
        want, info = orc.compress_tensor(*q, op, tensor_index=i, weight_format=FMT[fmt][1])
        assert np.float32(stats[i].median).view(np.uint32) == np.float32(info["median"]).view(np.uint32), i
        assert (stats[i].nnz_w, stats[i].nnz_o) == (info["nnz_w"], info["nnz_o"]), i
        assert raw[offs[i]:offs[i + 1]] == want, f"tensor {i} (numel {sizes[i]})"
        kept += info["nnz_w"]
    assert 0 < kept < sum(sizes)
    for in_place in (False, True):
        w_prev = [q[1].clone() for q in dquads]
        w_out = w_prev if in_place else [torch.full_like(t, 7.0) for t in w_prev]
        ea_out = [torch.full_like(q[2], 7.0) for q in dquads]
        eas_out = [torch.full_like(q[2], 7.0) for q in dquads]
        handle.decompress_checkpoint(blob, offs, w_prev, w_out, ea_out, eas_out, weight_format=fmt)
        for i, q in enumerate(quads):
            w_hat, ea_hat, eas_hat = orc.decompress_tensor(raw[offs[i]:offs[i + 1]], q[1], weight_format=FMT[fmt][1])
            np.testing.assert_array_equal(bits16(w_out[i]), w_hat.view(np.uint16), err_msg=f"tensor {i}")
            np.testing.assert_array_equal(ea_out[i].cpu().numpy().view(np.uint32), ea_hat.view(np.uint32))
            np.testing.assert_array_equal(eas_out[i].cpu().numpy().view(np.uint32), eas_hat.view(np.uint32))


@pytest.mark.parametrize("fmt", [binding.WEIGHTS_F16, binding.WEIGHTS_BF16])
def test_sixteen_bit_median_fallback_and_switches(handle, fmt):
    # the misleading-sample tensor (every 16th element large) takes the histogram path with 16-bit loads
    n = 1 << 20
    wt16, wp16, ea, eas = make(n, 4100, fmt)
    ofmt = FMT[fmt][1]
    w32 = orc.widen_weights(wp16, ofmt)
    big = w32.copy(); big[::16] += np.float32(0.5)
    wt16 = orc.narrow_weights(np.where(np.arange(n) % 16 == 0, big, orc.widen_weights(wt16, ofmt)).astype(np.float32), ofmt)
    q = (wt16, wp16, ea, eas)
    h2 = binding.Handle(workspace_numel=1 << 20)
    try:
        for flags in (0, binding.FLAG_NO_RESIDUAL | binding.FLAG_NO_W2M):
            p = binding.Params(alpha=5e-5, median_source=1, kmeans_iters=2, flags=flags)
            dq = (dev16(q[0], fmt), dev16(q[1], fmt), torch.as_tensor(ea).to(DEV), torch.as_tensor(eas).to(DEV))
            blob = torch.empty(binding.compress_bound(n), dtype=torch.uint8, device=DEV)
            offs, stats = h2.compress_checkpoint(p, [dq], blob, weight_format=fmt)
            want, info = orc.compress_tensor(*q, orc.Params(alpha=5e-5, median_source=1, kmeans_iters=2, flags=flags),
                                             weight_format=ofmt)
            assert blob[:offs[1]].cpu().numpy().tobytes() == want
            w_out = torch.empty_like(dq[1]); outs = [torch.empty_like(dq[2]) for _ in range(2)]
            h2.decompress_checkpoint(blob, offs, [dq[1]], [w_out], [outs[0]], [outs[1]], weight_format=fmt)
            w_hat, _, _ = orc.decompress_tensor(want, wp16, weight_format=ofmt)
            np.testing.assert_array_equal(bits16(w_out), w_hat.view(np.uint16))
    finally:
        h2.close()


def test_weight_format_errors(handle):
    q = make(5000, 4200, binding.WEIGHTS_F16)
    dq = (dev16(q[0], 1), dev16(q[1], 1), torch.as_tensor(q[2]).to(DEV), torch.as_tensor(q[3]).to(DEV))
    blob = torch.empty(binding.compress_bound(5000), dtype=torch.uint8, device=DEV)
    with pytest.raises(TypeError):                               # the binding checks the dtype against the format
        handle.compress_checkpoint(binding.Params(), [dq], blob, weight_format=binding.WEIGHTS_BF16)
    import ctypes as C
    n = 1
    arr = lambda t: (C.c_void_p * 1)(t.data_ptr())
    numel = (C.c_size_t * 1)(5000)
    offs = (C.c_size_t * 2)()
    cp = binding.Params().to_c()
    for bad in (0, 3, -1):                                       # only the two 16-bit formats
        st = handle.lib.excp_compress_checkpoint_w16(handle._h, C.byref(cp), n, arr(dq[0]), arr(dq[1]), arr(dq[2]), arr(dq[3]),
                                                     numel, bad, blob.data_ptr(), blob.numel(), offs, None,
                                                     torch.cuda.current_stream().cuda_stream)
        assert st == -1
