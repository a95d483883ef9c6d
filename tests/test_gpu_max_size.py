"""The largest tensor the library takes: just under 2^31 elements (34 GB of inputs), with a ragged tail.

The oracle needs a quarter of an hour for a tensor of this size, so what is checked here are properties that
hold at any size and that plain torch operations on the GPU establish without the library:
  * the median is THE order statistic of rank floor((n-1)/2): fewer than rank+1 elements lie below it and at
    least rank+1 at or below it;
  * the mean of |ea| agrees with a float64 sum;
  * M_w is exactly [ |dW| * sqrt(eas) > alpha * median ] (fp32, correctly rounded root) and M_o exactly
    [ |ea| > beta * mean ] and M_w: the populations and a slice of both bitmaps at either end of the tensor;
  * the record's size and header follow from the populations;
  * Algorithm 2 in place: pruned weights keep W^_(t-1) bit for bit, kept ones move by one of the record's 15
    centres, pruned moments are 0, kept ones are centres; the ragged tail is written and nothing past it.
From the oracle only the layout arithmetic is used (record size, bitmap size)."""
import struct

import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
N = (1 << 31) - 4099                                              # not a multiple of 4, of 32 or of the tile


def fill(n, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    w_prev = torch.empty(n, dtype=torch.float32, device=DEV).normal_(0.0, 0.02, generator=g)
    w_t = torch.empty(n, dtype=torch.float32, device=DEV).normal_(0.0, 1e-4, generator=g).add_(w_prev)
    ea = torch.empty(n, dtype=torch.float32, device=DEV).normal_(0.0, 1e-4, generator=g)
    eas = torch.empty(n, dtype=torch.float32, device=DEV).normal_(0.0, 1e-4, generator=g).square_().add_(1e-12)
    return w_t, w_prev, ea, eas


def chunks(n, step=1 << 28):
    for a in range(0, n, step):
        yield a, min(n, a + step)


def test_a_tensor_of_nearly_two_to_the_31_elements():
    free, _ = torch.cuda.mem_get_info()
    if free < 130e9:
        pytest.skip("needs about 130 GB of free device memory")
    w_t, w_prev, ea, eas = fill(N, 31)
    h = binding.Handle(workspace_numel=N)
    try:
        p = binding.Params(kmeans_iters=10, median_source=binding.MEDIAN_ABS_RESIDUAL)
        blob = torch.empty(int(0.85 * N), dtype=torch.uint8, device=DEV)
        nbytes, st = h.compress_tensor(p, w_t, w_prev, ea, eas, blob)
        rank = (N - 1) // 2
        med = torch.tensor(st.median, dtype=torch.float32, device=DEV)
        thr_w = torch.tensor(st.thr_w, dtype=torch.float32, device=DEV)
        thr_o = torch.tensor(st.thr_o, dtype=torch.float32, device=DEV)
        below = at_or_below = nnz_w = nnz_o = 0
        sum_abs = 0.0
        for a, b in chunks(N):
            dw = w_t[a:b] - w_prev[a:b]
            mag = dw.abs()
            below += int((mag < med).sum())
            at_or_below += int((mag <= med).sum())
            m_w = mag * eas[a:b].sqrt() > thr_w
            m_o = (ea[a:b].abs() > thr_o) & m_w
            nnz_w += int(m_w.sum())
            nnz_o += int(m_o.sum())
            sum_abs += float(ea[a:b].abs().sum(dtype=torch.float64))
            del dw, mag, m_w, m_o
        assert below <= rank < at_or_below                          # the exact lower median
        assert abs(st.mean_abs_ea - sum_abs / N) <= 1e-6 * st.mean_abs_ea
        assert st.thr_w == float(np.float32(5e-5) * np.float32(st.median)) and st.thr_o == float(np.float32(2.0) * np.float32(st.mean_abs_ea))
        assert (st.nnz_w, st.nnz_o) == (nnz_w, nnz_o)
        want = orc.record_bytes(N, nnz_w, nnz_o, 4)
        assert nbytes == want == st.blob_bytes
        head = struct.unpack("<IIQQQIIIIQQ", blob[:64].cpu().numpy().tobytes())
        assert head == (orc.MAGIC, 1, N, nnz_w, nnz_o, 4, 15, 256, 0, want, 0)
        cent = np.frombuffer(blob[64:64 + 180].cpu().numpy().tobytes(), dtype=np.float32).reshape(3, 15)
        assert np.all(np.diff(cent, axis=1) >= 0)

        # both bitmaps at either end of the tensor against the masks computed here
        bm_bytes = orc.bitmap_bytes(N)
        span = 1 << 20
        for a in (0, (N - span) // 32 * 32):
            b = min(N, a + span)
            dw = w_t[a:b] - w_prev[a:b]
            m_w = (dw.abs() * eas[a:b].sqrt() > thr_w)
            m_o = (ea[a:b].abs() > thr_o) & m_w
            for off, mask in ((256, m_w), (256 + bm_bytes, m_o)):
                raw = blob[off + a // 8: off + (b + 7) // 8].cpu().numpy()
                got = np.unpackbits(raw, bitorder="little")[:b - a].astype(bool)
                assert np.array_equal(got, mask.cpu().numpy()), (a, off)
        tail = blob[256 + (N // 32) * 4: 256 + bm_bytes].cpu().numpy()            # the last word and the padding
        assert int(np.unpackbits(tail, bitorder="little")[N % 32:].sum()) == 0

        # Algorithm 2 in place, then what every element must satisfy
        keep = w_prev[N - 4096:].clone(), w_prev[:4096].clone()
        guard = torch.full((1024,), 7.0, dtype=torch.float32, device=DEV)       # not part of any tensor
        h.decompress_tensor(blob, nbytes, w_prev, w_prev, ea, eas)                # W^ over W^_(t-1), moments over moments
        assert float(guard.min()) == 7.0 and float(guard.max()) == 7.0
        cw = torch.tensor(cent[0], device=DEV)
        ca = torch.tensor(np.concatenate([[0.0], cent[1]]).astype(np.float32), device=DEV)
        cs = torch.tensor(np.concatenate([[0.0], cent[2]]).astype(np.float32), device=DEV)
        for a, b in ((0, 1 << 22), (N - (1 << 22), N)):
            assert bool(torch.isin(ea[a:b], ca).all()) and bool(torch.isin(eas[a:b], cs).all())
            assert int((ea[a:b] != 0).sum()) == int((eas[a:b] != 0).sum())
        old_tail, old_head = keep
        for old, new in ((old_head, w_prev[:4096]), (old_tail, w_prev[N - 4096:])):
            moved = new != old
            step = (new - old)[moved]
            near = (step[:, None] - cw[None, :]).abs().min(dim=1).values
            assert float(near.max()) <= 1.5e-8                       # W^_(t-1) + centre rounded once, the difference once more, at |w| < 0.125
            assert 0.3 < float(moved.float().mean()) < 0.7
        del keep
    finally:
        h.close()
        del w_t, w_prev, ea, eas
        torch.cuda.empty_cache()
