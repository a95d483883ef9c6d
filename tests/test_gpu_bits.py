"""GPU parity for the code widths of the paper's quantisation-bins table (2 and 8 bits: K = 3 and 255
centres) next to the method's 4: records byte-identical to the oracle's, Algorithm 2 bit-identical."""
import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding
from test_gpu_parity import DEV, check_against_oracle, gpu_compress, gpu_decompress, rand_quad_np, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(workspace_numel=700_000)
    h.set_report_sse(True)
    yield h
    h.close()


@pytest.mark.parametrize("bits", [2, 8])
@pytest.mark.parametrize("mode", [binding.MEDIAN_ABS_WEIGHT, binding.MEDIAN_ABS_RESIDUAL])
def test_code_widths_match_the_oracle(handle, bits, mode):
    # two groups; empty, tiny (fewer survivors than centres), ragged and tile-aligned tensors
    sizes = [0, 1, 5, 33, 300, 4097, 70001, 12288, 300000, 65536]
    quads = [rand_quad_np(n, 3000 + 10 * bits + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    p = binding.Params(alpha=5e-5 if mode == 1 else 2e-7, median_source=mode, bits=bits, kmeans_iters=5, seed=3)
    cap = sum(binding.record_bytes(n, n, n, bits) for n in sizes)
    blob, offs, stats = gpu_compress(handle, p, dquads, capacity=cap)
    check_against_oracle(p, quads, blob, offs, stats)
    raw = blob.cpu().numpy().tobytes()
    for in_place in (False, True):
        w_out, ea_out, eas_out = gpu_decompress(handle, blob, offs, dquads, in_place)
        for i, q in enumerate(quads):
            want = orc.decompress_tensor(raw[offs[i]:offs[i + 1]], q[1])
            for got, w in zip((w_out[i], ea_out[i], eas_out[i]), want):
                np.testing.assert_array_equal(got.cpu().numpy().view(np.uint32), w.view(np.uint32))


@pytest.mark.parametrize("bits", [2, 8])
def test_widths_with_outliers_ten_iterations_and_oracle_written_records(handle, bits):
    n = 150001
    rng = np.random.default_rng(77 + bits)
    w_t, w_prev, ea, eas = rand_quad_np(n, 3100 + bits)
    w_t = w_t.copy(); w_t[rng.integers(0, n, n // 100)] += np.float32(3e-3)      # 1 % large residuals
    q = (w_t, w_prev, ea, eas)
    p = binding.Params(median_source=1, bits=bits, kmeans_iters=10)
    cap = binding.record_bytes(n, n, n, bits)
    blob, offs, stats = gpu_compress(handle, p, to_dev([q]), capacity=cap)
    check_against_oracle(p, [q], blob, offs, stats)
    # a record the oracle wrote decodes on the GPU
    want_blob, _ = orc.compress_tensor(*q, orc.Params(median_source=1, bits=bits, kmeans_iters=2, seed=5))
    t = torch.frombuffer(bytearray(want_blob), dtype=torch.uint8).to(DEV)
    wp = torch.as_tensor(w_prev).to(DEV)
    outs = [torch.empty_like(wp) for _ in range(3)]
    handle.decompress_tensor(t, len(want_blob), wp, *outs)
    for got, want in zip(outs, orc.decompress_tensor(want_blob, w_prev)):
        np.testing.assert_array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_width_errors(handle):
    q = rand_quad_np(5000, 3200)
    dq = to_dev([q])[0]
    blob = torch.empty(binding.record_bytes(5000, 5000, 5000, 8), dtype=torch.uint8, device=DEV)
    for bits in (0, 1, 3, 5, 16, 32):
        with pytest.raises(binding.ExcpError) as e:
            handle.compress_tensor(binding.Params(bits=bits), *dq, blob)
        assert e.value.status == -1
    nbytes, _ = handle.compress_tensor(binding.Params(median_source=1, bits=8), *dq, blob)
    dense = torch.empty(binding.dense_bytes(5000, 8), dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.ExcpError) as e:                  # the dense layout is built for 4-bit records only
        handle.record_to_dense(blob, nbytes, 5000, dense)
    assert e.value.status == -2
    outs = [torch.empty_like(dq[1]) for _ in range(3)]
    bad = blob.clone(); bad[32] = 4                              # claims 4-bit codes: sizes no longer agree
    with pytest.raises(binding.ExcpError) as e:
        handle.decompress_tensor(bad, nbytes, dq[1], *outs)
    assert e.value.status == -5
