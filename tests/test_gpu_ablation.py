"""GPU parity for the ablation switches (ViT table caption: no M2W / no W2M; ablation table of
Section 4.4: residual / prune / quant off): records byte-identical to the oracle's, Algorithm 2
bit-identical, for every switch alone and for combinations."""
import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding
from test_gpu_parity import DEV, check_against_oracle, gpu_compress, gpu_decompress, rand_quad_np, to_dev

pytestmark = pytest.mark.gpu

W2M, M2W, RES, PRUNE, QUANT = (binding.FLAG_NO_W2M, binding.FLAG_NO_M2W, binding.FLAG_NO_RESIDUAL,
                               binding.FLAG_NO_PRUNE, binding.FLAG_NO_QUANT)


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(workspace_numel=700_000)
    h.set_report_sse(True)
    yield h
    h.close()


def same_bits(t, a):
    np.testing.assert_array_equal(t.cpu().numpy().view(np.uint32), a.view(np.uint32))


@pytest.mark.parametrize("flags", [W2M, M2W, RES, PRUNE, QUANT, W2M | M2W, RES | PRUNE, RES | QUANT, W2M | QUANT,
                                   PRUNE | QUANT, RES | PRUNE | QUANT, 31])
@pytest.mark.parametrize("mode", [binding.MEDIAN_ABS_WEIGHT, binding.MEDIAN_ABS_RESIDUAL])
def test_switches_match_the_oracle(handle, flags, mode):
    sizes = [0, 1, 33, 4097, 70001, 12288, 300000, 65536, 65537]        # two groups; ragged and empty tensors
    quads = [rand_quad_np(n, 2000 + 7 * flags + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    if flags & M2W:                                   # alpha is the threshold itself: on |W_t| or on |dW|
        alpha = 0.01 if flags & RES else 5e-5
    elif flags & RES:                                 # |W_t| * sqrt(eas) against alpha * median(|W_t|)
        alpha = 1e-4
    else:
        alpha = 5e-5 if mode == 1 else 2e-7
    p = binding.Params(alpha=alpha, median_source=mode, kmeans_iters=4, flags=flags)
    bits = 32 if flags & QUANT else 4
    cap = sum(binding.record_bytes(n, n, n, bits) for n in sizes)
    blob, offs, stats = gpu_compress(handle, p, dquads, capacity=cap)
    raw = blob.cpu().numpy().tobytes()
    if flags & QUANT:                                                    # no centres to compare: whole records
        for i, q in enumerate(quads):
            want, info = orc.compress_tensor(*q, orc.Params(alpha=alpha, median_source=mode, kmeans_iters=4, flags=flags),
                                             tensor_index=i)
            assert (stats[i].nnz_w, stats[i].nnz_o) == (info["nnz_w"], info["nnz_o"])
            assert stats[i].thr_w == info["thr_w"] and stats[i].thr_o == info["thr_o"]
            assert raw[offs[i]:offs[i + 1]] == want, f"tensor {i}"
    else:
        check_against_oracle(p, quads, blob, offs, stats)
    some = sum(s.nnz_w for s in stats)
    assert 0 < some and (flags & PRUNE or some < sum(sizes))            # the case prunes something but not everything
    for in_place in (False, True):
        w_out, ea_out, eas_out = gpu_decompress(handle, blob, offs, dquads, in_place)
        for i, q in enumerate(quads):
            w_hat, ea_hat, eas_hat = orc.decompress_tensor(raw[offs[i]:offs[i + 1]], q[1])
            same_bits(w_out[i], w_hat); same_bits(ea_out[i], ea_hat); same_bits(eas_out[i], eas_hat)


def test_without_residual_w_prev_is_not_read(handle):
    q = rand_quad_np(50000, 2500)
    w_t, w_prev, ea, eas = to_dev([q])[0]
    p = binding.Params(alpha=2e-7, flags=RES)
    blob = torch.empty(binding.compress_bound(50000), dtype=torch.uint8, device=DEV)
    lib, hd = handle.lib, handle._h
    import ctypes as C
    nbytes = C.c_size_t(0)
    cp = p.to_c()
    st = lib.excp_compress_tensor(hd, C.byref(cp), w_t.data_ptr(), None, ea.data_ptr(), eas.data_ptr(), 50000,
                                  blob.data_ptr(), blob.numel(), C.byref(nbytes), None,
                                  torch.cuda.current_stream().cuda_stream)
    assert st == 0
    want, _ = orc.compress_tensor(q[0], np.zeros_like(q[1]), q[2], q[3], orc.Params(alpha=2e-7, flags=orc.FLAG_NO_RESIDUAL))
    assert blob[:nbytes.value].cpu().numpy().tobytes() == want
    # with the residual on, a missing W^_(t-1) is an argument error
    cp0 = binding.Params().to_c()
    st = lib.excp_compress_tensor(hd, C.byref(cp0), w_t.data_ptr(), None, ea.data_ptr(), eas.data_ptr(), 50000,
                                  blob.data_ptr(), blob.numel(), C.byref(nbytes), None,
                                  torch.cuda.current_stream().cuda_stream)
    assert st == -1


def test_flag_errors_and_record_flags(handle):
    q = rand_quad_np(9000, 2600)
    dq = to_dev([q])[0]
    blob = torch.empty(binding.record_bytes(9000, 9000, 9000, 32), dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.ExcpError) as e:                          # an unknown switch
        handle.compress_tensor(binding.Params(flags=32), *dq, blob)
    assert e.value.status == -1
    nbytes, st = handle.compress_tensor(binding.Params(median_source=1, flags=W2M), *dq, blob)
    outs = [torch.empty_like(dq[1]) for _ in range(3)]
    handle.decompress_tensor(blob, nbytes, dq[1], *outs)
    bad = blob.clone(); bad[44] = 0                                      # claims to be the full method, holds orphan moments
    with pytest.raises(binding.ExcpError) as e:
        handle.decompress_tensor(bad, nbytes, dq[1], *outs)
    assert e.value.status == -5
    bad = blob.clone(); bad[44] = 9                                      # an unknown record flag
    with pytest.raises(binding.ExcpError) as e:
        handle.decompress_tensor(bad, nbytes, dq[1], *outs)
    assert e.value.status == -5
    dense = torch.empty(binding.dense_bytes(9000), dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.ExcpError) as e:                          # variants have no dense layout
        handle.record_to_dense(blob, nbytes, 9000, dense)
    assert e.value.status == -2
    nbytes, _ = handle.compress_tensor(binding.Params(median_source=1, flags=PRUNE), *dq, blob)
    assert handle.record_to_dense(blob, nbytes, 9000, dense) == binding.dense_bytes(9000)   # no record flag: fine


def test_host_buffer_path_with_switches(handle):
    sizes = [5000, 0, 70000, 4096, 130000]
    quads = [rand_quad_np(n, 2700 + i) for i, n in enumerate(sizes)]
    hq = [tuple(torch.as_tensor(a).pin_memory() for a in q) for q in quads]
    p = binding.Params(median_source=1, kmeans_iters=3, flags=W2M | PRUNE)
    hblob = torch.empty(sum(binding.compress_bound(n) for n in sizes), dtype=torch.uint8).pin_memory()
    offs, _ = handle.compress_checkpoint_host(p, hq, hblob)
    raw = hblob.numpy().tobytes()
    for i, q in enumerate(quads):
        want, _ = orc.compress_tensor(*q, orc.Params(median_source=1, kmeans_iters=3, flags=W2M | PRUNE), tensor_index=i)
        assert raw[offs[i]:offs[i + 1]] == want
    with pytest.raises(binding.ExcpError) as e:                          # raw records do not go through the staging
        handle.compress_checkpoint_host(binding.Params(flags=QUANT), hq, hblob)
    assert e.value.status == -2
