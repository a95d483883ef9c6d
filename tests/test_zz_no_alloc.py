"""The allocation-free decode entry point (excp_decompress_tensor_noalloc).

Some callers restore checkpoints where they cannot ask the driver for memory: the training
framework's allocator already holds the whole device, or the device-wide synchronisation of
cudaMalloc is not acceptable while other streams run.  For them the library decodes with a
fixed scratch array of its own instead of a handle's workspace.  The test calls it through the
C ABI twice in a row (the array is shared and keeps the previous call's contents) and requires
the very bytes that the handle-based entry point produces.  This file sorts last on purpose."""
import numpy as np
import pytest
import torch

from paper_2406_11257_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _compress(h, n, seed):
    q = synth.make_quad(n, seed, 0, device=DEV)
    blob = torch.empty(binding.compress_bound(n), dtype=torch.uint8, device=DEV)
    nbytes, stats = h.compress_tensor(binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL, seed=seed), *q, blob)
    return q, blob, nbytes, stats


def test_noalloc_decode_matches_the_handle_path_twice_in_a_row():
    torch.cuda.set_device(0)
    h = binding.Handle(workspace_numel=400_000)
    try:
        cases = [_compress(h, 300_001, 1), _compress(h, 4097, 2)]      # a larger then a smaller tensor
        for q, blob, nbytes, stats in cases:
            assert stats.nnz_w > 0
            want = [torch.empty_like(q[1]) for _ in range(3)]
            h.decompress_tensor(blob, nbytes, q[1], *want)
            for call in range(2):
                got = [torch.full_like(q[1], 7.0) for _ in range(3)]
                binding.decompress_tensor_noalloc(blob, nbytes, q[1], *got)
                for g, w in zip(got, want):
                    np.testing.assert_array_equal(g.cpu().numpy().view(np.uint32), w.cpu().numpy().view(np.uint32))
        # in place, like the handle path allows
        q, blob, nbytes, _ = cases[0]
        w = q[1].clone()
        ea, eas = torch.empty_like(w), torch.empty_like(w)
        binding.decompress_tensor_noalloc(blob, nbytes, w, w, ea, eas)
        ref = [torch.empty_like(w) for _ in range(3)]
        h.decompress_tensor(blob, nbytes, q[1], *ref)
        assert torch.equal(w, ref[0]) and torch.equal(ea, ref[1])
    finally:
        h.close()


def test_noalloc_refuses_what_it_cannot_hold_and_reports_corruption():
    torch.cuda.set_device(0)
    h = binding.Handle(workspace_numel=100_000)
    try:
        q, blob, nbytes, _ = _compress(h, 20_000, 3)
    finally:
        h.close()
    outs = [torch.empty_like(q[1]) for _ in range(3)]
    big = torch.empty(binding.NOALLOC_MAX_NUMEL + 4, device=DEV)
    with pytest.raises(binding.ExcpError) as e:                       # beyond the fixed scratch
        binding.decompress_tensor_noalloc(blob, nbytes, big, big, big, big)
    assert e.value.status == -1
    bad = blob.clone()
    bad[0] = 0
    with pytest.raises(binding.ExcpError) as e:
        binding.decompress_tensor_noalloc(bad, nbytes, q[1], *outs)
    assert e.value.status == -5
    binding.decompress_tensor_noalloc(blob, nbytes, q[1], *outs)      # and it still works afterwards
