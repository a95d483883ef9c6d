"""GPU parity for the dense index layout (Sections 3.3 / 4.2: one code per element, 0 = pruned):
record -> dense container and Algorithm 2 on the container, against the oracle, byte for byte."""
import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding
from test_gpu_parity import DEV, gpu_compress, rand_quad_np, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    h = binding.Handle(workspace_numel=1_000_000)
    yield h
    h.close()


def to_dense(h, blob, offs, sizes):
    total = sum(binding.dense_bytes(n) for n in sizes)
    dense = torch.full((max(total, 16),), 0xCD, dtype=torch.uint8, device=DEV)      # dirty on purpose
    doffs = h.checkpoint_to_dense(blob, offs, sizes, dense)
    assert doffs[-1] == total
    return dense, doffs


def test_dense_bytes_matches_the_layout():
    for n in (0, 1, 2, 31, 32, 33, 4096, 100001):
        assert binding.dense_bytes(n) == orc.dense_bytes(n, 4) == 256 + 3 * 16 * ((n + 31) // 32)
    assert binding.dense_bytes(10, 3) == 0


def test_hand_example_dense_bytes(handle):
    g = {}
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "hand_example.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split(":", 1)
                g[k.strip()] = [int(x, 16) if x.startswith("0x") else float(x) for x in v.split()]
    q = tuple(np.array(g[k], dtype=np.float32) for k in ("w_t", "w_prev", "ea", "eas"))
    p = binding.Params(alpha=g["alpha"][0], beta=g["beta"][0])
    blob, offs, _ = gpu_compress(handle, p, to_dev([q]))
    dense, doffs = to_dense(handle, blob, offs, [8])
    raw = dense.cpu().numpy().tobytes()
    for j, key in enumerate(("w", "ea", "eas")):
        sec = raw[256 + 16 * j:256 + 16 * (j + 1)]
        assert list(sec[:4]) == [int(v) for v in g[f"dense_bytes_{key}_abs_weight"]]
        assert sec[4:] == b"\0" * 12


def test_record_to_dense_and_dense_decode_match_the_oracle(handle):
    # several groups (workspace 1 M elements), empty and ragged tensors, tile-aligned ones
    sizes = [0, 1, 7, 8, 9, 33, 4095, 4096, 4097, 70001, 12288, 300000, 600000, 65536]
    quads = [rand_quad_np(n, 1600 + i) for i, n in enumerate(sizes)]
    dquads = to_dev(quads)
    p = binding.Params(median_source=binding.MEDIAN_ABS_RESIDUAL)
    blob, offs, stats = gpu_compress(handle, p, dquads)
    raw = blob.cpu().numpy().tobytes()
    dense, doffs = to_dense(handle, blob, offs, sizes)
    draw = dense.cpu().numpy().tobytes()
    for i, n in enumerate(sizes):
        want = orc.record_to_dense(raw[offs[i]:offs[i + 1]])
        assert draw[doffs[i]:doffs[i + 1]] == want, f"tensor {i} (numel {n})"
    for in_place in (False, True):
        w_prev = [q[1].clone() for q in dquads]
        w_out = w_prev if in_place else [torch.full_like(t, 7.0) for t in w_prev]
        ea_out = [torch.full_like(t, 7.0) for t in w_prev]
        eas_out = [torch.full_like(t, 7.0) for t in w_prev]
        handle.decompress_checkpoint(dense, doffs, w_prev, w_out, ea_out, eas_out, dense=True)
        for i, q in enumerate(quads):
            want = orc.decompress_dense(draw[doffs[i]:doffs[i + 1]], q[1])
            also = orc.decompress_tensor(raw[offs[i]:offs[i + 1]], q[1])
            for got, a, b in zip((w_out[i], ea_out[i], eas_out[i]), want, also):
                np.testing.assert_array_equal(got.cpu().numpy().view(np.uint32), a.view(np.uint32))
                np.testing.assert_array_equal(a.view(np.uint32), b.view(np.uint32))


def test_gpu_decodes_a_dense_container_written_by_the_oracle(handle):
    q = rand_quad_np(33331, 1700)
    rec, _ = orc.compress_tensor(*q, orc.Params(median_source=1, seed=9))
    want_dense = orc.record_to_dense(rec)
    dense = torch.frombuffer(bytearray(want_dense), dtype=torch.uint8).to(DEV)
    w_prev = torch.as_tensor(q[1]).to(DEV)
    outs = [torch.empty_like(w_prev) for _ in range(3)]
    handle.decompress_dense_tensor(dense, len(want_dense), w_prev, *outs)
    for got, want in zip(outs, orc.decompress_dense(want_dense, q[1])):
        np.testing.assert_array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))
    # and the single-record conversion
    rec_t = torch.frombuffer(bytearray(rec), dtype=torch.uint8).to(DEV)
    out = torch.empty(len(want_dense), dtype=torch.uint8, device=DEV)
    assert handle.record_to_dense(rec_t, len(rec), 33331, out) == len(want_dense)
    assert out.cpu().numpy().tobytes() == want_dense


def test_dense_errors(handle):
    n = 9001
    q = rand_quad_np(n, 1800)
    rec, info = orc.compress_tensor(*q, orc.Params(median_source=1))
    good = bytearray(orc.record_to_dense(rec))
    w_prev = torch.as_tensor(q[1]).to(DEV)
    outs = [torch.empty_like(w_prev) for _ in range(3)]
    hb, sb = 256, orc.dense_section_bytes(n, 4)
    pruned = int(np.flatnonzero(~info["m_w"])[0])
    half = int(np.flatnonzero(info["m_w"] & ~info["m_o"])[0])

    def decode(buf, nbytes=None):
        t = torch.frombuffer(bytearray(buf), dtype=torch.uint8).to(DEV)
        handle.decompress_dense_tensor(t, len(buf) if nbytes is None else nbytes, w_prev, *outs)

    decode(good)
    cases = []
    for pos, flip in ((0, 1), (4, 3), (8, 1), (16, 0x80), (24, 0x80), (32, 12), (48, 0x10)):   # header fields
        b = bytearray(good); b[pos] ^= flip; cases.append(b)
    b = bytearray(good); b[hb + pruned // 2] |= 1 << (4 * (pruned % 2)); cases.append(b)       # one code too many
    b = bytearray(good); b[hb + sb + half // 2] |= 1 << (4 * (half % 2)); cases.append(b)      # moments disagree
    b = bytearray(good); b[hb + n // 2] |= 0x10; cases.append(b)                          # a code past the end
    for i, b in enumerate(cases):
        with pytest.raises(binding.ExcpError) as e:
            decode(b)
        assert e.value.status == -5, i
    with pytest.raises(binding.ExcpError) as e:                                                 # truncated
        decode(good, len(good) - 16)
    assert e.value.status == -5
    # conversion: too little room is refused before anything runs; a corrupt record is refused
    rec_t = torch.frombuffer(bytearray(rec), dtype=torch.uint8).to(DEV)
    small = torch.empty(len(good) - 16, dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.ExcpError) as e:
        handle.record_to_dense(rec_t, len(rec), n, small)
    assert e.value.status == -3
    bad = rec_t.clone(); bad[16] ^= 0x80
    with pytest.raises(binding.ExcpError) as e:
        handle.record_to_dense(bad, len(rec), n, torch.empty(len(good), dtype=torch.uint8, device=DEV))
    assert e.value.status == -5
    decode(good)                                                                                # the handle still works
