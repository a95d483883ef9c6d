"""Randomly drawn parity cases: shapes, value distributions, hyper-parameters, code widths and ablation
switches from a seeded generator, whole records and the decoded tensors against the oracle.

The distributions are chosen to reach what the workload-shaped inputs do not: values over a huge range of
exponents, a handful of distinct values (ties everywhere), coarse grids, mostly-zero streams with zeros of
either sign, subnormals, two far-apart clumps, second moments that are exactly zero, sizes around the tile
and block boundaries, several tensors per call in workspaces that split them into groups differently.
Inputs that overflow to infinity must be refused by both sides."""
import numpy as np
import pytest
import torch

from oracle import excp_oracle as orc
from paper_2406_11257_b200 import binding

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
N_MAX = 400_000
CASES = 240


def draw(rng, n, kind, scale):
    if kind == 0:
        x = rng.standard_normal(n) * scale
    elif kind == 1:
        x = rng.standard_t(3, n) * scale
    elif kind == 2:                                                 # a huge range of exponents
        x = np.exp(rng.standard_normal(n) * rng.uniform(1, 12)) * scale * rng.choice([-1, 1], n)
    elif kind == 3:                                                 # few distinct values
        vals = rng.standard_normal(rng.integers(1, 9)) * scale
        x = vals[rng.integers(0, len(vals), n)]
    elif kind == 4:                                                 # a coarse grid
        q = scale * 2.0 ** -rng.integers(1, 6)
        x = np.rint(rng.standard_normal(n) * scale / q) * q
    elif kind == 5:                                                 # mostly zero, zeros of either sign
        x = rng.standard_normal(n) * scale * (rng.random(n) < rng.uniform(0.001, 0.2))
    elif kind == 6:                                                 # subnormals among normals
        x = rng.standard_normal(n) * np.where(rng.random(n) < 0.5, 1e-41, scale)
    else:                                                           # two clumps far apart
        x = np.where(rng.random(n) < 0.3, rng.standard_normal(n) * scale * 1e-3 + scale * 50, rng.standard_normal(n) * scale)
    with np.errstate(all="ignore"):
        return x.astype(np.float32)


def draw_case(seed, extreme=False):
    """extreme: scales from 1e-42 to 1e36 and thresholds from 1e-44 to 1e37, so that products and thresholds
    underflow, overflow to infinity or sit among the subnormals, and some sums W_(t-1) + dW are not finite."""
    rng = np.random.default_rng(seed)
    quads = []
    for _ in range(int(rng.integers(1, 5))):
        r = rng.random()
        if r < 0.15:
            n = int(rng.integers(0, 200))
        elif r < 0.4:
            n = int(rng.choice([1024, 4096, 8192, 65536, 131072]) + rng.integers(-3, 4))
        else:
            n = int(np.exp(rng.uniform(np.log(200), np.log(N_MAX))))
        if extreme:
            sc = [float(10 ** rng.uniform(-3, 25)), float(10 ** rng.uniform(-40, 30)), float(10 ** rng.uniform(-42, 36)), float(10 ** rng.uniform(-22, 18))]
        else:
            sc = [0.02, float(10 ** rng.uniform(-6, -2)), float(10 ** rng.uniform(-7, -2)), float(10 ** rng.uniform(-6, -2))]
        with np.errstate(all="ignore"):
            w_prev = draw(rng, n, int(rng.integers(0, 2)), sc[0])
            dw = draw(rng, n, int(rng.integers(0, 8)), sc[1])
            w_t = (w_prev + dw).astype(np.float32)
            ea = draw(rng, n, int(rng.integers(0, 8)), sc[2])
            eas = np.square(draw(rng, n, int(rng.integers(0, 8)), sc[3])).astype(np.float32)
            if rng.random() < 0.7:
                eas = (eas + np.float32(1e-12)).astype(np.float32)
        quads.append((w_t, w_prev, ea, eas))
    p = dict(alpha=float(10 ** (rng.uniform(-44, 37) if extreme else rng.uniform(-7, -3))) if rng.random() < 0.8 else 0.0,
             beta=float(10 ** rng.uniform(-44, 37)) if extreme and rng.random() < 0.5 else float(rng.uniform(0, 4)),
             bits=int(rng.choice([2, 4, 4, 4, 8])), kmeans_iters=int(rng.integers(0, 13)), seed=int(rng.integers(0, 1 << 31)),
             median_source=int(rng.integers(0, 2)), flags=int(rng.integers(0, 32)) if rng.random() < 0.3 else 0)
    if p["median_source"] == 0 and rng.random() < 0.7:
        p["alpha"] *= 1e-2                                          # the median of |W_t| is large
    workspace = max(int(rng.choice([500_000, 1_000_000, 6_000_000])), max(q[0].size for q in quads) + 4096)
    return p, quads, workspace


@pytest.mark.parametrize("extreme", [False, True])
def test_randomly_drawn_cases_against_the_oracle(extreme):
    handles = {}
    refused = 0
    try:
        for seed in range(CASES // 2 if extreme else CASES):
            p, quads, workspace = draw_case(seed + (1000 if extreme else 0), extreme)
            if workspace not in handles:
                handles[workspace] = binding.Handle(workspace_numel=workspace)
            h = handles[workspace]
            dq = [tuple(torch.as_tensor(a).to(DEV) for a in q) for q in quads]
            width = 32 if p["flags"] & binding.FLAG_NO_QUANT else p["bits"]
            blob = torch.full((max(16, sum(binding.compress_bound(q[0].size, width) for q in quads)),), 0xAB, dtype=torch.uint8, device=DEV)
            try:
                with np.errstate(all="ignore"):
                    want = [orc.compress_tensor(*q, orc.Params(**p), tensor_index=i) for i, q in enumerate(quads)]
            except orc.InvalidInput:
                with pytest.raises(binding.ExcpError, match="NONFINITE"):
                    h.compress_checkpoint(binding.Params(**p), dq, blob)
                refused += 1
                continue
            offs, stats = h.compress_checkpoint(binding.Params(**p), dq, blob)
            raw = blob.cpu().numpy().tobytes()
            w_out = [q[1].clone() for q in dq]
            ea_out = [torch.full_like(q[1], 7.0) for q in dq]
            eas_out = [torch.full_like(q[1], 7.0) for q in dq]
            h.decompress_checkpoint(blob, offs, w_out, w_out, ea_out, eas_out)      # Algorithm 2 in place
            for i, (rec, info) in enumerate(want):
                tag = f"seed {seed}{' (extreme)' if extreme else ''}, tensor {i} of {quads[i][0].size} elements, {p}"
                assert (stats[i].nnz_w, stats[i].nnz_o) == (info["nnz_w"], info["nnz_o"]), tag
                assert raw[offs[i]:offs[i + 1]] == rec, tag
                for got, exp in zip((w_out[i], ea_out[i], eas_out[i]), orc.decompress_tensor(rec, quads[i][1])):
                    assert np.array_equal(got.cpu().numpy().view(np.uint32), np.ascontiguousarray(exp).view(np.uint32)), tag
        assert (0 < refused < CASES // 4) if extreme else refused < CASES // 10   # sums that overflow: common only at the extreme scales
    finally:
        for h in handles.values():
            h.close()


def test_kept_zeros_of_either_sign():
    """With pruning off the first-moment stream keeps its zeros; -0 and +0 then both become centres and
    their order (-0 first) is part of the record."""
    rng = np.random.default_rng(12)
    n = 70_001
    w_prev = (rng.standard_normal(n) * 0.02).astype(np.float32)
    w_t = (w_prev + rng.standard_normal(n).astype(np.float32) * np.float32(1e-4)).astype(np.float32)
    ea = (rng.standard_normal(n) * 1e-4 * (rng.random(n) < 0.1)).astype(np.float32)       # 90 % zeros, half of them -0
    eas = np.square(rng.standard_normal(n) * 1e-4).astype(np.float32)
    assert np.signbit(ea[ea == 0]).any() and not np.signbit(ea[ea == 0]).all()
    h = binding.Handle(workspace_numel=n)
    try:
        dq = tuple(torch.as_tensor(a).to(DEV) for a in (w_t, w_prev, ea, eas))
        reached = 0
        for bits in (2, 4, 8):
            for iters in (0, 6):
                p = dict(bits=bits, kmeans_iters=iters, median_source=1, seed=5, flags=binding.FLAG_NO_PRUNE)
                blob = torch.empty(binding.compress_bound(n, bits), dtype=torch.uint8, device=DEV)
                nbytes, st = h.compress_tensor(binding.Params(**p), *dq, blob)
                rec, info = orc.compress_tensor(w_t, w_prev, ea, eas, orc.Params(**p))
                zeros = info["c_ea"][info["c_ea"] == 0]
                reached += bool(np.signbit(zeros).any() and not np.signbit(zeros).all())
                assert blob[:nbytes].cpu().numpy().tobytes() == rec, (bits, iters)
        assert reached >= 4                                         # centres -0 and +0 side by side: every start, 8 bits after iterations too
    finally:
        h.close()
