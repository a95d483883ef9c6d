"""Pins for the CPU oracle: each oracle function is checked against something
that is not the oracle -- a hand-computed example (tests/golden), exact rational
arithmetic, brute force on tiny inputs, closed forms and invariants."""
import math
import os
import statistics
import struct
from fractions import Fraction

import numpy as np
import pytest

from oracle import excp_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_example.txt")


def load_golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":", 1)
            out[key.strip()] = [int(v, 16) if v.startswith("0x") else float(v) for v in vals.split()]
    return out


G = load_golden()
f32 = lambda k: np.array(G[k], dtype=np.float32)


# ---------------------------------------------------------------- hand example
def test_hand_residual_and_statistics():
    dw = orc.residual(f32("w_t"), f32("w_prev"))
    assert dw.dtype == np.float32
    np.testing.assert_array_equal(dw, f32("dw"))
    assert orc.lower_median_abs(f32("w_t")) == G["median_abs_weight"][0]
    assert orc.lower_median_abs(dw) == G["median_abs_residual"][0]
    assert orc.exact_mean_abs(f32("ea")) == G["mean_abs_ea"][0]


@pytest.mark.parametrize("mode,tag", [(orc.MEDIAN_ABS_WEIGHT, "abs_weight"),
                                      (orc.MEDIAN_ABS_RESIDUAL, "abs_residual")])
def test_hand_masks_and_bitmaps(mode, tag):
    p = orc.Params(alpha=G["alpha"][0], beta=G["beta"][0], bits=4, median_source=mode)
    blob, info = orc.compress_tensor(f32("w_t"), f32("w_prev"), f32("ea"), f32("eas"), p)
    np.testing.assert_array_equal(info["m_w"].astype(int), np.array(G["m_w_" + tag], dtype=int))
    np.testing.assert_array_equal(info["m_o"].astype(int), np.array(G["m_o_" + tag], dtype=int))
    assert info["thr_o"] == G["thr_o"][0]
    hb = orc.header_bytes(15)
    assert blob[hb] == G["bitmap_w_" + tag][0]
    assert blob[hb + 16] == G["bitmap_o_" + tag][0]
    assert blob[hb + 1:hb + 16] == b"\0" * 15


def test_hand_lossless_decode_when_fewer_survivors_than_centres():
    p = orc.Params(alpha=G["alpha"][0], beta=G["beta"][0], bits=4)
    blob, _ = orc.compress_tensor(f32("w_t"), f32("w_prev"), f32("ea"), f32("eas"), p)
    w_hat, ea_hat, eas_hat = orc.decompress_tensor(blob, f32("w_prev"))
    np.testing.assert_array_equal(w_hat, f32("w_hat_abs_weight"))
    np.testing.assert_array_equal(ea_hat, f32("ea_hat_abs_weight"))
    np.testing.assert_array_equal(eas_hat, f32("eas_hat_abs_weight"))


def test_hand_two_bit_kmeans_reaches_the_optimal_partition():
    p = orc.Params(alpha=G["alpha"][0], beta=G["beta"][0], bits=2)
    _, info = orc.compress_tensor(f32("w_t"), f32("w_prev"), f32("ea"), f32("eas"), p)
    np.testing.assert_array_equal(info["c_w"], f32("centres_2bit"))
    np.testing.assert_array_equal(info["codes_w"], np.array(G["codes_2bit"], dtype=np.uint8))
    s = info["s_w"].astype(np.float64)
    sse = float(np.sum((s - info["c_w"].astype(np.float64)[info["codes_w"] - 1]) ** 2))
    assert sse == G["sse_2bit"][0]
    assert info["sse_w"] == G["sse_2bit"][0]                  # the reported objective is that sum
    assert orc.optimal_kmeans_1d_sse(info["s_w"], 3) == Fraction(G["sse_2bit"][0])


# ---------------------------------------------------------------- median
@pytest.mark.parametrize("n", [1, 2, 3, 4, 7, 8, 33, 1000, 1001])
def test_lower_median_against_full_sort(n):
    rng = np.random.default_rng(n)
    x = rng.standard_normal(n).astype(np.float32)
    x[rng.integers(0, n, size=n // 3)] = x[0]          # repeated values
    want = sorted(abs(float(v)) for v in x)[(n - 1) // 2]
    assert float(orc.lower_median_abs(x)) == want
    assert float(orc.lower_median_abs(x)) == statistics.median_low([abs(float(v)) for v in x])


def test_lower_median_empty_and_even_is_not_mid_average():
    assert orc.lower_median_abs(np.zeros(0, np.float32)) == 0.0
    assert orc.lower_median_abs(np.array([1, -2, 3, -4], np.float32)) == 2.0


# ---------------------------------------------------------------- exact mean
def _nearest_f32_property(value: np.float32, q: Fraction):
    v = Fraction(float(value))
    up = Fraction(float(np.nextafter(value, np.float32(np.inf))))
    dn = Fraction(float(np.nextafter(value, np.float32(-np.inf))))
    assert abs(v - q) <= abs(up - q) and abs(v - q) <= abs(dn - q)
    if abs(v - q) == abs(up - q) or abs(v - q) == abs(dn - q):   # a tie: even mantissa wins
        assert (np.float32(value).view(np.uint32) & 1) == 0


def test_round_ratio_fixed_cases():
    r = orc.round_ratio_to_f32
    assert r(0, 5) == 0.0
    assert r(1, 3) == np.float32(1.0 / 3.0)
    assert r((1 << 24) + 1, 1) == float(1 << 24)            # tie -> even
    assert r((1 << 24) + 3, 1) == float((1 << 24) + 4)      # tie -> even, upwards
    assert r((1 << 25) + 2, 2) == float(1 << 24)
    assert r(1, 1 << 149) == np.float32(2.0 ** -149)        # smallest subnormal
    assert r(1, 1 << 150) == 0.0                            # half of it: tie -> 0
    assert r(3, 1 << 150) == np.float32(2.0 ** -148)        # 1.5 -> 2 (even)
    assert r(5, 1 << 151) == np.float32(2.0 ** -149)        # 0.625 -> 1
    assert float(r((1 << 25) - 1, 1 << 151)) == 2.0 ** -126  # largest subnormal + half: up into the normals


def test_round_ratio_is_nearest_on_random_rationals():
    rng = np.random.default_rng(7)
    for _ in range(300):
        num = int(rng.integers(1, 1 << 62)) << int(rng.integers(0, 80))
        den = int(rng.integers(1, 1 << 40)) << int(rng.integers(0, 200))
        _nearest_f32_property(orc.round_ratio_to_f32(num, den), Fraction(num, den))


@pytest.mark.parametrize("n,scale", [(1, 1.0), (5, 1e-4), (257, 1e-4), (1000, 3e10), (999, 1e-38)])
def test_exact_mean_abs_against_rationals(n, scale):
    rng = np.random.default_rng(n)
    x = (rng.standard_normal(n) * scale).astype(np.float32)
    x[::7] *= np.float32(1e-6)                              # wide exponent spread
    q = orc.brute_mean_abs(x)
    assert Fraction(orc.exact_sum_abs_units(x), 1 << 149) == q * n
    _nearest_f32_property(orc.exact_mean_abs(x), q)


def test_exact_mean_abs_closed_forms():
    assert orc.exact_mean_abs(np.full(1000, -0.1, np.float32)) == np.float32(0.1)
    # the mean of 1..n is (n+1)/2
    assert orc.exact_mean_abs(-np.arange(1, 4097, dtype=np.float32)) == 2048.5
    # one huge and many tiny terms: a running fp32 sum would lose every tiny one
    x = np.full(1 << 20, 2.0 ** -30, np.float32)
    x[0] = 1.0
    assert float(orc.exact_mean_abs(x)) == float(np.float32((1.0 + ((1 << 20) - 1) * 2.0 ** -30) / (1 << 20)))
    # agrees with the correctly rounded fp64 sum where no second rounding can matter
    y = (np.random.default_rng(3).standard_normal(4096) * 1e-4).astype(np.float32)
    assert orc.exact_mean_abs(y) == np.float32(math.fsum(abs(float(v)) for v in y) / 4096)


# ---------------------------------------------------------------- masks
def _rand_quad(n, seed):
    rng = np.random.default_rng(seed)
    w_prev = (rng.standard_normal(n) * 0.02).astype(np.float32)
    dw = (rng.standard_t(3, n) * 1e-4 / math.sqrt(3)).astype(np.float32)
    w_t = (w_prev + dw).astype(np.float32)
    ea = (rng.standard_normal(n) * 1e-4).astype(np.float32)
    eas = ((np.abs(rng.standard_normal(n)) * 1e-4) ** 2 + 1e-12).astype(np.float32)
    return w_t, w_prev, ea, eas


def test_mask_special_cases():
    w_t, w_prev, ea, eas = _rand_quad(5000, 1)
    eas[::11] = 0.0
    w_t[::13] = w_prev[::13]
    ea[::17] = 0.0
    dw = orc.residual(w_t, w_prev)
    # alpha = 0: every non-zero residual with a positive second moment survives
    m_w, thr = orc.weight_mask(dw, eas, 0.0, np.float32(0.3))
    assert thr == 0.0
    np.testing.assert_array_equal(m_w, (dw != 0) & (eas > 0))
    # beta = 0: M_o = M_w and ea != 0
    m_o, _ = orc.moment_mask(ea, m_w, 0.0, np.float32(1.0))
    np.testing.assert_array_equal(m_o, m_w & (ea != 0))
    # a huge alpha prunes everything
    m_w2, _ = orc.weight_mask(dw, eas, 1e30, np.float32(1.0))
    assert not m_w2.any()


def test_mask_matches_division_form_of_eq_rw_away_from_the_threshold():
    """Eq. (rw) as printed: keep where |dW| > alpha / sqrt(m_t) * median.  The
    product form used by the oracle must agree wherever the two sides are not
    within rounding of each other."""
    w_t, w_prev, ea, eas = _rand_quad(20000, 2)
    dw = orc.residual(w_t, w_prev)
    med = orc.lower_median_abs(dw)
    alpha = 5e-5
    m_w, _ = orc.weight_mask(dw, eas, alpha, med)
    r_w = alpha / np.sqrt(eas.astype(np.float64)) * float(med)
    a = np.abs(dw.astype(np.float64))
    clear = np.abs(a - r_w) > 1e-5 * r_w
    np.testing.assert_array_equal(m_w[clear], (a > r_w)[clear])
    assert 0.3 < m_w.mean() < 0.7            # the residual-median mode keeps about half


def test_joint_rule_and_invariants_on_random_tensor():
    w_t, w_prev, ea, eas = _rand_quad(30000, 3)
    p = orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL)
    blob, info = orc.compress_tensor(w_t, w_prev, ea, eas, p)
    m_w, m_o = info["m_w"], info["m_o"]
    assert not (m_o & ~m_w).any()                                       # M_o inside M_w
    assert ((np.abs(ea) > info["thr_o"]) & ~m_w).any()                  # the joint rule drops some
    lhs = np.abs(info["dw"]) * np.sqrt(eas)
    assert (lhs[~m_w] <= info["thr_w"]).all() and (lhs[m_w] > info["thr_w"]).all()
    rec = orc.parse_record(blob)
    assert rec["nnz_w"] == m_w.sum() == rec["codes_w"].size
    assert rec["nnz_o"] == m_o.sum() == rec["codes_ea"].size == rec["codes_eas"].size
    for c in ("codes_w", "codes_ea", "codes_eas"):
        assert rec[c].min() >= 1 and rec[c].max() <= 15
    w_hat, ea_hat, eas_hat = orc.decompress_tensor(blob, w_prev)
    np.testing.assert_array_equal(w_hat[~m_w].view(np.uint32), w_prev[~m_w].view(np.uint32))
    assert (ea_hat[~m_o] == 0).all() and (eas_hat[~m_o] == 0).all()
    assert (ea_hat[m_o] != 0).all() and (eas_hat[m_o] > 0).all()
    # centres sorted and inside the range of what they quantise
    for c, s in (("c_w", "s_w"), ("c_ea", "s_ea"), ("c_eas", "s_eas")):
        assert (np.diff(info[c]) >= 0).all()
        assert info[c].min() >= info[s].min() and info[c].max() <= info[s].max()
    # quantisation error is bounded by the widest cell
    err = np.abs((w_hat - w_t)[m_w])
    assert err.max() <= np.abs(info["s_w"]).max()


def test_recompressing_a_reconstruction_against_itself_prunes_everything():
    w_t, w_prev, ea, eas = _rand_quad(4000, 4)
    blob, info = orc.compress_tensor(w_t, w_t, ea, eas, orc.Params())
    assert info["nnz_w"] == 0 and info["nnz_o"] == 0
    w_hat, ea_hat, eas_hat = orc.decompress_tensor(blob, w_t)
    np.testing.assert_array_equal(w_hat, w_t)
    assert not ea_hat.any() and not eas_hat.any()
    assert len(blob) == orc.header_bytes(15) + 2 * orc.bitmap_bytes(4000)


def test_invalid_inputs_are_refused():
    w_t, w_prev, ea, eas = _rand_quad(64, 5)
    for arr in (w_t, w_prev, ea, eas):
        bad = arr.copy(); bad[3] = np.nan
        args = [bad if a is arr else a for a in (w_t, w_prev, ea, eas)]
        with pytest.raises(orc.InvalidInput):
            orc.compress_tensor(*args, orc.Params())
    neg = eas.copy(); neg[0] = -1e-9
    with pytest.raises(orc.InvalidInput):
        orc.compress_tensor(w_t, w_prev, ea, neg, orc.Params())


# ---------------------------------------------------------------- k-means
def test_mix64_is_splitmix64():
    # first outputs of SplitMix64 seeded with 0 (state advances by the golden gamma)
    gamma = 0x9E3779B97F4A7C15
    got = [orc.mix64((i * gamma) & ((1 << 64) - 1)) for i in range(3)]
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_assign_is_exact_nearest_with_midpoints_down():
    rng = np.random.default_rng(11)
    for trial in range(20):
        c = np.sort((rng.standard_normal(15) * 1e-4).astype(np.float32))
        if trial % 3 == 0:
            c[5] = c[4]; c[6] = c[4]                       # repeated centres
        x = (rng.standard_t(3, 300) * 1e-4).astype(np.float32)
        x[:14] = ((c[:-1].astype(np.float64) + c[1:]) / 2).astype(np.float32)   # near / on mid-points
        x[14:29] = c                                                      # on the centres
        got = orc.assign(x, c)
        want = np.array([orc.brute_nearest(v, c) for v in x])
        if trial % 3:
            np.testing.assert_array_equal(got, want)
        else:
            # coincident centres: still a nearest one (same value), and the points
            # split -- at or below go to the first copy, above to the last
            np.testing.assert_array_equal(c[got], c[want])
            near = c[want] == c[4]
            np.testing.assert_array_equal(got[near], np.where(x[near] <= c[4], 4, 6))
    # a point on a mid-point goes to the lower centre
    assert orc.assign(np.array([0.5], np.float32), np.array([0.0, 1.0], np.float32))[0] == 0
    assert orc.assign(np.array([np.nextafter(np.float32(0.5), np.float32(1))]), np.array([0.0, 1.0], np.float32))[0] == 1


def test_rsum_mean_is_close_to_exact_and_exact_on_dyadics():
    rng = np.random.default_rng(12)
    s = (rng.standard_t(3, 5000) * 1e-4).astype(np.float32)
    e = orc.rsum_exponent(s)
    assert 2.0 ** e <= np.abs(s).max() < 2.0 ** (e + 1)
    q = orc.rsum_quantize(s, e)
    assert np.abs(q).max() < (1 << 31)
    got = float(orc.rsum_mean(int(q.sum()), s.size, e))
    exact = float(sum(Fraction(float(v)) for v in s) / s.size)
    assert abs(got - exact) <= float(np.abs(s).max()) * 2.0 ** -31 + abs(exact) * 2.0 ** -23
    d = np.array([0.5, -0.25, 0.125, 1.0, -0.5], np.float32)
    ed = orc.rsum_exponent(d)
    assert ed == 0
    assert orc.rsum_mean(int(orc.rsum_quantize(d, ed).sum()), 5, ed) == np.float32(0.175)
    assert orc.rsum_exponent(np.zeros(3, np.float32)) == 0
    assert orc.rsum_exponent(np.array([1e-45], np.float32)) == -126
    # ties in rint go to even
    assert list(orc.rsum_quantize(np.array([2.0 ** -31, 3 * 2.0 ** -31, 1.0], np.float32), 0)) == [0, 2, 1 << 30]


def _sse(s, c, idx):
    return float(np.sum((s.astype(np.float64) - c.astype(np.float64)[idx]) ** 2))


def test_lloyd_never_beats_and_often_meets_the_optimum_on_tiny_inputs():
    rng = np.random.default_rng(13)
    met = 0
    for trial in range(30):
        n = int(rng.integers(4, 12))
        s = (rng.standard_normal(n)).astype(np.float32)
        c0 = orc.kmeans_start(s, 3, seed=trial, tensor_index=0, stream=0)
        c, idx = orc.lloyd(s, c0, 10)
        best = float(orc.optimal_kmeans_1d_sse(s, 3))
        got = _sse(s, c, idx)
        assert got >= best - 1e-9
        met += abs(got - best) < 1e-9
    assert met >= 10


def test_lloyd_finds_well_separated_clusters_exactly():
    rng = np.random.default_rng(14)
    centres = np.array([-4.0, -1.0, 2.0], np.float32)
    s = np.concatenate([c + (rng.integers(-8, 9, 40) / 64.0) for c in centres]).astype(np.float32)
    rng.shuffle(s)
    c0 = orc.kmeans_start(s, 3, seed=1, tensor_index=0, stream=0)
    c, idx = orc.lloyd(s, c0, 10)
    assert abs(_sse(s, c, idx) - float(orc.optimal_kmeans_1d_sse(s, 3))) < 1e-9
    for j in range(3):
        assert abs(float(c[j]) - float(s[idx == j].astype(np.float64).mean())) < 1e-6


def test_lloyd_sse_does_not_increase_and_centres_stay_sorted():
    rng = np.random.default_rng(15)
    s = (rng.standard_t(3, 20000) * 1e-4).astype(np.float32)
    c = orc.kmeans_start(s, 15, seed=5, tensor_index=2, stream=0)
    assert (np.diff(c) >= 0).all()
    prev = None
    for it in range(6):
        _, idx = orc.lloyd(s, c, 0)                # assignment under the current centres
        cur = _sse(s, c, idx)
        if prev is not None:
            assert cur <= prev * (1 + 1e-6)
        prev = cur
        c, _ = orc.lloyd(s, c, 1)
        assert (np.diff(c) >= 0).all()
        assert c.min() >= s.min() and c.max() <= s.max()


def test_kmeans_start_small_sets_and_constant_values():
    s = np.array([3.0, -1.0, 2.0], np.float32)
    c = orc.kmeans_start(s, 15, 0, 0, 0)
    assert sorted(set(c.tolist())) == [-1.0, 2.0, 3.0]
    c2, idx = orc.lloyd(s, c, 10)
    np.testing.assert_array_equal(c2[idx], s)                       # fewer values than centres: lossless
    const = np.full(500, 0.375, np.float32)
    c3, idx3 = orc.lloyd(const, orc.kmeans_start(const, 15, 9, 1, 2), 10)
    assert (c3 == np.float32(0.375)).all() and len(set(idx3.tolist())) == 1
    assert not orc.kmeans_start(np.zeros(0, np.float32), 15, 0, 0, 0).any()


def test_zeros_of_either_sign_among_the_kept_values_have_one_order():
    """-0 and +0 are equal as numbers but not as stored centres; they can only be kept when pruning is off.
    The order is fixed (-0 first), so the centres do not depend on the sorting routine or on the order
    in which equal values arrive."""
    x = np.array([0.0, 2.0, -0.0, -3.0, 0.0, -0.0, 1e-45, -1e-45], np.float32)
    for perm in (np.arange(8), np.arange(8)[::-1], np.array([2, 0, 5, 4, 1, 3, 7, 6])):
        got = orc.sort_values(x[perm])
        want = sorted(x[perm].tolist(), key=lambda v: (v, not math.copysign(1.0, v) < 0))     # python's sort: by value, then the sign
        assert got.tolist() == want and np.signbit(got).tolist() == [True, True, True, True, False, False, False, False]
    # a stream of zeros of both signs and a few values: the first centres are -0, then +0, whatever the order of the input
    rng = np.random.default_rng(3)
    s = np.zeros(4000, np.float32)
    s[rng.random(4000) < 0.5] = -0.0
    s[::400] = rng.standard_normal(10).astype(np.float32)
    c0 = orc.kmeans_start(s, 15, 1, 0, 1)
    zeros = c0[c0 == 0]
    assert zeros.size >= 10 and np.signbit(zeros).any() and not np.signbit(zeros).all()
    assert (np.diff(np.signbit(zeros).astype(int)) <= 0).all()      # all -0 before all +0
    c, idx = orc.lloyd(s, c0, 5)
    zeros = c[c == 0]
    assert (np.diff(c) >= 0).all() and (np.diff(np.signbit(zeros).astype(int)) <= 0).all()
    assert (c[idx][s == 0] == 0).all()


def test_kmeans_start_sample_is_stratified():
    s = np.arange(10240, dtype=np.float32)
    c = orc.kmeans_start(s, 15, 123, 4, 1)
    # sample i lies in [10 i, 10 i + 10): the j-th quantile is within one stratum of its ideal place
    for j in range(15):
        pick = ((2 * j + 1) * 1024) // 30
        assert 10 * pick <= c[j] < 10 * pick + 10
    assert not np.array_equal(c, orc.kmeans_start(s, 15, 124, 4, 1))


# ---------------------------------------------------------------- byte layout
def test_record_layout_by_independent_parse():
    w_t, w_prev, ea, eas = _rand_quad(1000, 6)
    p = orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL)
    blob, info = orc.compress_tensor(w_t, w_prev, ea, eas, p)
    magic, ver = struct.unpack_from("<II", blob, 0)
    assert blob[:4] == b"EXCP" and ver == 1
    numel, nnz_w, nnz_o = struct.unpack_from("<QQQ", blob, 8)
    bits, k, hb = struct.unpack_from("<III", blob, 32)
    total, = struct.unpack_from("<Q", blob, 48)
    assert (numel, bits, k, hb, total) == (1000, 4, 15, 256, len(blob))
    assert nnz_w == info["nnz_w"] and nnz_o == info["nnz_o"]
    cents = np.frombuffer(blob, "<f4", 45, 64)
    np.testing.assert_array_equal(cents[:15], info["c_w"])
    np.testing.assert_array_equal(cents[30:], info["c_eas"])
    words = np.frombuffer(blob, "<u4", 32, hb)                      # ceil(1000/32) = 32 words
    for i in (0, 1, 31, 32, 33, 500, 999):
        assert bool((words[i // 32] >> (i % 32)) & 1) == bool(info["m_w"][i])
    assert words[31] >> 8 == 0                                      # bits past numel are zero
    off_codes = hb + 2 * 128
    raw = blob[off_codes:off_codes + (nnz_w + 1) // 2]
    for r in (0, 1, 2, nnz_w - 1):
        nib = (raw[r // 2] >> (4 * (r % 2))) & 15
        assert nib == info["codes_w"][r]
    if nnz_w % 2:
        assert raw[-1] >> 4 == 0
    assert len(blob) % 16 == 0


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_pack_unpack_codes_roundtrip(bits):
    rng = np.random.default_rng(bits)
    for n in (0, 1, 2, 3, 7, 8, 9, 31, 100):
        codes = rng.integers(1, 1 << bits, n).astype(np.uint8)
        raw = orc.pack_codes(codes, bits)
        assert len(raw) == orc.code_bytes(n, bits)
        np.testing.assert_array_equal(orc.unpack_codes(raw, n, bits), codes)
    assert orc.pack_codes(np.array([1, 2, 3], np.uint8), 4)[:2] == bytes([0x21, 0x03])
    assert orc.pack_codes(np.array([1, 2, 3, 1, 2], np.uint8), 2)[:2] == bytes([0b01111001, 0b10])


def test_corrupt_records_are_refused():
    w_t, w_prev, ea, eas = _rand_quad(300, 8)
    blob, _ = orc.compress_tensor(w_t, w_prev, ea, eas, orc.Params(median_source=1))
    for pos, val in ((0, 0), (4, 9), (8, 1), (16, 255), (32, 3), (48, 1)):
        bad = bytearray(blob); bad[pos] = val
        with pytest.raises(orc.CorruptBlob):
            orc.parse_record(bytes(bad))
    bad = bytearray(blob); bad[256] ^= 1                            # flip a mask bit: population changes
    with pytest.raises(orc.CorruptBlob):
        orc.parse_record(bytes(bad))
    with pytest.raises(orc.CorruptBlob):
        orc.parse_record(blob[:40])
    # padding is zero by the layout: a bit set past the last element (300 elements: bits 300..319 of the
    # tenth word, then two whole padding words up to 48 bytes) leaves the first 300 bits and their
    # population untouched and must still be refused, in either bitmap
    hb, bb = orc.header_bytes(15), orc.bitmap_bytes(300)
    assert (hb, bb) == (256, 48)
    for start in (hb, hb + bb):
        for bit in (300, 319, 320, 383):
            bad = bytearray(blob); bad[start + bit // 8] |= 1 << (bit % 8)
            with pytest.raises(orc.CorruptBlob):
                orc.parse_record(bytes(bad))
    assert orc.parse_record(blob)["numel"] == 300                   # the record itself is fine


# ---------------------------------------------------------------- chain (Algorithm 3's loop)
def test_chain_error_does_not_accumulate():
    rng = np.random.default_rng(21)
    n = 6000
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    w_hat = w.copy()
    p = orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL)
    errs = []
    for k in range(5):
        d = (rng.standard_t(3, n) * 1e-4 / math.sqrt(3)).astype(np.float32)
        w = (w + d).astype(np.float32)
        ea = (rng.standard_normal(n) * 1e-4).astype(np.float32)
        eas = ((np.abs(rng.standard_normal(n)) * 1e-4) ** 2 + 1e-12).astype(np.float32)
        blob, info = orc.compress_tensor(w, w_hat, ea, eas, p, tensor_index=0)
        new_hat, _, _ = orc.decompress_tensor(blob, w_hat)
        # residual taken against the reconstruction: the error of step k is the
        # quantisation/pruning error of this step's residual alone
        dq = np.zeros(n, np.float32)
        dq[info["m_w"]] = info["c_w"][info["codes_w"].astype(int) - 1]
        np.testing.assert_allclose(w - new_hat, info["dw"] - dq, atol=4e-9)
        errs.append(float(np.abs(w - new_hat).max()))
        w_hat = new_hat
    assert max(errs) < 3 * min(errs) + 1e-6


def test_checkpoint_container_offsets():
    quads = [_rand_quad(n, 30 + n) for n in (0, 1, 33, 500)]
    blob, offs, infos = orc.compress_checkpoint(quads, orc.Params(median_source=1, seed=3))
    assert offs[0] == 0 and offs[-1] == len(blob) and all(o % 16 == 0 for o in offs)
    outs = orc.decompress_checkpoint(blob, offs, [q[1] for q in quads])
    for (w_t, w_prev, ea, eas), (w_hat, ea_hat, eas_hat), info in zip(quads, outs, infos):
        assert w_hat.size == w_t.size
        np.testing.assert_array_equal(w_hat[~info["m_w"]], w_prev[~info["m_w"]])
    # the tensor index enters the K-means start
    b0, _ = orc.compress_tensor(*quads[3], orc.Params(median_source=1, seed=3), tensor_index=3)
    assert b0 == blob[offs[3]:offs[4]]


# ------------------------------------------- dense index layout (Sections 3.3 / 4.2) and the archiver
def rand_quad(n, seed):
    rng = np.random.default_rng(seed)
    wp = rng.normal(0, 0.02, n).astype(np.float32)
    wt = (wp + rng.standard_t(3, n) * 1e-4).astype(np.float32)
    ea = rng.normal(0, 1e-4, n).astype(np.float32)
    eas = ((np.abs(rng.normal(0, 1, n)) * 1e-4) ** 2 + 1e-12).astype(np.float32)
    return wt, wp, ea, eas


def test_hand_dense_layout():
    p = orc.Params(alpha=G["alpha"][0], beta=G["beta"][0], bits=4)
    blob, info = orc.compress_tensor(f32("w_t"), f32("w_prev"), f32("ea"), f32("eas"), p)
    dense = orc.record_to_dense(blob)
    hb = orc.header_bytes(15)
    assert len(dense) == hb + 3 * 16 == orc.dense_bytes(8, 4)
    head = struct.unpack_from("<IIQQQIIIIQQ", dense, 0)
    assert head == (0x44435845, 1, 8, 5, 2, 4, 15, hb, 0, len(dense), 0)
    assert dense[64:hb] == blob[64:hb]                          # the same centres
    for j, key in enumerate(("w", "ea", "eas")):
        sec = dense[hb + 16 * j:hb + 16 * (j + 1)]
        assert list(sec[:4]) == [int(v) for v in G[f"dense_bytes_{key}_abs_weight"]]
        assert sec[4:] == b"\0" * 12
    r = orc.parse_dense(dense)
    for key in ("w", "ea", "eas"):
        assert list(r["idx_" + key]) == [int(v) for v in G[f"dense_idx_{key}_abs_weight"]]
    w, ea, eas = orc.decompress_dense(dense, f32("w_prev"))
    np.testing.assert_array_equal(w, f32("w_hat_abs_weight"))
    np.testing.assert_array_equal(ea, f32("ea_hat_abs_weight"))
    np.testing.assert_array_equal(eas, f32("eas_hat_abs_weight"))


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("n", [1, 31, 1000, 4099])
def test_dense_layout_by_independent_unpacking(bits, n):
    wt, wp, ea, eas = rand_quad(n, 100 + n + bits)
    p = orc.Params(bits=bits, median_source=orc.MEDIAN_ABS_RESIDUAL, kmeans_iters=3)
    blob, info = orc.compress_tensor(wt, wp, ea, eas, p)
    dense = orc.record_to_dense(blob)
    k = (1 << bits) - 1
    hb = 16 * ((64 + 12 * k + 15) // 16)
    sb = 16 * (((n * bits + 7) // 8 + 15) // 16)
    assert len(dense) == hb + 3 * sb
    # element i is `bits` bits at bit i*bits of its section; 0 exactly where the mask prunes,
    # else the code of the survivor with i's rank
    for j, (mask, codes) in enumerate(((info["m_w"], info["codes_w"]), (info["m_o"], info["codes_ea"]),
                                       (info["m_o"], info["codes_eas"]))):
        sec = int.from_bytes(dense[hb + j * sb:hb + (j + 1) * sb], "little")
        rank = 0
        for i in range(n):
            got = (sec >> (i * bits)) & k
            if mask[i]:
                assert got == codes[rank]
                rank += 1
            else:
                assert got == 0
        assert sec >> (n * bits) == 0                         # padding
    a = orc.decompress_tensor(blob, wp)
    b = orc.decompress_dense(dense, wp)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x.view(np.uint32), y.view(np.uint32))


def test_corrupt_dense_containers_are_refused():
    wt, wp, ea, eas = rand_quad(500, 7)
    blob, info = orc.compress_tensor(wt, wp, ea, eas, orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL))
    dense = bytearray(orc.record_to_dense(blob))
    hb = orc.header_bytes(15)
    sb = orc.dense_section_bytes(500, 4)
    orc.parse_dense(bytes(dense))
    for mutate in ("magic", "short", "population", "orphan moment", "moments disagree"):
        d = bytearray(dense)
        if mutate == "magic":
            d[0] ^= 1
        elif mutate == "short":
            d = d[:-16]
        elif mutate == "population":
            i = int(np.flatnonzero(~info["m_w"])[0])
            d[hb + i // 2] |= 1 << (4 * (i % 2))
        elif mutate == "orphan moment":
            i = int(np.flatnonzero(~info["m_w"])[0])
            for j in (1, 2):
                d[hb + j * sb + i // 2] |= 1 << (4 * (i % 2))
            struct.pack_into("<Q", d, 24, info["nnz_o"] + 1)
        else:
            i = int(np.flatnonzero(info["m_w"] & ~info["m_o"])[0])
            d[hb + sb + i // 2] |= 1 << (4 * (i % 2))
            struct.pack_into("<Q", d, 24, info["nnz_o"] + 1)
        with pytest.raises(orc.CorruptBlob):
            orc.parse_dense(bytes(d))


def test_archiver_round_trip_and_sizes():
    wt, wp, ea, eas = rand_quad(20000, 11)
    blob, _ = orc.compress_tensor(wt, wp, ea, eas, orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL))
    dense = orc.record_to_dense(blob)
    a, b = orc.archive_sizes([blob]), orc.archive_sizes([dense])
    assert a["raw_bytes"] == len(blob) and b["raw_bytes"] == len(dense)
    assert 0 < a["archived_bytes"] <= len(blob) + 128 and 0 < b["archived_bytes"] < len(dense)
    z = orc.archive_sizes([b"\0" * 100000])
    assert z["archived_bytes"] < 400                          # LZMA2 collapses a run of zeros


# ------------------------------------------------ ablation switches (ViT table caption, Section 4.4)
def hand_params(flags):
    return orc.Params(alpha=G["alpha"][0], beta=G["beta"][0], bits=4, flags=flags)


def test_hand_ablation_masks():
    q = (f32("w_t"), f32("w_prev"), f32("ea"), f32("eas"))
    _, a = orc.compress_tensor(*q, hand_params(orc.FLAG_NO_W2M))
    np.testing.assert_array_equal(a["m_w"].astype(int), np.array(G["m_w_abs_weight"], dtype=int))
    np.testing.assert_array_equal(a["m_o"].astype(int), np.array(G["m_o_no_w2m"], dtype=int))
    _, b = orc.compress_tensor(*q, hand_params(orc.FLAG_NO_M2W))
    assert b["thr_w"] == np.float32(0.25)
    np.testing.assert_array_equal(b["m_w"].astype(int), np.array(G["m_w_no_m2w"], dtype=int))
    np.testing.assert_array_equal(b["m_o"].astype(int), np.array(G["m_o_no_m2w"], dtype=int))
    blob, c = orc.compress_tensor(*q, hand_params(orc.FLAG_NO_RESIDUAL))
    np.testing.assert_array_equal(c["m_w"].astype(int), np.array(G["m_w_no_residual"], dtype=int))
    w_hat, _, _ = orc.decompress_tensor(blob, f32("w_prev"))
    np.testing.assert_array_equal(w_hat, f32("w_hat_no_residual"))
    _, d = orc.compress_tensor(*q, hand_params(orc.FLAG_NO_PRUNE))
    assert d["m_w"].all() and d["m_o"].all() and d["nnz_w"] == d["nnz_o"] == 8


@pytest.mark.parametrize("flags", [1, 2, 4, 8, 16, 1 | 16, 4 | 8, 2 | 1, 4 | 16, 31])
def test_ablation_variants_by_independent_parse_and_definitions(flags):
    n = 3000
    wt, wp, ea, eas = rand_quad(n, 300 + flags)
    p = orc.Params(alpha=5e-5 if not flags & orc.FLAG_NO_M2W else 1e-4, median_source=orc.MEDIAN_ABS_RESIDUAL,
                   kmeans_iters=3, flags=flags)
    blob, info = orc.compress_tensor(wt, wp, ea, eas, p)
    dw = wt if flags & 4 else (wt - wp).astype(np.float32)
    np.testing.assert_array_equal(info["dw"], dw)
    # the masks, straight from their definitions
    if flags & 8:
        m_w = np.ones(n, bool); m_o = np.ones(n, bool)
    else:
        if flags & 2:
            m_w = np.abs(dw) > np.float32(1e-4)
        else:
            med = np.sort(np.abs(dw))[(n - 1) // 2]
            m_w = np.abs(dw) * np.sqrt(eas) > np.float32(np.float32(5e-5) * med)
        m_o = np.abs(ea) > np.float32(np.float32(2.0) * orc.exact_mean_abs(ea))
        if not flags & 1:
            m_o &= m_w
    np.testing.assert_array_equal(info["m_w"], m_w)
    np.testing.assert_array_equal(info["m_o"], m_o)
    # the header's words, read with struct alone
    head = struct.unpack_from("<IIQQQIIIIQQ", blob, 0)
    want_flags = (1 if flags & 1 else 0) | (2 if flags & 4 else 0) | (4 if flags & 16 else 0)
    bits, k = (32, 0) if flags & 16 else (4, 15)
    hb = 64 if flags & 16 else 256
    assert head[5:9] == (bits, k, hb, want_flags)
    nw, no = int(m_w.sum()), int(m_o.sum())
    a16 = lambda x: (x + 15) // 16 * 16
    bb = a16(4 * ((n + 31) // 32))
    assert len(blob) == head[9] == hb + 2 * bb + a16((nw * bits + 7) // 8) + 2 * a16((no * bits + 7) // 8)
    w_hat, ea_hat, eas_hat = orc.decompress_tensor(blob, wp)
    if flags & 16:                                       # raw survivors: fp32 straight out of the sections
        off = hb + 2 * bb
        np.testing.assert_array_equal(np.frombuffer(blob, "<f4", nw, off), dw[m_w])
        off += a16(4 * nw)
        np.testing.assert_array_equal(np.frombuffer(blob, "<f4", no, off), ea[m_o])
        np.testing.assert_array_equal(np.frombuffer(blob, "<f4", no, off + a16(4 * no)), eas[m_o])
        base = np.zeros(n, np.float32) if flags & 4 else wp
        want_w = base.copy(); want_w[m_w] = (base[m_w] + dw[m_w]).astype(np.float32)
        np.testing.assert_array_equal(w_hat, want_w)
        np.testing.assert_array_equal(ea_hat, np.where(m_o, ea, 0).astype(np.float32))
        np.testing.assert_array_equal(eas_hat, np.where(m_o, eas, 0).astype(np.float32))
    else:
        base = np.zeros(n, np.float32) if flags & 4 else wp
        np.testing.assert_array_equal(w_hat[~m_w], base[~m_w])
        assert np.all(ea_hat[~m_o] == 0) and np.all(eas_hat[~m_o] == 0)
        r = orc.parse_record(blob)
        np.testing.assert_array_equal(w_hat[m_w], (base[m_w] + r["c_w"][r["codes_w"].astype(int) - 1]).astype(np.float32))
    if want_flags:
        with pytest.raises(ValueError):
            orc.record_to_dense(blob)


def test_flagged_records_keep_their_rules():
    wt, wp, ea, eas = rand_quad(2000, 41)
    blob, info = orc.compress_tensor(wt, wp, ea, eas, orc.Params(median_source=1, flags=orc.FLAG_NO_W2M))
    assert np.any(info["m_o"] & ~info["m_w"])            # moments kept where weights are pruned ...
    b = bytearray(blob); struct.pack_into("<I", b, 44, 0)
    with pytest.raises(orc.CorruptBlob):                 # ... which a record of the full method may not hold
        orc.parse_record(bytes(b))
    b = bytearray(blob); struct.pack_into("<I", b, 44, 8)
    with pytest.raises(orc.CorruptBlob):
        orc.parse_record(bytes(b))
    with pytest.raises(ValueError):
        orc.compress_tensor(wt, wp, ea, eas, orc.Params(flags=32))


# ------------------------------------------------ 16-bit weight storage (Section 4.3: float16 weights)
def test_widening_is_exact_on_known_patterns():
    f16 = np.array([0x3C00, 0xBC00, 0x0001, 0x7BFF, 0x0400, 0x8000], dtype=np.uint16).view(np.float16)
    want = np.array([1.0, -1.0, 2.0 ** -24, 65504.0, 2.0 ** -14, -0.0], dtype=np.float32)
    got = orc.widen_weights(f16, orc.WEIGHTS_F16)
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    bf = np.array([0x3F80, 0xBF80, 0x0001, 0x7F7F, 0x0080, 0x8000], dtype=np.uint16)
    want = np.array([1.0, -1.0, 2.0 ** -133, (2 - 2.0 ** -7) * 2.0 ** 127, 2.0 ** -126, -0.0], dtype=np.float32)
    got = orc.widen_weights(bf, orc.WEIGHTS_BF16)
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))


def _nearest_even(x: float, candidates):
    """Nearest of the candidate values (exact rationals), ties to the one with an even index."""
    fx = Fraction(x)
    best = min(range(len(candidates)), key=lambda i: (abs(Fraction(candidates[i]) - fx), i % 2))
    return candidates[best]


@pytest.mark.parametrize("fmt", [orc.WEIGHTS_F16, orc.WEIGHTS_BF16])
def test_narrowing_is_round_to_nearest_even(fmt):
    rng = np.random.default_rng(5)
    # all positive values of the format in [2^-3, 2^1], in order: index parity = mantissa parity
    if fmt == orc.WEIGHTS_F16:
        pats = np.arange(0x3000, 0x4001, dtype=np.uint16)
        grid = [float(v) for v in pats.view(np.float16).astype(np.float64)]
    else:
        pats = np.arange(0x3E00, 0x4001, dtype=np.uint16)
        grid = [float(v) for v in (pats.astype(np.uint32) << 16).view(np.float32).astype(np.float64)]
    xs = rng.uniform(0.125, 2.0, 400).astype(np.float32)
    ties = np.array([(grid[i] + grid[i + 1]) / 2 for i in range(0, 60)], dtype=np.float32)   # exact mid-points
    for x in np.concatenate([xs, ties, -ties[:8]]):
        want = _nearest_even(abs(float(x)), grid) * (1 if x > 0 else -1)
        got = orc.widen_weights(orc.narrow_weights(np.array([x], np.float32), fmt), fmt)[0]
        assert float(got) == want, (x, got, want)
    # stored values survive a round trip bit for bit
    back = orc.narrow_weights(orc.widen_weights(pats.view(np.float16) if fmt == orc.WEIGHTS_F16 else pats, fmt), fmt)
    np.testing.assert_array_equal(back.view(np.uint16), pats)


@pytest.mark.parametrize("fmt", [orc.WEIGHTS_F16, orc.WEIGHTS_BF16])
def test_sixteen_bit_weights_take_the_fp32_path_after_widening(fmt):
    wt, wp, ea, eas = rand_quad(5000, 61)
    n16 = lambda a: orc.narrow_weights(a, fmt)
    wp16 = n16(wp)
    wt16 = n16((orc.widen_weights(wp16, fmt) + (wt - wp) * 30).astype(np.float32))   # residuals a 16-bit format can hold
    p = orc.Params(median_source=orc.MEDIAN_ABS_RESIDUAL, kmeans_iters=3)
    blob, info = orc.compress_tensor(wt16, wp16, ea, eas, p, weight_format=fmt)
    blob32, _ = orc.compress_tensor(orc.widen_weights(wt16, fmt), orc.widen_weights(wp16, fmt), ea, eas, p)
    assert blob == blob32 and 0 < info["nnz_w"] < 5000
    w_hat, ea_hat, eas_hat = orc.decompress_tensor(blob, wp16, weight_format=fmt)
    assert w_hat.dtype == (np.float16 if fmt == orc.WEIGHTS_F16 else np.uint16)
    w32, ea32, eas32 = orc.decompress_tensor(blob, orc.widen_weights(wp16, fmt))
    np.testing.assert_array_equal(w_hat.view(np.uint16), n16(w32).view(np.uint16))
    np.testing.assert_array_equal(ea_hat, ea32)
    pruned = ~info["m_w"]
    np.testing.assert_array_equal(w_hat.view(np.uint16)[pruned], wp16.view(np.uint16)[pruned])
