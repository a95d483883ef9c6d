"""CPU oracle for the ExCP per-tensor compression path (arXiv 2406.11257).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, single-threaded
statement of what the CUDA library must compute.  It shares no code with the
CUDA path and is never imported by it; only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

What is written from the paper, and where the paper is silent:

  * residual                 Section 3.1, Eq. (ckpt_res); Algorithm 1, step 1
  * weight mask  (M2W)       Section 3.2, Eq. (rw)
  * moment mask  (W2M)       Section 3.2, Eq. (ro)
  * joint application        Algorithm 1, step 2 ("joint_prune")
  * non-uniform quantisation Section 3.3 (K-means to 2^n - 1 centres, zero keeps
                             one code) and Section 4.2 (n = 4, two codes per byte)
  * reconstruction           Algorithm 2

The paper does not say how the median, the mean, the K-means start, its
iteration count, its arithmetic or the byte layout are to be taken.  The
readings used here (all of them deterministic, so that the result is unique):

  R1  median(W) in Eq. (rw) is the LOWER median (rank floor((n-1)/2)) of the
      absolute values of either W_t (the letter of the text) or dW_t (the
      quantity actually pruned); `median_source` selects.
  R2  the mask of Eq. (rw) compares |dW(i)| * sqrt(m_t(i)) > alpha * median in
      fp32 (the product form of |dW(i)| > alpha / sqrt(m_t(i)) * median, which
      also settles m_t(i) = 0 as "pruned").
  R3  mean(v_t) in Eq. (ro) is the mean of |v_t|, taken EXACTLY (as a rational
      number) and rounded once to fp32, round-to-nearest-even.
  R4  both Adam moments take the mask M_o (Appendix A prunes "the moments").
  R5  K-means is Lloyd's algorithm in one dimension, per tensor and per stream
      (dW, first moment, second moment), K = 2^bits - 1 centres:
        start   the K equal-mass quantiles of a seeded, index-stratified sample
                of at most 1024 surviving values;
        assign  nearest centre, a point on a mid-point going to the lower
                centre, the mid-point of two neighbours taken in fp64:
                cluster(x) = #{ j : 2x > c_j + c_(j+1) }
                (of coincident centres the first takes the points at or
                below them, the last those above);
        update  fixed-point mean (rule R-SUM below); a cluster without members
                keeps its centre; centres are re-sorted ascending;
        T fixed iterations, then one last assignment gives the codes 1..K.
  R-SUM a sum that feeds a centre is taken in fixed point so that its value
      cannot depend on the order of summation: with E = max(floor(log2(max|x|)),
      -126) over the stream, Q(x) = rint(x * 2^(30-E)) (half-to-even), the sum
      of Q in int64, mean = fp32( fp64(sum) / fp64(count) * 2^(E-30) ).
  R6  byte layout: see `encode_record`; the layout the paper prints (an index
      per element, 0 = pruned) is `encode_dense`, derived from the record.

The paper calls Adam's first moment v_t and its second moment m_t; to stay clear
of the clash with the usual letters the code below says `ea` (first moment,
exp_avg) and `eas` (second moment, exp_avg_sq).

Parity status: every function below is pinned by tests/test_oracle_pins.py
(hand-computed example, brute force, exact rational arithmetic, invariants).
"""
from __future__ import annotations

import math
import struct
from dataclasses import dataclass
from fractions import Fraction

import numpy as np

MAGIC = 0x50435845  # "EXCP", little endian
VERSION = 1
SAMPLE_MAX = 1024
HEADER_FIXED = 64

MEDIAN_ABS_WEIGHT = 0
MEDIAN_ABS_RESIDUAL = 1

# Ablation switches (the M2W / W2M columns of the ViT table, the residual / prune / quant columns
# of the ablation table in Section 4.4).  0 = the full method.
FLAG_NO_W2M = 1        # M_o(i) = [ |ea(i)| > r_o ] without the conjunction with M_w
FLAG_NO_M2W = 2        # weights pruned by a set threshold: M_w(i) = [ |dW(i)| > alpha ]
FLAG_NO_RESIDUAL = 4   # the weights themselves are compressed, not their residual
FLAG_NO_PRUNE = 8      # every element is kept
FLAG_NO_QUANT = 16     # the survivors are stored as fp32, no K-means
FLAGS_ALL = 31
# What a record says about itself at header offset 44
REC_MOMENTS_FREE = 1   # M_o need not lie inside M_w
REC_ABSOLUTE = 2       # the weight stream is W, not dW: Algorithm 2 does not add W^_(t-1)
REC_RAW = 4            # sections hold fp32 survivors (bits = 32, K = 0)

_M64 = (1 << 64) - 1


# Storage format of the WEIGHT tensors (W_t, W^_(t-1), the reconstructed W^_t).  Section 4.3 notes
# that the PanGu-pi weights are saved in float16.  The moments stay fp32.
WEIGHTS_F32 = 0
WEIGHTS_F16 = 1        # numpy float16 arrays
WEIGHTS_BF16 = 2       # numpy uint16 arrays holding the upper 16 bits of an fp32 pattern


def widen_weights(w: np.ndarray, weight_format: int) -> np.ndarray:
    """Stored weights -> fp32, exactly (both 16-bit formats are subsets of fp32)."""
    if weight_format == WEIGHTS_F32:
        return np.ascontiguousarray(w, dtype=np.float32).ravel()
    if weight_format == WEIGHTS_F16:
        w = np.ascontiguousarray(w).ravel()
        if w.dtype != np.float16:
            raise TypeError("float16 expected")
        return w.astype(np.float32)
    if weight_format == WEIGHTS_BF16:
        w = np.ascontiguousarray(w).ravel()
        if w.dtype != np.uint16:
            raise TypeError("uint16 bit patterns expected")
        return (w.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError("weight format")


def narrow_weights(w32: np.ndarray, weight_format: int) -> np.ndarray:
    """fp32 -> the stored format, round to nearest, ties to even (finite inputs; a magnitude
    beyond the format's range becomes infinity, as IEEE rounding has it)."""
    w32 = np.ascontiguousarray(w32, dtype=np.float32)
    if weight_format == WEIGHTS_F32:
        return w32
    if weight_format == WEIGHTS_F16:
        with np.errstate(over="ignore"):
            return w32.astype(np.float16)
    if weight_format == WEIGHTS_BF16:
        bits = w32.view(np.uint32).astype(np.uint64)
        bits = bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1))
        return (bits >> np.uint64(16)).astype(np.uint16)
    raise ValueError("weight format")


@dataclass
class Params:
    """Hyper-parameters.  alpha, beta, bits: Section 4.2 (5e-5, 2.0, 4)."""
    alpha: float = 5e-5
    beta: float = 2.0
    bits: int = 4
    kmeans_iters: int = 10
    seed: int = 0
    median_source: int = MEDIAN_ABS_WEIGHT
    flags: int = 0


class InvalidInput(ValueError):
    """A NaN, an infinity, or a negative second moment in the inputs."""


class CorruptBlob(ValueError):
    """The record does not parse."""


# --------------------------------------------------------------------------
# Section 3.1: residual
# --------------------------------------------------------------------------
def residual(w_t: np.ndarray, w_prev: np.ndarray) -> np.ndarray:
    """dW_t = W_t - W^_(t-1), fp32 (Eq. ckpt_res; Algorithm 1, first step)."""
    return np.subtract(w_t, w_prev, dtype=np.float32)


# --------------------------------------------------------------------------
# Section 3.2: statistics behind the two thresholds
# --------------------------------------------------------------------------
def lower_median_abs(x: np.ndarray) -> np.float32:
    """Lower median of |x| (reading R1): the element of rank floor((n-1)/2)."""
    n = x.size
    if n == 0:
        return np.float32(0.0)
    a = np.abs(x.astype(np.float32, copy=False))
    k = (n - 1) // 2
    return np.float32(np.partition(a, k)[k])


def round_ratio_to_f32(num: int, den: int) -> np.float32:
    """The fp32 value nearest to num/den (num >= 0, den > 0), ties to even,
    subnormals included; integer arithmetic only."""
    if num < 0 or den <= 0:
        raise ValueError("num >= 0 and den > 0 required")
    if num == 0:
        return np.float32(0.0)
    e = num.bit_length() - den.bit_length()
    # make 2^e <= num/den < 2^(e+1)
    if e >= 0:
        below = num < (den << e)
    else:
        below = (num << -e) < den
    if below:
        e -= 1
    u = max(e - 23, -149)            # exponent of the last kept bit
    if u >= 0:
        n_, d_ = num, den << u
    else:
        n_, d_ = num << -u, den
    m, r = divmod(n_, d_)
    if 2 * r > d_ or (2 * r == d_ and (m & 1)):
        m += 1
    return np.float32(math.ldexp(m, u))


def exact_sum_abs_units(x: np.ndarray) -> int:
    """sum |x_i| as an integer count of 2^-149 (every fp32 is a multiple of it)."""
    a = np.abs(x.astype(np.float32, copy=False)).ravel()
    if a.size >= (1 << 29):
        raise ValueError("tensor too large for the exact per-exponent sums")
    bits = a.view(np.uint32)
    e = (bits >> 23).astype(np.int64)
    m = (bits & np.uint32(0x7FFFFF)).astype(np.int64)
    m = np.where(e > 0, m | (1 << 23), m)
    e1 = np.maximum(e, 1)            # subnormals share the exponent of 2^-126
    total = 0
    # 24-bit mantissas times fewer than 2^29 terms stay below 2^53: the
    # float64 weights of bincount add without rounding.
    per_exp = np.bincount(e1, weights=m.astype(np.float64), minlength=256)
    for ee in range(1, 256):
        s = int(per_exp[ee])
        if s:
            total += s << (ee - 1)   # value = m * 2^(ee-150) = m * 2^(ee-1) units
    return total


def exact_mean_abs(x: np.ndarray) -> np.float32:
    """mean(|x|), exact then rounded once to fp32 (reading R3)."""
    n = x.size
    if n == 0:
        return np.float32(0.0)
    return round_ratio_to_f32(exact_sum_abs_units(x), n << 149)


def validate_inputs(w_t, w_prev, ea, eas) -> None:
    for a in (w_t, w_prev, ea, eas):
        if not np.all(np.isfinite(a)):
            raise InvalidInput("non-finite input")
    if np.any(eas < 0):
        raise InvalidInput("negative second moment")


# --------------------------------------------------------------------------
# Section 3.2: the two masks and their joint application
# --------------------------------------------------------------------------
def weight_mask(dw: np.ndarray, eas: np.ndarray, alpha, med) -> tuple[np.ndarray, np.float32]:
    """M_w of Eq. (rw) in the product form of reading R2."""
    thr_w = np.float32(np.float32(alpha) * np.float32(med))
    lhs = np.abs(dw).astype(np.float32) * np.sqrt(eas.astype(np.float32))
    return lhs > thr_w, thr_w


def moment_mask(ea: np.ndarray, m_w: np.ndarray, beta, mean) -> tuple[np.ndarray, np.float32]:
    """M_o of Eq. (ro): |first moment| above beta * mean AND the weight kept."""
    thr_o = np.float32(np.float32(beta) * np.float32(mean))
    return (np.abs(ea) > thr_o) & m_w, thr_o


def weight_mask_set_threshold(dw: np.ndarray, alpha) -> tuple[np.ndarray, np.float32]:
    """The "no M2W" row of the ViT table: the weights are pruned by a threshold that is set,
    not derived from the second moment; here alpha itself is that threshold."""
    thr_w = np.float32(alpha)
    return np.abs(dw).astype(np.float32) > thr_w, thr_w


def moment_mask_alone(ea: np.ndarray, beta, mean) -> tuple[np.ndarray, np.float32]:
    """The "no W2M" row of the ViT table: M_o(i) = [ |ea(i)| > r_o ], the weight mask ignored."""
    thr_o = np.float32(np.float32(beta) * np.float32(mean))
    return np.abs(ea) > thr_o, thr_o


# --------------------------------------------------------------------------
# Section 3.3: non-uniform quantisation (reading R5)
# --------------------------------------------------------------------------
def mix64(z: int) -> int:
    """One step of the SplitMix64 generator (Steele, Lea, Flood 2014) from state z."""
    z = (z + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def sample_hash(seed: int, tensor_index: int, stream: int, i: int) -> int:
    h = mix64((seed + tensor_index) & _M64)
    h = mix64((h + stream) & _M64)
    return mix64((h + i) & _M64)


def sort_values(x: np.ndarray) -> np.ndarray:
    """x in ascending order; of two zeros the negative one comes first.  Without the second rule
    the order of -0 and +0 (equal as numbers, different as stored centres) would be whatever the
    sorting routine happens to do.  They only meet when pruning is switched off: a kept value is
    never zero otherwise."""
    return x[np.lexsort((~np.signbit(x), x))]


def kmeans_start(s: np.ndarray, k: int, seed: int, tensor_index: int, stream: int) -> np.ndarray:
    """K equal-mass quantiles of a seeded, index-stratified sample of s."""
    nnz = s.size
    c = np.zeros(k, dtype=np.float32)
    if nnz == 0:
        return c
    m = min(nnz, SAMPLE_MAX)
    picks = np.empty(m, dtype=np.float32)
    for i in range(m):
        lo = (i * nnz) // m
        hi = ((i + 1) * nnz) // m
        picks[i] = s[lo + sample_hash(seed, tensor_index, stream, i) % (hi - lo)]
    picks = sort_values(picks)
    for j in range(k):
        c[j] = picks[((2 * j + 1) * m) // (2 * k)]
    return c


def assign(s: np.ndarray, c: np.ndarray) -> np.ndarray:
    """Nearest centre: the number of mid-points lying strictly below x."""
    x2 = 2.0 * s.astype(np.float64)
    idx = np.zeros(s.shape, dtype=np.int64)
    for j in range(len(c) - 1):
        idx += x2 > (np.float64(c[j]) + np.float64(c[j + 1]))
    return idx


def rsum_exponent(s: np.ndarray) -> int:
    if s.size == 0:
        return 0
    mx = float(np.max(np.abs(s)))
    if mx == 0.0:
        return 0
    return max(math.frexp(mx)[1] - 1, -126)


def rsum_quantize(s: np.ndarray, e: int) -> np.ndarray:
    return np.rint(np.ldexp(s.astype(np.float64), 30 - e)).astype(np.int64)


def rsum_mean(qsum: int, count: int, e: int) -> np.float32:
    return np.float32(math.ldexp(float(qsum) / float(count), e - 30))


def lloyd(s: np.ndarray, c0: np.ndarray, iters: int) -> tuple[np.ndarray, np.ndarray]:
    """T Lloyd iterations from c0, then the final assignment.
    Returns (centres, cluster index per value)."""
    c = c0.astype(np.float32).copy()
    k = len(c)
    if s.size == 0:
        return c, np.zeros(0, dtype=np.int64)
    e = rsum_exponent(s)
    q = rsum_quantize(s, e)
    for _ in range(iters):
        idx = assign(s, c)
        for j in range(k):
            members = idx == j
            cnt = int(np.count_nonzero(members))
            if cnt:
                c[j] = rsum_mean(int(q[members].sum(dtype=np.int64)), cnt, e)
        c = sort_values(c)
    return c, assign(s, c)


def quantisation_sse(s: np.ndarray, c: np.ndarray, idx: np.ndarray) -> float:
    """Sum of squared distances of the values to their assigned centres (the K-means objective of
    Section 3.3), in fp64.  A diagnostic: nothing in the record depends on it."""
    if s.size == 0:
        return 0.0
    d = s.astype(np.float64) - c.astype(np.float64)[idx]
    return float(np.sum(d * d))


# --------------------------------------------------------------------------
# Byte layout (reading R6)
# --------------------------------------------------------------------------
def _align16(n: int) -> int:
    return (n + 15) & ~15


def centres_of(bits: int) -> int:
    """K = 2^bits - 1 centres; none when the survivors are stored raw (bits = 32)."""
    return 0 if bits == 32 else (1 << bits) - 1


def header_bytes(k: int) -> int:
    return _align16(HEADER_FIXED + 3 * 4 * k)


def bitmap_bytes(numel: int) -> int:
    return _align16(4 * ((numel + 31) // 32))


def code_bytes(nnz: int, bits: int) -> int:
    return _align16((nnz * bits + 7) // 8)


def record_bytes(numel: int, nnz_w: int, nnz_o: int, bits: int) -> int:
    k = centres_of(bits)
    return (header_bytes(k) + 2 * bitmap_bytes(numel) + code_bytes(nnz_w, bits)
            + 2 * code_bytes(nnz_o, bits))


def pack_codes(codes: np.ndarray, bits: int) -> bytes:
    """Code r sits at bit r*bits of the stream, low bits first (Section 4.2:
    two 4-bit codes per byte)."""
    per = 8 // bits
    n = codes.size
    padded = np.zeros(((n + per - 1) // per) * per, dtype=np.uint8)
    padded[:n] = codes
    out = np.zeros(padded.size // per, dtype=np.uint8)
    for r in range(per):
        out |= (padded[r::per] << np.uint8(r * bits)).astype(np.uint8)
    raw = out.tobytes()
    return raw + b"\0" * (code_bytes(n, bits) - len(raw))


def unpack_codes(raw: bytes, nnz: int, bits: int) -> np.ndarray:
    per = 8 // bits
    b = np.frombuffer(raw, dtype=np.uint8)
    out = np.zeros(b.size * per, dtype=np.uint8)
    for r in range(per):
        out[r::per] = (b >> np.uint8(r * bits)) & np.uint8((1 << bits) - 1)
    return out[:nnz]


def pack_bitmap(mask: np.ndarray) -> bytes:
    """Bit k of 32-bit little-endian word w is element 32*w + k."""
    raw = np.packbits(mask.astype(np.uint8), bitorder="little").tobytes()
    return raw + b"\0" * (bitmap_bytes(mask.size) - len(raw))


def unpack_bitmap(raw: bytes, numel: int) -> np.ndarray:
    """The first numel bits.  The layout says that padding is zero: a bit set at or past numel
    (in the last word or in the words that fill the section up to 16 bytes) makes the record corrupt."""
    b = np.frombuffer(raw, dtype=np.uint8)
    bits = np.unpackbits(b, bitorder="little")
    if np.any(bits[numel:]):
        raise CorruptBlob("bitmap bit past the last element")
    return bits[:numel].astype(bool)


def encode_record(numel, bits, m_w, m_o, c_w, c_ea, c_eas, codes_w, codes_ea, codes_eas, rec_flags: int = 0) -> bytes:
    """One tensor's record.  Little endian; every section starts on 16 bytes;
    padding is zero.

      0  u32 magic "EXCP"     4  u32 version (1)    8  u64 numel
     16  u64 nnz_w           24  u64 nnz_o         32  u32 bits   36 u32 K
     40  u32 header bytes    44  u32 record flags  48  u64 record bytes
     56  u64 zero
     64  fp32 centres of dW [K], of the first moment [K], of the second [K]
     ..  bitmap of M_w, bitmap of M_o       (u32 words, LSB = lowest index)
     ..  codes of dW, of the first moment, of the second moment (survivors in
         index order, `bits` each, value 1..K)
    Record flags (ablation variants; 0 for the full method): REC_MOMENTS_FREE, REC_ABSOLUTE,
    REC_RAW.  With REC_RAW bits = 32, K = 0, there are no centres and the three sections hold
    the survivors themselves as fp32 (codes_* are then float32 arrays).
    """
    k = centres_of(bits)
    nnz_w = int(np.count_nonzero(m_w))
    nnz_o = int(np.count_nonzero(m_o))
    hb = header_bytes(k)
    total = record_bytes(numel, nnz_w, nnz_o, bits)
    head = struct.pack("<IIQQQIIIIQQ", MAGIC, VERSION, numel, nnz_w, nnz_o, bits, k, hb, rec_flags, total, 0)
    if k:
        head += np.asarray(c_w, dtype="<f4").tobytes()
        head += np.asarray(c_ea, dtype="<f4").tobytes()
        head += np.asarray(c_eas, dtype="<f4").tobytes()
    head += b"\0" * (hb - len(head))
    out = head + pack_bitmap(m_w) + pack_bitmap(m_o)
    for c in (codes_w, codes_ea, codes_eas):
        if bits == 32:
            raw = np.asarray(c, dtype="<f4").tobytes()
            out += raw + b"\0" * (code_bytes(len(c), 32) - len(raw))
        else:
            out += pack_codes(c, bits)
    assert len(out) == total
    return out


def parse_record(blob: bytes) -> dict:
    if len(blob) < HEADER_FIXED:
        raise CorruptBlob("short header")
    (magic, version, numel, nnz_w, nnz_o, bits, k, hb, rflags, total, z1) = struct.unpack_from(
        "<IIQQQIIIIQQ", blob, 0)
    if magic != MAGIC or version != VERSION:
        raise CorruptBlob("magic/version")
    if rflags & ~(REC_MOMENTS_FREE | REC_ABSOLUTE | REC_RAW):
        raise CorruptBlob("record flags")
    raw_values = bool(rflags & REC_RAW)
    if bits not in ((32,) if raw_values else (2, 4, 8)) or k != centres_of(bits) or hb != header_bytes(k):
        raise CorruptBlob("bits/K/header size")
    free = bool(rflags & REC_MOMENTS_FREE)
    if (nnz_o > nnz_w and not free) or nnz_w > numel or nnz_o > numel:
        raise CorruptBlob("counts")
    if total != record_bytes(numel, nnz_w, nnz_o, bits) or len(blob) < total:
        raise CorruptBlob("record size")
    cents = np.frombuffer(blob, dtype="<f4", count=3 * k, offset=HEADER_FIXED).reshape(3, k)
    off = hb
    bb = bitmap_bytes(numel)
    m_w = unpack_bitmap(blob[off:off + bb], numel); off += bb
    m_o = unpack_bitmap(blob[off:off + bb], numel); off += bb
    if np.count_nonzero(m_w) != nnz_w or np.count_nonzero(m_o) != nnz_o:
        raise CorruptBlob("bitmap population")
    if np.any(m_o & ~m_w) and not free:
        raise CorruptBlob("moment kept where the weight is pruned")
    cw = code_bytes(nnz_w, bits)
    co = code_bytes(nnz_o, bits)
    if raw_values:
        codes_w = np.frombuffer(blob, dtype="<f4", count=nnz_w, offset=off).copy(); off += cw
        codes_ea = np.frombuffer(blob, dtype="<f4", count=nnz_o, offset=off).copy(); off += co
        codes_eas = np.frombuffer(blob, dtype="<f4", count=nnz_o, offset=off).copy(); off += co
    else:
        codes_w = unpack_codes(blob[off:off + cw], nnz_w, bits); off += cw
        codes_ea = unpack_codes(blob[off:off + co], nnz_o, bits); off += co
        codes_eas = unpack_codes(blob[off:off + co], nnz_o, bits); off += co
        for c in (codes_w, codes_ea, codes_eas):
            if c.size and (c.min() < 1 or c.max() > k):
                raise CorruptBlob("code out of range")
    return dict(numel=numel, nnz_w=nnz_w, nnz_o=nnz_o, bits=bits, k=k, record_bytes=total, rec_flags=rflags,
                c_w=cents[0].copy(), c_ea=cents[1].copy(), c_eas=cents[2].copy(),
                m_w=m_w, m_o=m_o, codes_w=codes_w, codes_ea=codes_ea, codes_eas=codes_eas)


# --------------------------------------------------------------------------
# Algorithm 1 (without the archiver) and Algorithm 2
# --------------------------------------------------------------------------
def compress_tensor(w_t, w_prev, ea, eas, p: Params, tensor_index: int = 0, weight_format: int = WEIGHTS_F32):
    """Algorithm 1 for one tensor, up to (not including) the archiver.
    Returns (record bytes, dict of every intermediate).  Weights stored in a 16-bit format are
    widened exactly and then take the same path."""
    w_t = widen_weights(w_t, weight_format)
    w_prev = widen_weights(w_prev, weight_format)
    ea = np.ascontiguousarray(ea, dtype=np.float32).ravel()
    eas = np.ascontiguousarray(eas, dtype=np.float32).ravel()
    n = w_t.size
    if not (w_prev.size == ea.size == eas.size == n):
        raise ValueError("size mismatch")
    if p.bits not in (2, 4, 8):
        raise ValueError("bits")
    if p.flags & ~FLAGS_ALL:
        raise ValueError("flags")
    validate_inputs(w_t, w_prev, ea, eas)
    k = (1 << p.bits) - 1
    fl = p.flags

    # Algorithm 1, step 1 (ablation "residual" off: the weights themselves go on)
    dw = w_t.copy() if fl & FLAG_NO_RESIDUAL else residual(w_t, w_prev)
    src = w_t if p.median_source == MEDIAN_ABS_WEIGHT else dw
    med = lower_median_abs(src)
    mean = exact_mean_abs(ea)
    if fl & FLAG_NO_M2W:
        m_w, thr_w = weight_mask_set_threshold(dw, p.alpha)
    else:
        m_w, thr_w = weight_mask(dw, eas, p.alpha, med)               # Eq. (rw)
    if fl & FLAG_NO_W2M:
        m_o, thr_o = moment_mask_alone(ea, p.beta, mean)
    else:
        m_o, thr_o = moment_mask(ea, m_w, p.beta, mean)               # Eq. (ro)
    if fl & FLAG_NO_PRUNE:                                            # ablation "prune" off
        m_w = np.ones(n, dtype=bool)
        m_o = np.ones(n, dtype=bool)
    s_w, s_ea, s_eas = dw[m_w], ea[m_o], eas[m_o]                     # joint_prune

    rec_flags = ((REC_MOMENTS_FREE if fl & FLAG_NO_W2M else 0) | (REC_ABSOLUTE if fl & FLAG_NO_RESIDUAL else 0)
                 | (REC_RAW if fl & FLAG_NO_QUANT else 0))
    cents, codes, sse = [], [], []
    if fl & FLAG_NO_QUANT:                                            # ablation "quant" off
        zero = np.zeros(0, dtype=np.float32)
        cents = [zero, zero, zero]
        codes = [s_w, s_ea, s_eas]
        sse = [0.0, 0.0, 0.0]
        blob = encode_record(n, 32, m_w, m_o, zero, zero, zero, s_w, s_ea, s_eas, rec_flags)
    else:
        for stream, s in enumerate((s_w, s_ea, s_eas)):               # quantize(.)
            c0 = kmeans_start(s, k, p.seed, tensor_index, stream)
            c, idx = lloyd(s, c0, p.kmeans_iters)
            cents.append(c)
            codes.append((idx + 1).astype(np.uint8))
            sse.append(quantisation_sse(s, c, idx))
        blob = encode_record(n, p.bits, m_w, m_o, cents[0], cents[1], cents[2], *codes, rec_flags=rec_flags)
    info = dict(numel=n, dw=dw, median=med, mean_abs_ea=mean, thr_w=thr_w, thr_o=thr_o,
                m_w=m_w, m_o=m_o, nnz_w=int(m_w.sum()), nnz_o=int(m_o.sum()),
                s_w=s_w, s_ea=s_ea, s_eas=s_eas, c_w=cents[0], c_ea=cents[1], c_eas=cents[2],
                codes_w=codes[0], codes_ea=codes[1], codes_eas=codes[2],
                sse_w=sse[0], sse_ea=sse[1], sse_eas=sse[2])
    return blob, info


def decompress_tensor(blob: bytes, w_prev, weight_format: int = WEIGHTS_F32):
    """Algorithm 2: codes -> centres, W^_t = W^_(t-1) + dW^Q*; pruned entries
    keep W^_(t-1) unchanged and decode to 0 in both moments.  With 16-bit weights the sum is
    taken in fp32 and rounded once to the stored format (a pruned weight keeps its bits)."""
    r = parse_record(blob)
    w_prev = widen_weights(w_prev, weight_format)
    if w_prev.size != r["numel"]:
        raise ValueError("size mismatch")
    raw_values = bool(r["rec_flags"] & REC_RAW)
    val = (lambda c, codes: codes) if raw_values else (lambda c, codes: c[codes.astype(np.int64) - 1])
    kept = r["m_w"]
    if r["rec_flags"] & REC_ABSOLUTE:            # the stream is W itself: pruned weights are 0
        w_hat = np.zeros(r["numel"], dtype=np.float32)
        w_hat[kept] = val(r["c_w"], r["codes_w"])
    else:
        w_hat = w_prev.copy()
        w_hat[kept] = w_prev[kept] + val(r["c_w"], r["codes_w"])
    ea_hat = np.zeros(r["numel"], dtype=np.float32)
    eas_hat = np.zeros(r["numel"], dtype=np.float32)
    ea_hat[r["m_o"]] = val(r["c_ea"], r["codes_ea"])
    eas_hat[r["m_o"]] = val(r["c_eas"], r["codes_eas"])
    return narrow_weights(w_hat, weight_format), ea_hat, eas_hat


def compress_checkpoint(tensors, p: Params):
    """Algorithm 1 over a tensor list: records back to back; tensor i starts at
    offsets[i] and uses i as its index in the K-means start."""
    blobs, infos, offsets = [], [], [0]
    for i, (w_t, w_prev, ea, eas) in enumerate(tensors):
        b, info = compress_tensor(w_t, w_prev, ea, eas, p, tensor_index=i)
        blobs.append(b)
        infos.append(info)
        offsets.append(offsets[-1] + len(b))
    return b"".join(blobs), offsets, infos


def decompress_checkpoint(blob: bytes, offsets, w_prev_list):
    return [decompress_tensor(blob[offsets[i]:offsets[i + 1]], w_prev_list[i])
            for i in range(len(w_prev_list))]


# --------------------------------------------------------------------------
# The index layout as Sections 3.3 and 4.2 print it: one code per ELEMENT, the
# pruned ones holding the code of the zero centre (0), no bitmap.  This is the
# (I, C) pair that Algorithm 1 hands to its archiver.
# --------------------------------------------------------------------------
DENSE_MAGIC = 0x44435845  # "EXCD", little endian


def dense_section_bytes(numel: int, bits: int) -> int:
    return _align16((numel * bits + 7) // 8)


def dense_bytes(numel: int, bits: int) -> int:
    return header_bytes((1 << bits) - 1) + 3 * dense_section_bytes(numel, bits)


def dense_indices(mask: np.ndarray, codes: np.ndarray) -> np.ndarray:
    """I(i) = code of element i (1..K) where the mask keeps it, 0 (the zero
    centre of Section 4.2) where it is pruned."""
    idx = np.zeros(mask.size, dtype=np.uint8)
    idx[mask] = codes
    return idx


def encode_dense(numel, bits, nnz_w, nnz_o, c_w, c_ea, c_eas, idx_w, idx_ea, idx_eas) -> bytes:
    """The dense container.  The header is the record's with magic "EXCD" and
    the container's size at offset 48; after the centres come the indices of
    dW, of the first moment and of the second, `bits` per element, element i at
    bit i*bits of its section (Section 4.2: two int4 per int8), each section
    padded with zeros to 16 bytes."""
    k = (1 << bits) - 1
    hb = header_bytes(k)
    total = dense_bytes(numel, bits)
    head = struct.pack("<IIQQQIIIIQQ", DENSE_MAGIC, VERSION, numel, nnz_w, nnz_o, bits, k, hb, 0, total, 0)
    head += np.asarray(c_w, dtype="<f4").tobytes()
    head += np.asarray(c_ea, dtype="<f4").tobytes()
    head += np.asarray(c_eas, dtype="<f4").tobytes()
    head += b"\0" * (hb - len(head))
    out = head
    for idx in (idx_w, idx_ea, idx_eas):
        raw = pack_codes(np.asarray(idx, dtype=np.uint8), bits)      # padded for `numel` codes
        out += raw[:dense_section_bytes(numel, bits)]
    assert len(out) == total
    return out


def record_to_dense(blob: bytes) -> bytes:
    """Bitmap + compacted codes -> one code per element (0 = pruned).  Only records of the
    method proper (no record flags) have this layout."""
    r = parse_record(blob)
    if r["rec_flags"]:
        raise ValueError("ablation variants have no dense layout")
    return encode_dense(r["numel"], r["bits"], r["nnz_w"], r["nnz_o"], r["c_w"], r["c_ea"], r["c_eas"],
                        dense_indices(r["m_w"], r["codes_w"]),
                        dense_indices(r["m_o"], r["codes_ea"]),
                        dense_indices(r["m_o"], r["codes_eas"]))


def parse_dense(buf: bytes) -> dict:
    if len(buf) < HEADER_FIXED:
        raise CorruptBlob("short header")
    (magic, version, numel, nnz_w, nnz_o, bits, k, hb, z0, total, z1) = struct.unpack_from(
        "<IIQQQIIIIQQ", buf, 0)
    if magic != DENSE_MAGIC or version != VERSION:
        raise CorruptBlob("magic/version")
    if bits not in (2, 4, 8) or k != (1 << bits) - 1 or hb != header_bytes(k):
        raise CorruptBlob("bits/K/header size")
    if nnz_o > nnz_w or nnz_w > numel:
        raise CorruptBlob("counts")
    if total != dense_bytes(numel, bits) or len(buf) < total:
        raise CorruptBlob("container size")
    cents = np.frombuffer(buf, dtype="<f4", count=3 * k, offset=HEADER_FIXED).reshape(3, k)
    sb = dense_section_bytes(numel, bits)
    idx = [unpack_codes(buf[hb + j * sb:hb + (j + 1) * sb], numel, bits) for j in range(3)]
    if np.count_nonzero(idx[0]) != nnz_w or np.count_nonzero(idx[1]) != nnz_o:
        raise CorruptBlob("population")
    if np.any((idx[1] != 0) != (idx[2] != 0)):
        raise CorruptBlob("the two moments disagree on what is kept")
    if np.any((idx[1] != 0) & (idx[0] == 0)):
        raise CorruptBlob("moment kept where the weight is pruned")
    return dict(numel=numel, nnz_w=nnz_w, nnz_o=nnz_o, bits=bits, k=k, dense_bytes=total,
                c_w=cents[0].copy(), c_ea=cents[1].copy(), c_eas=cents[2].copy(),
                idx_w=idx[0], idx_ea=idx[1], idx_eas=idx[2])


def decompress_dense(buf: bytes, w_prev):
    """Algorithm 2 on the dense layout: every element looks its code up;
    code 0 leaves W^_(t-1) untouched and gives 0 in both moments."""
    r = parse_dense(buf)
    w_prev = np.ascontiguousarray(w_prev, dtype=np.float32).ravel()
    if w_prev.size != r["numel"]:
        raise ValueError("size mismatch")
    w_hat = w_prev.copy()
    kept = r["idx_w"] != 0
    w_hat[kept] = w_prev[kept] + r["c_w"][r["idx_w"][kept].astype(np.int64) - 1]
    ea_hat = np.zeros(r["numel"], dtype=np.float32)
    eas_hat = np.zeros(r["numel"], dtype=np.float32)
    ko = r["idx_ea"] != 0
    ea_hat[ko] = r["c_ea"][r["idx_ea"][ko].astype(np.int64) - 1]
    eas_hat[ko] = r["c_eas"][r["idx_eas"][ko].astype(np.int64) - 1]
    return w_hat, ea_hat, eas_hat


def archive_sizes(parts, preset_extreme: bool = True) -> dict:
    """The archiver step of Algorithm 1 (its last but one line) on the host: LZMA2 as the xz
    container of Python's lzma module, preset 9 (extreme), over the concatenated parts."""
    import lzma
    raw = b"".join(parts)
    preset = 9 | (lzma.PRESET_EXTREME if preset_extreme else 0)
    packed = lzma.compress(raw, format=lzma.FORMAT_XZ, preset=preset)
    if lzma.decompress(packed) != raw:
        raise AssertionError("archiver round trip")
    return dict(raw_bytes=len(raw), archived_bytes=len(packed))


# --------------------------------------------------------------------------
# Brute-force helpers used only by the pins
# --------------------------------------------------------------------------
def brute_mean_abs(x) -> Fraction:
    return sum((Fraction(abs(float(v))) for v in x), Fraction(0)) / len(x)


def brute_nearest(x: float, c) -> int:
    """argmin_j |x - c_j| in exact rational arithmetic, lowest index on ties."""
    best, bj = None, 0
    for j, cj in enumerate(c):
        d = abs(Fraction(float(x)) - Fraction(float(cj)))
        if best is None or d < best:
            best, bj = d, j
    return bj


def optimal_kmeans_1d_sse(values, k: int) -> Fraction:
    """Smallest within-cluster sum of squares over all partitions of the sorted
    values into at most k contiguous groups (dynamic programme, exact)."""
    v = sorted(Fraction(float(x)) for x in values)
    n = len(v)

    def cost(i, j):  # group v[i:j]
        seg = v[i:j]
        mu = sum(seg) / len(seg)
        return sum((t - mu) ** 2 for t in seg)

    dp = [[None] * (n + 1) for _ in range(k + 1)]
    dp[0][0] = Fraction(0)
    for g in range(1, k + 1):
        for j in range(1, n + 1):
            best = dp[g - 1][j] if g > 1 else None  # fewer groups also allowed
            for i in range(g - 1, j):
                if dp[g - 1][i] is None:
                    continue
                cand = dp[g - 1][i] + cost(i, j)
                if best is None or cand < best:
                    best = cand
            dp[g][j] = best
    return dp[k][n]
