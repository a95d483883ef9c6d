// Non-uniform quantisation of the survivors (Section 3.3): Lloyd's algorithm in
// one dimension, K = 2^bits - 1 centres (3, 15 or 255), per tensor and per stream.
//
//   start    K equal-mass quantiles of a seeded, index-stratified sample
//   assign   cluster(x) = #{ j : x > thr_j },  thr_j = largest fp32 not above the
//            fp64 mid-point of centres j and j+1 (so the comparison is exactly
//            "2x > c_j + c_j+1" in fp64)
//   sums     Q(x) = rint(x * 2^(30-E)) in int32, summed as integers, so that the
//            result is independent of the order of summation
//   update   mean = fp32(fp64(sum)/fp64(count) * 2^(E-30)); empty clusters keep
//            their centre; centres re-sorted; new thresholds
//
// The iterations do not sweep the survivors.  The clusters are intervals and the sums
// are integers, so an iteration needs, per threshold, the count and the sum of the
// survivors at or below it.  One sweep files the survivors into 4096 value cells (a
// monotone map, fine where the values are dense) with each cell's count and sum; the
// cells below a threshold then count whole, and only the one cell the threshold falls
// into has to be looked at value by value.  Which cells those will be over all T
// iterations is predicted by running the iterations on the cell table alone (a
// threshold's own cell split by interpolation); a second sweep copies the values of
// the predicted cells and their neighbours, cell after cell, into a gathered copy (a
// seventh of the survivors at 4 bits), and the exact iterations run on that copy, one
// block per tensor and stream.  Should an exact threshold ever leave the gathered
// cells, the stream stops at that iteration; a second round predicts again from there with a
// wider neighbourhood, a third gathers every cell; the centres are those of full sweeps either way.
//
//   kmeans_start    start sample; the cell map
//   cell_count      sweep: count and fixed-point sum of every cell
//   cell_plan       prefixes; predicted thresholds -> selected cells -> their places
//   cell_gather     sweep: values of the selected cells into the gathered copy
//   kmeans_iterate  the exact iterations
#include "excp_common.cuh"
#include <cooperative_groups.h>
#include <cstdio>

namespace excp {

// Cell of a value.  Monotone: x < y implies cell_of(x) <= cell_of(y), which is all the K-means
// iterations need of it.  The value's bit pattern is first turned into a key that orders like the
// values (negative: all bits flipped; non-negative: sign bit set); the key's top nine bits are its
// (sign, exponent) class in value order, and the class's table entry gives its first cell and how far
// the 23 mantissa bits are shifted down to number the class's cells.  Any bit pattern maps inside
// the table.
__device__ __forceinline__ u32 value_key(float x) {
    const u32 bits = __float_as_uint(x);
    return bits ^ ((u32)((int)bits >> 31) | 0x80000000u);
}
__device__ __forceinline__ u32 cell_of(float x, const u32* __restrict__ tab) {
    const u32 key = value_key(x);
    const u32 ent = tab[key >> 23];                    // (first cell << 8) | shift
    return (ent >> 8) + __funnelshift_r(key & 0x7fffffu, 0u, ent);   // the shift is the entry's low five bits
}

__device__ inline u64 mix64(u64 z) {   // SplitMix64 output function
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ float mid_threshold(float a, float b) {
    return __double2float_rd(((double)a + (double)b) * 0.5) + 0.f;   // -0 -> +0
}

// Thresholds of K sorted centres; threads idx, idx + stride, ... of the caller share the work.
__device__ inline void set_thresholds(const float* cent, float* thr, int K, int idx, int stride) {
    for (int j = idx; j < KCAP; j += stride)
        thr[j] = j < K - 1 ? mid_threshold(cent[j], cent[j + 1]) : __uint_as_float(0x7f800000u);
}

constexpr int CELL_SAMPLE = 4096;    // survivors whose classes apportion the cells
constexpr u32 SMALL_STREAM = 16384;  // at most this many survivors: every cell is gathered
constexpr u32 SMALL_STREAM_WIDE = 1u << 20;   // the same with 255 centres: a cluster then has few values per cell, the prediction
                                              // of such a stream fails four times in ten, and its whole copy costs less than the second round

// One block per (tensor, stream).
__global__ void __launch_bounds__(SAMPLE_MAX) kmeans_start_kernel(const TensorDesc* __restrict__ descs,
                                                                  TensorState* __restrict__ st,
                                                                  Workspace ws, KmArrays km, u64 seed, int K, int iters,
                                                                  const CallState* call) {
    __shared__ float smp[SAMPLE_MAX];
    __shared__ u32 chist[NCLASS];                     // sampled survivors per (sign, exponent) class
    __shared__ u32 wtot[NCLASS / 32];
    __shared__ u32 cvalid;
    if (call_aborted(call)) return;
    const int t = blockIdx.x, stream = blockIdx.y, tid = threadIdx.x;
    StreamState& s = st[t].s[stream];
    CellStream& cs = ws.cst[t].s[stream];
    const u32 nnz = stream == 0 ? st[t].nnz_w : st[t].nnz_o;
    const u32 tb = descs[t].tile_begin, ntl = descs[t].num_tiles;
    const u32* toff = (stream == 0 ? ws.tile_off_w : ws.tile_off_o) + tb;
    const u32* tcnt = (stream == 0 ? ws.tile_cnt_w : ws.tile_cnt_o) + tb;
    const float* data = ws.surv[stream] + (u64)tb * TILE;
    if (t == 0 && stream == 0 && tid == 0) *km.pending = 0;
    if (nnz == 0) {                                   // the zeroed state is a valid (one-cell) map
        if (tid < KCAP) { s.cent[tid] = 0.f; s.thr[tid] = __uint_as_float(0x7f800000u); }
        if (tid == 0) { cs.it_done = (u32)iters; cs.active = 0; }
        return;
    }
    const u32 m = min(nnz, (u32)SAMPLE_MAX);
    float v = __uint_as_float(0x7f800000u);           // +inf pads the sort
    if ((u32)tid < m) {
        const u64 lo = ((u64)tid * nnz) / m, hi = ((u64)(tid + 1) * nnz) / m;
        u64 h = mix64(seed + descs[t].tensor_index);
        h = mix64(h + (u64)stream);
        h = mix64(h + (u64)tid);
        const u32 r = (u32)(lo + h % (hi - lo));      // rank of the pick among the survivors
        u32 a = 0, b = ntl - 1;                       // tile whose segment holds rank r
        while (a < b) {
            const u32 mid = (a + b + 1) >> 1;
            if (toff[mid] <= r) a = mid; else b = mid - 1;
        }
        if (EXCP_IN_BOUNDS(call, r - toff[a] < (u32)TILE)) v = data[(u64)a * TILE + (r - toff[a])];
    }
    smp[tid] = v;
    if (tid < NCLASS) chist[tid] = 0;
    if (tid == 0) cvalid = 0;
    __syncthreads();
    // The cell map: a second, larger sample (a survivor of each of 4096 evenly spaced tiles) says how
    // the survivors spread over the (sign, exponent) classes.  Any map that is monotone gives the same
    // centres; this one makes the cells roughly equally full.
#pragma unroll
    for (int r = 0; r < CELL_SAMPLE / SAMPLE_MAX; ++r) {
        const u32 i = (u32)tid + (u32)r * SAMPLE_MAX;
        const u32 tile = (u32)(((u64)i * ntl) / CELL_SAMPLE);
        const u32 c = min(tcnt[tile], (u32)TILE);
        if (c) {
            const float x = data[(u64)tile * TILE + ((i * 2654435761u) >> 8) % c];
            atomicAdd(&chist[__float_as_uint(x) >> 23], 1u);
            atomicAdd(&cvalid, 1u);
        }
    }
    for (int k = 2; k <= SAMPLE_MAX; k <<= 1) {       // bitonic sort, ascending, -0 before +0 (the order of the keys)
        for (int j = k >> 1; j > 0; j >>= 1) {
            const int p = tid ^ j;
            if (p > tid) {
                const float x = smp[tid], y = smp[p];
                const bool up = (tid & k) == 0;
                if ((value_key(x) > value_key(y)) == up) { smp[tid] = y; smp[p] = x; }
            }
            __syncthreads();
        }
    }
    if (tid < KCAP) s.cent[tid] = tid < K ? smp[((2 * tid + 1) * m) / (2 * K)] : 0.f;
    // Cells per class: one each, and the rest in proportion to the class's share of the sample,
    // rounded down to a power of two.  Classes in value order (the order of the value key's top nine
    // bits): negative ones from the largest exponent down (sign-and-exponent fields 511..256), then the
    // positive ones upwards (0..255).
    u32 lg = 0, ncell = 0, incl = 0;
    const int cls = tid < 256 ? 511 - tid : tid - 256;    // class at place `tid` of the value order (tid < 512)
    if (tid < NCLASS) {
        const u32 want = cvalid ? (u32)(((u64)chist[cls] * (NCELL - NCLASS)) / cvalid) : 0u;
        lg = want >= 2 ? 31u - (u32)__clz((int)want) : 0u;
        ncell = 1u << lg;
        incl = ncell;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const u32 x = __shfl_up_sync(0xffffffffu, incl, o);
            if ((tid & 31) >= o) incl += x;
        }
        if ((tid & 31) == 31) wtot[tid >> 5] = incl;
    }
    __syncthreads();
    if (tid < NCLASS) {
        u32 base = 0;
        for (int w = 0; w < (tid >> 5); ++w) base += wtot[w];
        const u32 f = base + incl - ncell;                // first cell of the class
        cs.tab[tid] = (f << 8) | (23u - lg);              // place `tid` of the value order = class of the value key
        if (cls == 0) cs.first_pos = f;
    }
    if (tid == 0) { cs.it_done = 0; cs.active = iters > 0 ? 1u : 0u; }
    __syncthreads();
    set_thresholds(s.cent, s.thr, K, tid, SAMPLE_MAX);
}

// ---------------------------------------------------------------------------
constexpr int KM_GRID_PER_SM = 2;    // blocks per SM of the two K-means sweeps
constexpr int CWARPS = 16;           // warps per block of those sweeps

// A warp's pass over the survivor segments of the tiles [wlo, whi): f8(a, b, two) gets two groups
// of four values (the second only if `two`), f1(x) the up to three last values of a segment, one per
// lane.  The counts of 32 tiles are read at a time, one per lane; up to four 16-byte loads per lane
// are in flight.
template <typename F8, typename F1>
__device__ __forceinline__ void sweep_segments(const float* __restrict__ surv, const u32* __restrict__ tile_cnt,
                                               u32 wlo, u32 whi, int lane, F8&& f8, F1&& f1) {
    for (u32 t0 = wlo; t0 < whi; t0 += 32) {
        const u32 nt32 = min(32u, whi - t0);
        const u32 mycnt = (u32)lane < nt32 ? min(tile_cnt[t0 + lane], (u32)TILE) : 0u;   // a count never leads out of its segment
        for (u32 i = 0; i < nt32; ++i) {
            const u32 cnt = __shfl_sync(0xffffffffu, mycnt, i);
            if (!cnt) continue;
            const float* seg = surv + (u64)(t0 + i) * TILE;
            const float4* seg4 = reinterpret_cast<const float4*>(seg);
            const u32 whole = cnt >> 2;                        // groups of four that exist entirely
            for (u32 f = lane; f < whole; f += 128) {
                float4 v[4];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    v[k] = f + 32u * k < whole ? __ldcs(seg4 + f + 32u * k) : make_float4(0.f, 0.f, 0.f, 0.f);
                f8(v[0], v[1], f + 32u < whole);
                if (f + 64u < whole) f8(v[2], v[3], f + 96u < whole);
            }
            if ((u32)lane < cnt - 4u * whole) f1(seg[4u * whole + lane]);
        }
    }
}

template <int NS>
struct CellCountSmem {
    u32 tab[NS][NCLASS];
    u32 cnt[NS][NCELL];              // the block's counts of the tensor
    u32 lo[NS][NCELL];               // and sums of |Q|: low word,
    u32 hi[NS][NCELL];               //   carries out of it
};

// Sweep 1: survivors per cell and the sum of their |Q| (a cell holds one sign).  A block takes a
// contiguous share of the tiles and goes through it tensor by tensor; its warps split the tensor's
// tiles and add into one table in shared memory, flushed to the tensor's own with integer atomics.
// NS = 1: dW; NS = 2: both moment streams.
template <int NS>
__global__ void __launch_bounds__(CWARPS * 32, 2) cell_count_kernel(const TensorDesc* __restrict__ descs,
                                                                    const TensorState* __restrict__ st, int nt, u32 tiles,
                                                                    Workspace ws, KmArrays km, int stream0, CallState* call) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CellCountSmem<NS>& sm = *reinterpret_cast<CellCountSmem<NS>*>(smem_raw);
    if (call_aborted(call)) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    const u32* tile_cnt = stream0 == 0 ? ws.tile_cnt_w : ws.tile_cnt_o;
#pragma unroll
    for (int k = 0; k < NS; ++k)
        for (int c = tid; c < NCELL; c += CWARPS * 32) {
            sm.cnt[k][c] = 0;
            sm.lo[k][c] = 0; sm.hi[k][c] = 0;
        }
    u32 tile = lo;
    while (tile < hi) {
        const int cur = find_tensor(descs, nt, tile);
        const u32 seg_end = min(hi, descs[cur].tile_begin + descs[cur].num_tiles);
#pragma unroll
        for (int k = 0; k < NS; ++k)
            for (int c = tid; c < NCLASS; c += CWARPS * 32) sm.tab[k][c] = ws.cst[cur].s[stream0 + k].tab[c];
        __syncthreads();
        const u32 n = seg_end - tile;
        const u32 wlo = tile + (u32)(((u64)n * warp) / CWARPS), whi = tile + (u32)(((u64)n * (warp + 1)) / CWARPS);
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            const u32* tab = sm.tab[k];
            u32* cnt = sm.cnt[k];
            u32* slo = sm.lo[k];
            u32* shi = sm.hi[k];
            const float a1 = st[cur].s[stream0 + k].scale1, a2 = st[cur].s[stream0 + k].scale2;
            auto tally = [&](float x) {
                const u32 c = cell_of(x, tab);
                if (!EXCP_IN_BOUNDS(call, c < (u32)NCELL)) return;
                const u32 q = (u32)abs(__float2int_rn(__fmul_rn(__fmul_rn(x, a1), a2)));   // |Q(x)| < 2^31
                atomicAdd(&cnt[c], 1u);
                const u32 old = atomicAdd(&slo[c], q);
                if (old + q < old) atomicAdd(&shi[c], 1u);
            };
            auto tally8 = [&](const float4& va, const float4& vb, bool two) {      // all table look-ups first
                const float xs[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                u32 c[8], q[8], old[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    c[i] = cell_of(xs[i], tab);
                    if (!EXCP_IN_BOUNDS(call, c[i] < (u32)NCELL)) c[i] = 0;
                    q[i] = (u32)abs(__float2int_rn(__fmul_rn(__fmul_rn(xs[i], a1), a2)));
                }
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (i < 4 || two) atomicAdd(&cnt[c[i]], 1u);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (i < 4 || two) old[i] = atomicAdd(&slo[c[i]], q[i]);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if ((i < 4 || two) && old[i] + q[i] < old[i]) atomicAdd(&shi[c[i]], 1u);
            };
            sweep_segments(ws.surv[stream0 + k], tile_cnt, wlo, whi, lane, tally8, tally);
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            CellStream& cs = ws.cst[cur].s[stream0 + k];
            u32* row = km.rows[stream0 + k] + (u64)(blockIdx.x + cur) * NCELL;    // this block's share of the tensor
            for (int c = tid; c < NCELL; c += CWARPS * 32) {
                const u32 n_c = sm.cnt[k][c];
                row[c] = n_c;
                if (n_c) {
                    atomicAdd(&cs.cnt[c], n_c);
                    const u64 mag = ((u64)sm.hi[k][c] << 32) | sm.lo[k][c];
                    sm.lo[k][c] = 0; sm.hi[k][c] = 0;
                    if (mag) atomicAdd(&cs.mag[c], mag);
                    sm.cnt[k][c] = 0;
                }
            }
        }
        __syncthreads();
        tile = seg_end;
    }
}

// ---------------------------------------------------------------------------
// Exclusive prefix over 4 x 1024 items, four consecutive ones per thread; the total to every thread.
// wt: 32 words of shared memory.  Whole block of 1024 threads.
template <typename T>
__device__ inline T block_scan4(T (&v)[4], T* wt) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T mine = v[0] + v[1] + v[2] + v[3];
    T incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const T x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    __syncthreads();                  // wt may still be read from the previous scan
    if (lane == 31) wt[warp] = incl;
    __syncthreads();
    T base = 0, total = 0;
    for (int w = 0; w < 32; ++w) {
        if (w < warp) base += wt[w];
        total += wt[w];
    }
    T run = base + incl - mine;
#pragma unroll
    for (int k = 0; k < 4; ++k) { const T x = v[k]; v[k] = run; run += x; }
    return total;
}

constexpr int PLAN_THREADS = 1024;

// Block of a grid of g blocks whose share [tiles * b / g, tiles * (b + 1) / g) holds tile x (see block_range).
__device__ inline u32 block_of_tile(u32 x, u32 tiles, u32 g) {
    u32 b = (u32)(((u64)x * g) / tiles);
    while ((u32)(((u64)tiles * (b + 1)) / g) <= x) ++b;
    return b;
}

// Prefixes of the cell table; the cells the coming iterations will need; their places in the
// gathered copy.  One block per (tensor, stream).  Round 0 predicts; the later rounds are only for
// streams that met a cell they had not gathered: one more prediction, then every cell.
constexpr int KM_ROUNDS = 3;
__global__ void __launch_bounds__(PLAN_THREADS) cell_plan_kernel(const TensorDesc* __restrict__ descs,
                                                                 TensorState* __restrict__ st, Workspace ws, KmArrays km, int K,
                                                                 int iters, int margin, int w16, int round, u32 tiles,
                                                                 u32 grid, const CallState* call) {
    __shared__ u32 tab[NCLASS];
    __shared__ u32 selw[NCELL / 32];
    __shared__ float cent[KCAP], thr[KCAP], cnew[KCAP];
    __shared__ double Lp[KCAP], Sp[KCAP];
    __shared__ s64 wt64[32];
    __shared__ u32 wt32[32];
    __shared__ u32 smax;
    if (call_aborted(call)) return;
    const int t = blockIdx.x, stream = blockIdx.y, tid = threadIdx.x;
    CellStream& cs = ws.cst[t].s[stream];
    if (!cs.active) return;
    const StreamState& s = st[t].s[stream];
    const u32 nnz = stream == 0 ? st[t].nnz_w : st[t].nnz_o;
    const bool gridded = w16 && stream == 0;           // dW of weights stored in 16 bits
    const u32 c0 = 4u * tid;                           // this thread's cells
    u32 cnt[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) cnt[k] = cs.cnt[c0 + k];
    if (tid < NCELL / 32) selw[tid] = 0xffffffffu;
    if (tid == 0) smax = 0;
    __syncthreads();
    atomicMax(&smax, max(max(cnt[0], cnt[1]), max(cnt[2], cnt[3])));
    __syncthreads();
    // Where single cells hold far more than their share (values on a coarse grid, as with weights stored in 16
    // bits), the iterations on the cell table drift further from the exact ones: a wider neighbourhood is copied.
    if (margin >= 0 && (u64)smax * NCELL > 16ull * nnz) margin = max(margin, 8);
    // A stream whose first round met a cell it had not copied predicts again from where it stopped (its centres
    // are exact up to there), with a wider neighbourhood; the last round takes every cell.
    // (With 255 centres a cluster is about 16 cells wide and eight cells either side would be every cell already:
    // there the second round widens to two.)
    if (round > 0 && margin >= 0) margin = K > 15 ? max(2 * margin, 2) : max(8 * margin, 8);
    u32 tc = 0;
    s64 ts = 0;
    if (round == 0) {
        const u32 first_pos = cs.first_pos;
        u32 pc[4];
        s64 ps[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            pc[k] = cnt[k];
            const s64 mag = (s64)cs.mag[c0 + k];
            ps[k] = c0 + k < first_pos ? -mag : mag;
        }
        tc = block_scan4(pc, wt32);
        ts = block_scan4(ps, wt64);
#pragma unroll
        for (int k = 0; k < 4; ++k) { cs.cntpre[c0 + k] = pc[k]; cs.sumpre[c0 + k] = ps[k]; }
        if (tid == 0) { cs.cntpre[NCELL] = tc; cs.sumpre[NCELL] = ts; }
    } else {
        tc = cs.cntpre[NCELL];
        ts = cs.sumpre[NCELL];
    }
    if (round < KM_ROUNDS - 1) {
        const bool predict = nnz > (K > 15 ? SMALL_STREAM_WIDE : SMALL_STREAM) && margin < NCELL;
        if (predict) {
            if (tid < NCELL / 32) selw[tid] = 0;
            if (tid < NCLASS) tab[tid] = cs.tab[tid];
            if (tid < KCAP) { cent[tid] = s.cent[tid]; thr[tid] = s.thr[tid]; }
        }
        __syncthreads();                               // also: this block's prefixes are visible to it
        if (predict && margin >= 0) {
            const double scale = __longlong_as_double((s64)(s.e - 30 + 1023) << 52);
            for (int it = (int)cs.it_done; it < iters; ++it) {
                if (tid < K - 1) {
                    const float tj = thr[tid];
                    const u32 c = cell_of(tj, tab);
                    for (int d = -margin; d <= margin; ++d) {
                        const int cc = (int)c + d;
                        if (cc >= 0 && cc < NCELL) atomicOr(&selw[cc >> 5], 1u << (cc & 31));
                    }
                    // the share of cell c at or below the threshold, by its place between the cell's edges
                    const u32 bits = __float_as_uint(tj), sh = tab[value_key(tj) >> 23] & 31u;
                    const u32 a_lo = (bits & 0x7fffffffu) >> sh << sh;
                    const u32 a_hi = min(a_lo + (1u << sh), 0x7f7fffffu);
                    const double v_lo = (double)__uint_as_float(a_lo), v_hi = (double)__uint_as_float(a_hi);
                    const double n_c = (double)(cs.cntpre[c + 1] - cs.cntpre[c]);
                    const double s_c = (double)(cs.sumpre[c + 1] - cs.sumpre[c]);
                    // The cell's values are taken as spread evenly over the widest interval inside the cell
                    // that is centred on their mean: the whole cell when the mean is its middle, a point when
                    // the mean sits on an edge.
                    double f = 1.0;
                    if (n_c > 0.0) {
                        const double mean = fmin(fmax(fabs(s_c / n_c * scale), v_lo), v_hi);
                        const double half = fmin(mean - v_lo, v_hi - mean);
                        const double x = fabs((double)tj);
                        if (gridded && mean - v_lo <= v_hi - mean && v_hi > v_lo) {
                            // Values known to lie on a grid (residuals of 16-bit weights): grid points are cell edges, so
                            // the cell is taken as a point mass on its lower edge plus an even spread, with the cell's mean.
                            // f is the share of magnitudes at or below x above zero, strictly below x under it.
                            const double w = v_hi - v_lo, pm = 1.0 - 2.0 * (mean - v_lo) / w;
                            f = (!(bits >> 31) || x > v_lo ? pm : 0.0) + (1.0 - pm) * (x - v_lo) / w;
                        } else
                        f = half > 0.0 ? (x - (mean - half)) / (2.0 * half) : (x >= mean ? 1.0 : 0.0);
                        f = fmin(fmax(f, 0.0), 1.0);
                        // A threshold exactly on the cell's lower edge (the first thresholds are mid-points of sampled values,
                        // and values on a grid, such as residuals of 16-bit weights, sit on cell edges): the values equal to it
                        // count as at or below it.  If the cell is a point mass on that edge plus an even spread, its mean
                        // says how much the point holds.  (Below zero the equal values count already: 1 - f.)
                        if (!(bits >> 31) && x == v_lo && v_hi > v_lo) f = fmax(f, fmax(0.0, 1.0 - 2.0 * (mean - v_lo) / (v_hi - v_lo)));
                    }
                    if (bits >> 31) f = 1.0 - f;
                    Lp[tid] = (double)cs.cntpre[c] + f * n_c;
                    Sp[tid] = (double)cs.sumpre[c] + f * s_c;
                } else if (tid == K - 1) {
                    Lp[tid] = (double)tc;
                    Sp[tid] = (double)ts;
                }
                __syncthreads();
                float c = __uint_as_float(0x7f800000u);
                if (tid < K) {
                    const double n = tid == 0 ? Lp[0] : Lp[tid] - Lp[tid - 1];
                    const double sum = tid == 0 ? Sp[0] : Sp[tid] - Sp[tid - 1];
                    c = n >= 0.5 ? __double2float_rn(sum / n * scale) : cent[tid];
                    cnew[tid] = c;
                }
                __syncthreads();
                if (tid < K) {
                    int rank = 0;
                    for (int i = 0; i < K; ++i) {
                        const float o = cnew[i];
                        rank += (o < c) || (o == c && i < tid);
                    }
                    cent[rank] = c;
                }
                __syncthreads();
                set_thresholds(cent, thr, K, tid, PLAN_THREADS);
                __syncthreads();
            }
        }
    }
    __syncthreads();
    // places of the selected cells in the gathered copy; the gather cursors start at zero
    u32 g[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) g[k] = ((selw[(c0 + k) >> 5] >> ((c0 + k) & 31)) & 1u) ? cnt[k] : 0u;
    block_scan4(g, wt32);
#pragma unroll
    for (int k = 0; k < 4; ++k) cs.mag[c0 + k] = (u64)g[k];
    if (tid < NCELL / 32) cs.sel[tid] = selw[tid];
    // Where every block of the sweeps puts its values of a cell: the blocks that share the tensor,
    // in order, each after the ones before it (the counting sweep left their counts in km_rows).
    const u32 tb = descs[t].tile_begin, tl = tb + descs[t].num_tiles - 1;
    const u32 b0 = block_of_tile(tb, tiles, grid), b1 = block_of_tile(tl, tiles, grid);
    const u32* rows = km.rows[stream];
    u32* pos = km.pos[stream];
    for (u32 b = b0; b <= b1; ++b) {
        const u64 r = (u64)(b + (u32)t) * NCELL + c0;
        const uint4 n = *reinterpret_cast<const uint4*>(rows + r);
        *reinterpret_cast<uint4*>(pos + r) = make_uint4(g[0], g[1], g[2], g[3]);
        g[0] += n.x; g[1] += n.y; g[2] += n.z; g[3] += n.w;
    }
}

// ---------------------------------------------------------------------------
template <int NS>
struct CellGatherSmem {
    u32 tab[NS][NCLASS];
    u32 cur[NS][NCELL];              // where the block's next value of each selected cell goes; NOT_TAKEN for the others
};
constexpr u32 NOT_TAKEN = 0xffffffffu;

// Sweep 2: the values of the selected cells into the gathered copy, every cell contiguous (the
// order inside a cell is arbitrary: what is taken from it are integer sums).  Same grid and same
// shares of the tiles as the counting sweep, so every block owns a reserved run inside every cell
// (km.pos) and no two blocks ever contend for a place.  A tensor with nothing to gather is skipped.
template <int NS>
__global__ void __launch_bounds__(CWARPS * 32, 2) cell_gather_kernel(const TensorDesc* __restrict__ descs, int nt, u32 tiles,
                                                                     Workspace ws, KmArrays km, int stream0, CallState* call,
                                                                     int round) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CellGatherSmem<NS>& sm = *reinterpret_cast<CellGatherSmem<NS>*>(smem_raw);
    if (call_aborted(call)) return;
    if (round > 0 && *km.pending == 0) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    const u32* tile_cnt = stream0 == 0 ? ws.tile_cnt_w : ws.tile_cnt_o;
    u32 tile = lo;
    while (tile < hi) {
        const int cur = find_tensor(descs, nt, tile);
        const u32 tb = descs[cur].tile_begin;
        const u32 seg_end = min(hi, tb + descs[cur].num_tiles);
        bool act[NS];
        bool any = false;
#pragma unroll
        for (int k = 0; k < NS; ++k) { act[k] = ws.cst[cur].s[stream0 + k].active != 0; any |= act[k]; }
        if (!any) { tile = seg_end; continue; }           // the same for the whole block
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            const CellStream& cs = ws.cst[cur].s[stream0 + k];
            const u32* pos = km.pos[stream0 + k] + (u64)(blockIdx.x + cur) * NCELL;
            for (int c = tid; c < NCLASS; c += CWARPS * 32) sm.tab[k][c] = cs.tab[c];
            for (int c = tid; c < NCELL; c += CWARPS * 32)
                sm.cur[k][c] = ((cs.sel[c >> 5] >> (c & 31)) & 1u) ? pos[c] : NOT_TAKEN;
        }
        __syncthreads();
        const u32 n = seg_end - tile;
        const u32 wlo = tile + (u32)(((u64)n * warp) / CWARPS), whi = tile + (u32)(((u64)n * (warp + 1)) / CWARPS);
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            if (!act[k]) continue;
            const u32* tab = sm.tab[k];
            u32* cursor = sm.cur[k];
            float* out = ws.bkt[stream0 + k] + (u64)tb * TILE;
            const u64 room = (u64)descs[cur].num_tiles * TILE;               // the tensor's share of the gathered copy
            auto put = [&](u32 c, float x) {
                const u32 at = atomicAdd(&cursor[c], 1u);
                if (EXCP_IN_BOUNDS(call, at < room)) out[at] = x;
            };
            auto file = [&](float x) {
                const u32 c = cell_of(x, tab);
                if (!EXCP_IN_BOUNDS(call, c < (u32)NCELL)) return;
                if (cursor[c] != NOT_TAKEN) put(c, x);
            };
            auto file8 = [&](const float4& va, const float4& vb, bool two) {       // all look-ups first
                const float xs[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                u32 c[8];
                u32 hit = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    c[i] = cell_of(xs[i], tab);
                    if (!EXCP_IN_BOUNDS(call, c[i] < (u32)NCELL)) c[i] = 0;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) hit |= (cursor[c[i]] != NOT_TAKEN ? 1u : 0u) << i;
                if (!two) hit &= 15u;
                if (hit) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if ((hit >> i) & 1u) put(c[i], xs[i]);
                }
            };
            sweep_segments(ws.surv[stream0 + k], tile_cnt, wlo, whi, lane, file8, file);
        }
        __syncthreads();
        tile = seg_end;
    }
}

// ---------------------------------------------------------------------------
constexpr int IT_THREADS = 1024;
constexpr int IT_WARPS = IT_THREADS / 32;
constexpr int IT_PARTS = 4;          // at most this many warps of a block share one threshold's cell
constexpr int IT_CLUSTER = 4;        // blocks (one thread-block cluster) that share a large stream's iterations at wide codes
constexpr u32 IT_LARGE = 2u << 20;   // survivors from which a stream counts as large (measured: 4 x 2 M best of 2..8 x 1..24 M)

// Count and fixed-point sum of the values of data[a, e) at or below thr; whole warp.
__device__ __forceinline__ void scan_range(const float* __restrict__ data, u32 a, u32 e, float thr, float s1,
                                           float s2, int lane, u32& cnt, s64& sum) {
    auto test = [&](float x) {
        if (!(x > thr)) {
            ++cnt;
            sum += __float2int_rn(__fmul_rn(__fmul_rn(x, s1), s2));
        }
    };
    const u32 h = min(e, (a + 3u) & ~3u);                    // up to three values before a 16-byte boundary
    if (a + lane < h) test(__ldg(data + a + lane));
    const u32 be = h + ((e - h) & ~3u);
    constexpr int INFL = 8;                                  // 16-byte loads in flight per lane
    for (u32 i = h + 4u * lane; i < be; i += 128u * INFL) {
        float4 v[INFL];
#pragma unroll
        for (int k = 0; k < INFL; ++k)
            if (i + 128u * k < be) v[k] = __ldg(reinterpret_cast<const float4*>(data + i + 128u * k));
#pragma unroll
        for (int k = 0; k < INFL; ++k)
            if (i + 128u * k < be) { test(v[k].x); test(v[k].y); test(v[k].z); test(v[k].w); }
    }
    if (be + lane < e) test(__ldg(data + be + lane));
}

// The exact iterations of one stream, from iteration it_done on: one block, or one thread-block
// cluster, per (tensor, stream); streams whose number of survivors is outside [nnz_lo, nnz_hi) are
// left to another launch.  L_j = survivors at or below threshold j = the cells below its cell,
// whole, + the part of its own cell found by looking at the gathered values; cluster k has
// L_k - L_(k-1) members (L_-1 = 0, L_(K-1) = all), and its sum likewise.  If a threshold's cell has
// values and was not gathered, the stream stops here, stays active and is counted in km_pending.
// Launched as clusters, the blocks split every threshold's cell between them (with 255 centres a large
// tensor's ten iterations read hundreds of MB, and one block's load bandwidth would set the time of the
// launch), leave their counts and integer sums in their own shared memory, and after the cluster's
// barrier every block reads all of them through distributed shared memory and computes the same new
// centres, so nothing is sent back.  The shares are double-buffered: one barrier per iteration.
// Every block of a cluster takes the same way through the kernel (what decides it: the call's time-out
// flag, which no K-means kernel sets; the stream's state, which only block 0 writes, after the last
// barrier; thresholds that are the same in every block), so every barrier is reached by all of them
// and none leaves while another may still read its shared memory.
// CL: launched as clusters (otherwise the kernel is the plain one-block form: a block barrier, one buffer).
template <bool CL>
__global__ void __launch_bounds__(IT_THREADS) kmeans_iterate_kernel(const TensorDesc* __restrict__ descs,
                                                                    TensorState* __restrict__ st, Workspace ws, KmArrays km, int K,
                                                                    int iters, const CallState* call, u32 nnz_lo, u32 nnz_hi) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ u32 tab[NCLASS];
    __shared__ u32 selw[NCELL / 32];
    __shared__ float cent[KCAP], thr[KCAP], cnew[KCAP];
    __shared__ u32 cellj[KCAP];
    __shared__ u32 pcnt[CL ? 2 : 1][KCAP][IT_PARTS];
    __shared__ s64 psum[CL ? 2 : 1][KCAP][IT_PARTS];
    __shared__ u64 Ls[KCAP];
    __shared__ s64 Ss[KCAP];
    if (call_aborted(call)) return;
    const u32 crank = CL ? cluster.block_rank() : 0u, csize = CL ? cluster.num_blocks() : 1u;
    const u32 unit = blockIdx.x / csize;                 // a cluster's blocks are neighbours in x
    const u32 nt = gridDim.x / (3u * csize);             // all dW streams first: they are the long ones
    const int t = (int)(unit % nt), stream = (int)(unit / nt), tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    CellStream& cs = ws.cst[t].s[stream];
    if (!cs.active) return;
    {
        const u64 nnz = stream == 0 ? st[t].nnz_w : st[t].nnz_o;
        if (nnz < nnz_lo || nnz >= nnz_hi) return;
    }
    StreamState& s = st[t].s[stream];
    if (tid < NCLASS) tab[tid] = cs.tab[tid];
    if (tid < NCELL / 32) selw[tid] = cs.sel[tid];
    if (tid < KCAP) { cent[tid] = s.cent[tid]; thr[tid] = s.thr[tid]; }
    const float s1 = s.scale1, s2 = s.scale2;
    const double scale = __longlong_as_double((s64)(s.e - 30 + 1023) << 52);
    const float* data = ws.bkt[stream] + (u64)descs[t].tile_begin * TILE;
    const int parts = max(1, min(IT_PARTS, IT_WARPS / max(K - 1, 1)));
    __syncthreads();
    int it = (int)cs.it_done;
    const u32 allparts = (u32)parts * csize;             // shares of a threshold's cell over the whole cluster
    int buf = 0;
    for (; it < iters; ++it, buf ^= CL ? 1 : 0) {
        bool ok = true;
        if (tid < K - 1) {
            const u32 c = cell_of(thr[tid], tab);
            cellj[tid] = c;
            ok = ((selw[c >> 5] >> (c & 31)) & 1u) || cs.cntpre[c + 1] == cs.cntpre[c];
        }
        if (__syncthreads_or(!ok)) break;
        for (int item = warp; item < (K - 1) * parts; item += IT_WARPS) {
            const int j = item / parts, p = item - j * parts;
            const u32 c = cellj[j];
            u32 cnt = 0;
            s64 sum = 0;
            if ((selw[c >> 5] >> (c & 31)) & 1u) {
                const u32 b = (u32)cs.mag[c], n = cs.cntpre[c + 1] - cs.cntpre[c];
                const u32 gp = crank * (u32)parts + (u32)p;              // this warp's share among the cluster's
                if (EXCP_IN_BOUNDS(call, (u64)b + n <= (u64)descs[t].num_tiles * TILE))
                scan_range(data, b + (u32)(((u64)n * gp) / allparts), b + (u32)(((u64)n * (gp + 1)) / allparts), thr[j], s1, s2,
                           lane, cnt, sum);
            }
            cnt = __reduce_add_sync(0xffffffffu, cnt);
#pragma unroll
            for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) { pcnt[buf][j][p] = cnt; psum[buf][j][p] = sum; }
        }
        if (CL) cluster.sync();                          // every block's shares are in its shared memory
        else __syncthreads();
        u64 L = 0;
        s64 S = 0;
        if (tid < K - 1) {
            const u32 c = cellj[tid];
            L = cs.cntpre[c];
            S = cs.sumpre[c];
            if (CL) {
                for (u32 r = 0; r < csize; ++r) {
                    const u32* rc = cluster.map_shared_rank(&pcnt[buf][tid][0], r);
                    const s64* rs = cluster.map_shared_rank(&psum[buf][tid][0], r);
                    for (int p = 0; p < parts; ++p) { L += rc[p]; S += rs[p]; }
                }
            } else {
                for (int p = 0; p < parts; ++p) { L += pcnt[0][tid][p]; S += psum[0][tid][p]; }
            }
        } else if (tid == K - 1) {
            L = cs.cntpre[NCELL];
            S = cs.sumpre[NCELL];
        }
        if (tid < KCAP) { Ls[tid] = L; Ss[tid] = S; }
        __syncthreads();
        float c = __uint_as_float(0x7f800000u);
        if (tid < K) {
            const u64 n = tid == 0 ? L : L - Ls[tid - 1];
            const s64 sum = tid == 0 ? S : S - Ss[tid - 1];
            c = cent[tid];
            if (n) c = __double2float_rn(__ll2double_rn(sum) / __ull2double_rn(n) * scale);
            cnew[tid] = c;
        }
        __syncthreads();
        if (tid < K) {                    // sort ascending, -0 before +0: rank of each centre among the K (equal bits by index)
            int rank = 0;
            const u32 kc = value_key(c);
            for (int i = 0; i < K; ++i) {
                const u32 ko = value_key(cnew[i]);
                rank += (ko < kc) || (ko == kc && i < tid);
            }
            cent[rank] = c;
        }
        __syncthreads();
        set_thresholds(cent, thr, K, tid, IT_THREADS);
        __syncthreads();
    }
    if (CL) {
        cluster.sync();                                  // nobody still reads this block's shares
        if (crank != 0) return;
    }
    if (tid < KCAP) { s.cent[tid] = cent[tid]; s.thr[tid] = thr[tid]; }
    if (tid == 0) {
        cs.it_done = (u32)it;
        if (it == iters) cs.active = 0;
        else atomicAdd(km.pending, 1u);
#ifdef EXCP_TRACE_KMEANS
        if (it != iters) printf("kmeans miss: tensor %d stream %d numel %llu stopped at iteration %d\n", t, stream, descs[t].numel, it);
#endif
    }
}

// With up to 15 centres: one block per (tensor, stream).  With more, the large streams go to a second
// launch as clusters of IT_CLUSTER blocks, side by side in x (a block of either launch whose stream
// belongs to the other returns at once).
static void launch_iterate(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, const Workspace& ws,
                           const KmArrays& km, int K, int iters, const CallState* call) {
    const bool split = K > 15;
    kmeans_iterate_kernel<false><<<(unsigned)nt * 3u, IT_THREADS, 0, cfg.stream>>>(descs, st, ws, km, K, iters, call, 0u,
                                                                           split ? IT_LARGE : 0xffffffffu);
    if (!split) return;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)nt * 3u * (unsigned)IT_CLUSTER, 1, 1);
    lc.blockDim = dim3(IT_THREADS, 1, 1);
    lc.dynamicSmemBytes = 0;
    lc.stream = cfg.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = IT_CLUSTER;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    cudaLaunchKernelEx(&lc, kmeans_iterate_kernel<true>, descs, st, ws, km, K, iters, call, (u32)IT_LARGE, 0xffffffffu);
}

void launch_kmeans(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                   const Workspace& ws, const KmArrays& km, const Params& p, CallState* call) {
    const int K = centres_of(p.bits);
    kmeans_start_kernel<<<dim3(nt, 3), SAMPLE_MAX, 0, cfg.stream>>>(descs, st, ws, km, p.seed, K, p.kmeans_iters, call);
    prof_mark(cfg, ST_KMEANS_START, 1);
    if (!tiles || p.kmeans_iters == 0) return;
    // the two sweeps use one grid: a block's share of the tiles is its share of every cell
    const u32 grid = min(tiles, min((u32)KM_GRID_PER_SM * (u32)cfg.sms, (u32)KM_MAX_GRID));
    {
        const size_t m1 = sizeof(CellCountSmem<1>), m2 = sizeof(CellCountSmem<2>);
        cudaFuncSetAttribute(cell_count_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m1);
        cudaFuncSetAttribute(cell_count_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m2);
        cell_count_kernel<1><<<grid, CWARPS * 32, m1, cfg.stream>>>(descs, st, nt, tiles, ws, km, 0, call);
        cell_count_kernel<2><<<grid, CWARPS * 32, m2, cfg.stream>>>(descs, st, nt, tiles, ws, km, 1, call);
        prof_mark(cfg, ST_CELL_COUNT, 2);
    }
    const size_t g1 = sizeof(CellGatherSmem<1>), g2 = sizeof(CellGatherSmem<2>);
    cudaFuncSetAttribute(cell_gather_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g1);
    cudaFuncSetAttribute(cell_gather_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g2);
    for (int round = 0; round < KM_ROUNDS; ++round) {
        cell_plan_kernel<<<dim3(nt, 3), PLAN_THREADS, 0, cfg.stream>>>(descs, st, ws, km, K, p.kmeans_iters, p.km_margin, p.wfmt != WF_F32, round,
                                                                     tiles, grid, call);
        if (round == 0) prof_mark(cfg, ST_CELL_PLAN, 1);
        cell_gather_kernel<1><<<grid, CWARPS * 32, g1, cfg.stream>>>(descs, nt, tiles, ws, km, 0, call, round);
        cell_gather_kernel<2><<<grid, CWARPS * 32, g2, cfg.stream>>>(descs, nt, tiles, ws, km, 1, call, round);
        if (round == 0) prof_mark(cfg, ST_CELL_GATHER, 2);
        launch_iterate(cfg, descs, st, nt, ws, km, K, p.kmeans_iters, call);
        prof_mark(cfg, round == 0 ? ST_KMEANS_ITERATE : ST_KMEANS_RETRY, (round == 0 ? 0 : 3) + (K > 15 ? 2 : 1));   // launches since the last mark
    }
}

}  // namespace excp
