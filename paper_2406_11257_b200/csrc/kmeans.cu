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
// The iterations do not sweep the survivors.  Because the clusters are intervals
// and the sums are integers, the survivors are first grouped ONCE into 256 value
// buckets (a cheap monotone function of the value, scaled to the range of the
// start sample) with each bucket's count and sum.  An iteration then
// needs, per threshold, only the bucket the threshold falls into: buckets below
// it count whole, and the one bucket is scanned.  That is a small part of the
// data per iteration, and the sums are exactly those of a full sweep.
//
//   bucket_count    sweep: survivors per bucket and every bucket's fixed-point sum
//   bucket_offsets  prefix of the counts -> where each bucket starts
//   bucket_scatter  sweep: survivors into their buckets
//   bucket_prefix   prefix of the sums; first plan
//   per iteration:  bucket_scan (the K - 1 threshold buckets), bucket_update
#include "excp_common.cuh"
#include "seg_ring.cuh"

namespace excp {

__device__ inline u64 mix64(u64 z) {   // SplitMix64 output function
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Thresholds of K sorted, final centres; threads idx, idx + stride, ... of the caller share the work.
__device__ inline void set_thresholds(StreamState& s, int K, int idx, int stride) {
    for (int j = idx; j < KCAP; j += stride) {
        float t = __uint_as_float(0x7f800000u);
        if (j < K - 1)
            t = __double2float_rd(((double)s.cent[j] + (double)s.cent[j + 1]) * 0.5) + 0.f;   // -0 -> +0
        s.thr[j] = t;
    }
}

// One block per (tensor, stream).
__global__ void __launch_bounds__(SAMPLE_MAX) kmeans_start_kernel(const TensorDesc* __restrict__ descs,
                                                                  TensorState* __restrict__ st,
                                                                  Workspace ws, u64 seed, int K) {
    __shared__ float smp[SAMPLE_MAX];
    __shared__ u32 amin, amax;                        // smallest / largest magnitude pattern in the sample
    const int t = blockIdx.x, stream = blockIdx.y, tid = threadIdx.x;
    StreamState& s = st[t].s[stream];
    const u32 nnz = stream == 0 ? st[t].nnz_w : st[t].nnz_o;
    const u32 tb = descs[t].tile_begin, ntl = descs[t].num_tiles;
    const u32* toff = (stream == 0 ? ws.tile_off_w : ws.tile_off_o) + tb;
    const float* data = ws.surv[stream] + (u64)tb * TILE;
    BucketStream& bk = ws.bst[t].s[stream];
    if (nnz == 0) {
        if (tid < KCAP) { s.cent[tid] = 0.f; s.thr[tid] = __uint_as_float(0x7f800000u); }
        if (tid == 0) { bk.fn.lo = 0; bk.fn.shift = 0; bk.fn.sgn = stream != 2; }
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
        v = data[(u64)a * TILE + (r - toff[a])];
    }
    smp[tid] = v;
    if (tid == 0) { amin = 0x7fffffffu; amax = 0u; }
    __syncthreads();
    if ((u32)tid < m) {
        atomicMin(&amin, __float_as_uint(v) & 0x7fffffffu);
        atomicMax(&amax, __float_as_uint(v) & 0x7fffffffu);
    }
    for (int k = 2; k <= SAMPLE_MAX; k <<= 1) {       // bitonic sort, ascending
        for (int j = k >> 1; j > 0; j >>= 1) {
            const int p = tid ^ j;
            if (p > tid) {
                const float x = smp[tid], y = smp[p];
                const bool up = (tid & k) == 0;
                if ((x > y) == up) { smp[tid] = y; smp[p] = x; }
            }
            __syncthreads();
        }
    }
    if (tid < KCAP) s.cent[tid] = tid < K ? smp[((2 * tid + 1) * m) / (2 * K)] : 0.f;
    // bucket function: its steps span the magnitudes seen in the sample (any monotone map
    // would give the same centres; this one spreads these survivors over the 256 buckets)
    if (tid == 0) {
        const u32 d = amax - amin;
        const int half_bits = stream != 2 ? 7 : 8;            // log2 of the steps per sign
        const int len = 32 - __clz(d);                        // d < 2^len
        bk.fn.lo = amin; bk.fn.shift = len > half_bits ? len - half_bits : 0; bk.fn.sgn = stream != 2;
    }
    __syncthreads();
    set_thresholds(s, K, tid, SAMPLE_MAX);
}


// ---------------------------------------------------------------------------
constexpr int BWARPS = TPB / 32;
constexpr int BST = 2;               // stages per warp

template <int NS, int CH>
struct BucketCountSmem {
    float buf[BWARPS][BST][NS][CH];
    unsigned long long bar[BWARPS][BST];
    u32 hist[BWARPS][NS][NBKT];      // each warp's counts since its last flush
    u32 slo[BWARPS][NS][NBKT];       // and fixed-point sums, as sums of the low 16 bits
    u32 shi[BWARPS][NS][NBKT];       //   and of the (signed) high 16 bits of every value's Q
};
constexpr u32 COUNT_FLUSH_CHUNKS = 32768 / 512;   // at most 32768 values per warp between flushes: the 16-bit sums fit

// Sweep 1 of the grouping: survivors per bucket and their fixed-point sums.  NS = 1: dW; NS = 2:
// both moment streams.
template <int NS, int CH>
__global__ void __launch_bounds__(TPB) bucket_count_kernel(const TensorDesc* __restrict__ descs,
                                                           const TensorState* __restrict__ st, int nt, u32 tiles,
                                                           Workspace ws, int stream0, CallState* call) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    BucketCountSmem<NS, CH>& sm = *reinterpret_cast<BucketCountSmem<NS, CH>*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u32 gw = blockIdx.x * BWARPS + warp, nw = gridDim.x * BWARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    SegRing<NS, CH, BST> ring;
    ring.init(&sm.buf[warp][0][0][0], sm.bar[warp], lane, wlo, whi);
    const u32* tile_cnt = stream0 == 0 ? ws.tile_cnt_w : ws.tile_cnt_o;
    const float* surv[NS];
    BucketFn fn[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) {
        surv[k] = ws.surv[stream0 + k];
        fn[k] = BucketFn{0, 0, 0, 0};
        for (int b = lane; b < NBKT; b += 32) { sm.hist[warp][k][b] = 0; sm.slo[warp][k][b] = 0; sm.shi[warp][k][b] = 0; }
    }
    __syncwarp();
    int cur = -1;
    u32 tb = 0, ntl = 0, since = 0;
    float s1[NS], s2[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) { s1[k] = 0.f; s2[k] = 0.f; }

    auto flush = [&](int tns) {
        __syncwarp();
#pragma unroll
        for (int k = 0; k < NS; ++k)
            for (int b = lane; b < NBKT; b += 32) {
                const u32 c = sm.hist[warp][k][b];
                if (c) {
                    BucketStream& bk = ws.bst[tns].s[stream0 + k];
                    atomicAdd(&bk.cnt[b], c);
                    const s64 sum = ((s64)(int)sm.shi[warp][k][b] << 16) + (s64)sm.slo[warp][k][b];
                    if (sum) atomicAdd(reinterpret_cast<u64*>(&bk.sum[b]), (u64)sum);
                    sm.hist[warp][k][b] = 0; sm.slo[warp][k][b] = 0; sm.shi[warp][k][b] = 0;
                }
            }
        since = 0;
        __syncwarp();
    };

    while (ring.next_window(tile_cnt, lane, whi)) {
        while (ring.have()) {
            ring.issue_ahead(lane, surv);
            const u32 tile = ring.tile();
            if (cur < 0 || tile >= tb + ntl) {
                if (cur >= 0) flush(cur);
                cur = find_tensor(descs, nt, tile);
                tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
#pragma unroll
                for (int k = 0; k < NS; ++k) {
                    fn[k] = ws.bst[cur].s[stream0 + k].fn;
                    s1[k] = st[cur].s[stream0 + k].scale1; s2[k] = st[cur].s[stream0 + k].scale2;
                }
            }
            const u32 nel = ring.nel();
            if (!ring.wait()) {
                if (lane == 0) atomicOr(&call->flags, FLAG_TIMEOUT);
                return;
            }
#pragma unroll
            for (int k = 0; k < NS; ++k) {
                const float* data = ring.stage() + k * CH;
                u32* hist = sm.hist[warp][k];
                u32* slo = sm.slo[warp][k];
                u32* shi = sm.shi[warp][k];
                const float a1 = s1[k], a2 = s2[k];
                auto tally = [&](float x) {
                    const u32 b = bucket_index(x, fn[k]);
                    const int q = __float2int_rn(__fmul_rn(__fmul_rn(x, a1), a2));      // Q(x), |Q| < 2^31
                    atomicAdd(&hist[b], 1u);
                    atomicAdd(&slo[b], (u32)q & 0xffffu);
                    atomicAdd(&shi[b], (u32)(q >> 16));
                };
                const u32 whole = nel / 4;                             // groups of four that exist entirely
                for (u32 f = lane; f < whole; f += 32) {
                    const float4 v = *reinterpret_cast<const float4*>(data + 4 * f);
                    tally(v.x); tally(v.y); tally(v.z); tally(v.w);
                }
                if (lane < nel - 4 * whole) tally(data[4 * whole + lane]);
            }
            if (++since >= COUNT_FLUSH_CHUNKS * 512u / CH) flush(cur);
            ring.advance();
        }
    }
    if (cur >= 0) flush(cur);
}

// Where each bucket starts in the bucketed copy (exclusive prefix of the counts).
__global__ void __launch_bounds__(NBKT) bucket_offsets_kernel(Workspace ws) {
    __shared__ u32 wtot[NBKT / 32];
    BucketStream& bk = ws.bst[blockIdx.x].s[blockIdx.y];
    const int b = threadIdx.x, lane = b & 31, warp = b >> 5;
    const u32 c = bk.cnt[b];
    u32 incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const u32 v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    u32 base = 0;
    for (int w = 0; w < warp; ++w) base += wtot[w];
    bk.off[b] = base + incl - c;
    bk.cursor[b] = base + incl - c;
    if (b == NBKT - 1) bk.off[NBKT] = base + incl;
}

constexpr int SPT = 32;               // survivors a thread holds per window
constexpr int SCAP = SPT * TPB;       // survivors staged per window of tiles (8192)

struct ScatterSmem {
    float val[SCAP];                 // the window's survivors sorted by bucket
    unsigned char bid[SCAP];         // and their buckets
    u32 cnt[NBKT];                   // survivors of the window per bucket
    u32 lcur[NBKT];                  // next free place of each bucket in val[]
    u32 delta[NBKT];                 // place in the bucketed copy minus place in val[], per bucket
    u32 pre[33];                     // survivors before tile i of the window
    u32 wtot[TPB / 32];
    u32 wn;                          // tiles in the window
};

// Sweep 2 of the grouping: survivors into their buckets.
// A block takes windows of tiles of one tensor holding at most SCAP survivors.  Every thread
// loads its 32 survivors of the window at once (they stay in registers), the block counts them
// per bucket, reserves room in every bucket of the bucketed copy with one integer atomic,
// sorts the window by bucket in shared memory and writes each bucket's run with consecutive
// threads (one 4-byte store per survivor straight to its bucket would be bound by the number
// of write requests, not by bytes).
__global__ void __launch_bounds__(TPB, 4) bucket_scatter_kernel(const TensorDesc* __restrict__ descs,
                                                                const TensorState* __restrict__ st, int nt,
                                                                u32 tiles, Workspace ws, int stream) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    ScatterSmem& sm = *reinterpret_cast<ScatterSmem*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    const u32* tile_cnt = stream == 0 ? ws.tile_cnt_w : ws.tile_cnt_o;
    const float* surv = ws.surv[stream];
    int cur = -1;
    u32 tb = 0, ntl = 0;
    BucketFn fn = BucketFn{0, 0, 0, 0};
    u32 tile = lo;
    while (tile < hi) {
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            fn = ws.bst[cur].s[stream].fn;
        }
        const u32 wend = min(hi, tb + ntl);
        if (warp == 0) {              // the window: leading tiles whose survivors fit the stage
            const u32 c = tile + lane < wend ? tile_cnt[tile + lane] : 0u;
            u32 incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const u32 v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const u32 ok = __ballot_sync(0xffffffffu, tile + lane < wend && incl <= (u32)SCAP);
            sm.pre[lane] = incl - c;
            if (lane == 31) sm.pre[32] = incl;
            if (lane == 0) sm.wn = ok == 0xffffffffu ? 32u : (u32)__ffs((int)~ok) - 1u;
        }
        sm.cnt[tid] = 0;
        __syncthreads();
        const u32 wn = sm.wn, total = sm.pre[wn];
        if (total) {
            // this thread's survivors: window ranks tid, tid + 256, ...  (tile found by walking pre[])
            float x[SPT];
            u32 ti = 0;
#pragma unroll
            for (int k = 0; k < SPT; ++k) {
                const u32 idx = k * TPB + tid;
                x[k] = 0.f;
                if (idx < total) {
                    while (idx >= sm.pre[ti + 1]) ++ti;
                    x[k] = surv[(u64)(tile + ti) * TILE + (idx - sm.pre[ti])];
                }
            }
            u32 bk[SPT / 4];            // the buckets of x[], one byte each
#pragma unroll
            for (int g = 0; g < SPT / 4; ++g) {
                u32 w = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int k = 4 * g + j;
                    const u32 b = bucket_of(x[k], fn);
                    w |= b << (8 * j);
                    if (k * TPB + tid < total) atomicAdd(&sm.cnt[b], 1u);
                }
                bk[g] = w;
            }
            __syncthreads();
            {                          // exclusive prefix of the counts; room in the bucketed copy
                const u32 c = sm.cnt[tid];
                u32 incl = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const u32 v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                if (lane == 31) sm.wtot[warp] = incl;
                __syncthreads();
                u32 base = 0;
                for (int w = 0; w < warp; ++w) base += sm.wtot[w];
                sm.lcur[tid] = base + incl - c;
                const u32 g = c ? atomicAdd(&ws.bst[cur].s[stream].cursor[tid], c) : 0u;
                sm.delta[tid] = g - (base + incl - c);
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < SPT; ++k) {
                if (k * TPB + tid < total) {
                    const u32 b = (bk[k / 4] >> (8 * (k & 3))) & 255u;
                    const u32 r = atomicAdd(&sm.lcur[b], 1u);
                    sm.val[r] = x[k];
                    sm.bid[r] = (unsigned char)b;
                }
            }
            __syncthreads();
            float* dst = ws.bkt[stream] + (u64)tb * TILE;
            for (u32 i = tid; i < total; i += TPB) dst[i + sm.delta[sm.bid[i]]] = sm.val[i];
        }
        tile += wn;
        __syncthreads();
    }
}

// The bucket each threshold falls into; the partial sums of the coming scan start at zero.
// Threads idx, idx + stride, ... of the caller share the K - 1 thresholds.
__device__ inline void plan_scan(const StreamState& s, BucketStream& bk, int K, int idx, int stride) {
    for (int j = idx; j < K - 1; j += stride) {
        bk.bstar[j] = bucket_of(s.thr[j], bk.fn);
        bk.part_cnt[j] = 0;
        bk.part_sum[j] = 0;
    }
}

// Exclusive prefix of the bucket sums; plan of the first iteration.  Grid (tensors, 3).
__global__ void __launch_bounds__(NBKT) bucket_prefix_kernel(const TensorState* __restrict__ st, Workspace ws, int K) {
    __shared__ s64 wtot[NBKT / 32];
    BucketStream& bk = ws.bst[blockIdx.x].s[blockIdx.y];
    const int b = threadIdx.x, lane = b & 31, warp = b >> 5;
    const s64 c = bk.sum[b];
    s64 incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const s64 v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    s64 base = 0;
    for (int w = 0; w < warp; ++w) base += wtot[w];
    bk.sumpre[b] = base + incl - c;
    if (b == NBKT - 1) bk.sumpre[NBKT] = base + incl;
    plan_scan(st[blockIdx.x].s[blockIdx.y], bk, K, b, NBKT);
}

// One iteration's data pass: for threshold j of a stream, the survivors of its bucket that lie
// at or below it.  Grid (work items, 3 * 14): a tensor has scan_n items that split each bucket.
__global__ void __launch_bounds__(TPB) bucket_scan_kernel(const TensorDesc* __restrict__ descs,
                                                          const TensorState* __restrict__ st, int nt,
                                                          Workspace ws, int K) {
    __shared__ s64 rsum[TPB / 32];
    __shared__ u32 rcnt[TPB / 32];
    int lo = 0, hi = nt - 1;                       // tensor that owns this work item
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (descs[mid].scan_first <= blockIdx.x) lo = mid; else hi = mid - 1;
    }
    const int t = lo, k = blockIdx.y / (K - 1), j = blockIdx.y % (K - 1);
    const u32 split = blockIdx.x - descs[t].scan_first, nsplit = descs[t].scan_n;
    BucketStream& bk = ws.bst[t].s[k];
    const u32 b = bk.bstar[j];
    const u32 b_lo = bk.off[b], n = bk.off[b + 1] - b_lo;
    if (n == 0) return;
    const u32 a = b_lo + (u32)(((u64)n * split) / nsplit), e = b_lo + (u32)(((u64)n * (split + 1)) / nsplit);
    const StreamState& ss = st[t].s[k];
    const float thr = ss.thr[j], s1 = ss.scale1, s2 = ss.scale2;
    const float* data = ws.bkt[k] + (u64)descs[t].tile_begin * TILE;
    u32 cnt = 0;
    s64 sum = 0;
    u32 i = a + threadIdx.x;
    for (; i + 7 * TPB < e; i += 8 * TPB) {                 // eight independent loads in flight
        float x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = __ldcs(data + i + j * TPB);
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (!(x[j] > thr)) {
                ++cnt;
                sum += __float2int_rn(__fmul_rn(__fmul_rn(x[j], s1), s2));
            }
    }
    for (; i < e; i += TPB) {
        const float x = __ldcs(data + i);
        if (!(x > thr)) {
            ++cnt;
            sum += __float2int_rn(__fmul_rn(__fmul_rn(x, s1), s2));
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    cnt = __reduce_add_sync(0xffffffffu, cnt);
#pragma unroll
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) { rcnt[warp] = cnt; rsum[warp] = sum; }
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 c = 0; s64 s = 0;
        for (int w = 0; w < TPB / 32; ++w) { c += rcnt[w]; s += rsum[w]; }
        if (c) {
            atomicAdd(&bk.part_cnt[j], c);
            atomicAdd(reinterpret_cast<u64*>(&bk.part_sum[j]), (u64)s);
        }
    }
}

// New centres from the finished scan; one block per (tensor, stream), thread j = cluster j.
// L_j = survivors at or below threshold j = whole buckets below its bucket + the scanned part;
// cluster k has L_k - L_(k-1) members (L_-1 = 0, L_(K-1) = all), and its sum likewise.
__global__ void __launch_bounds__(KCAP) bucket_update_kernel(TensorState* __restrict__ st, Workspace ws, int K) {
    __shared__ u64 Ls[KCAP];
    __shared__ s64 Ss[KCAP];
    __shared__ float cs[KCAP];
    const int t = blockIdx.x, stream = blockIdx.y, j = threadIdx.x;
    StreamState& s = st[t].s[stream];
    BucketStream& bk = ws.bst[t].s[stream];
    u64 L = 0;
    s64 S = 0;
    if (j < K - 1) {
        const u32 b = bk.bstar[j];
        L = (u64)bk.off[b] + bk.part_cnt[j];
        S = bk.sumpre[b] + bk.part_sum[j];
    } else if (j == K - 1) {
        L = bk.off[NBKT];
        S = bk.sumpre[NBKT];
    }
    Ls[j] = L; Ss[j] = S;
    __syncthreads();
    float c = __uint_as_float(0x7f800000u);
    if (j < K) {
        const u64 n = j == 0 ? L : L - Ls[j - 1];
        const s64 sum = j == 0 ? S : S - Ss[j - 1];
        c = s.cent[j];
        if (n) {
            const double mean = __ll2double_rn(sum) / __ull2double_rn(n);
            const double scale = __longlong_as_double((s64)(s.e - 30 + 1023) << 52);
            c = __double2float_rn(mean * scale);
        }
    }
    cs[j] = c;
    __syncthreads();
    if (j < K) {                      // sort ascending: rank of each centre among the K (ties by index)
        int rank = 0;
        for (int i = 0; i < K; ++i) {
            const float o = cs[i];
            rank += (o < c) || (o == c && i < j);
        }
        s.cent[rank] = c;
    }
    __syncthreads();
    set_thresholds(s, K, j, KCAP);
    __syncthreads();
    plan_scan(s, bk, K, j, KCAP);
}

void launch_kmeans(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                   u32 scan_items, const Workspace& ws, const Params& p, CallState* call) {
    const int K = centres_of(p.bits);
    kmeans_start_kernel<<<dim3(nt, 3), SAMPLE_MAX, 0, cfg.stream>>>(descs, st, ws, p.seed, K);
    prof_mark(cfg, ST_KMEANS_START, 1);
    if (!tiles || p.kmeans_iters == 0) return;
    const u32 grid = min((tiles + BWARPS - 1) / BWARPS, (u32)cfg.sms * 5u);
    {
        const size_t m1 = sizeof(BucketCountSmem<1, 512>), m2 = sizeof(BucketCountSmem<2, 256>);
        cudaFuncSetAttribute(bucket_count_kernel<1, 512>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m1);
        cudaFuncSetAttribute(bucket_count_kernel<2, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m2);
        bucket_count_kernel<1, 512><<<grid, TPB, m1, cfg.stream>>>(descs, st, nt, tiles, ws, 0, call);
        bucket_count_kernel<2, 256><<<grid, TPB, m2, cfg.stream>>>(descs, st, nt, tiles, ws, 1, call);
        prof_mark(cfg, ST_BUCKET_IDS, 2);
    }
    bucket_offsets_kernel<<<dim3(nt, 3), NBKT, 0, cfg.stream>>>(ws);
    {
        const u32 sgrid = min(tiles, (u32)cfg.sms * 4u);
        cudaFuncSetAttribute(bucket_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ScatterSmem));
        for (int k = 0; k < 3; ++k)
            bucket_scatter_kernel<<<sgrid, TPB, sizeof(ScatterSmem), cfg.stream>>>(descs, st, nt, tiles, ws, k);
    }
    prof_mark(cfg, ST_BUCKET_SCATTER, 4);
    bucket_prefix_kernel<<<dim3(nt, 3), NBKT, 0, cfg.stream>>>(st, ws, K);
    prof_mark(cfg, ST_BUCKET_SUM, 1);
    for (int it = 0; it < p.kmeans_iters; ++it) {
        bucket_scan_kernel<<<dim3(scan_items, 3 * (K - 1)), TPB, 0, cfg.stream>>>(descs, st, nt, ws, K);
        prof_mark(cfg, ST_BUCKET_SCAN, 1);
        bucket_update_kernel<<<dim3(nt, 3), KCAP, 0, cfg.stream>>>(st, ws, K);
        prof_mark(cfg, ST_KMEANS_UPDATE, 1);
    }
}

}  // namespace excp
