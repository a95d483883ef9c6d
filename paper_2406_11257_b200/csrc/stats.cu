// Per-tensor statistics behind the two thresholds of Section 3.2:
//   the lower median of |W_t| or |dW_t| (Eq. rw), an exact order statistic found on
//   fp32 bit patterns, and the exact mean of |ea| (Eq. ro) by integer accumulation.
//
// One sweep over the data is the rule:
//   median_sample  65536 evenly spaced elements per tensor; two order statistics of the sample
//                  bracket the median (a tensor no larger than the sample is settled here)
//   stats_sweep    counts the elements below the bracket, gathers the keys inside it (about
//                  2.5 % of the tensor), and accumulates the exact sum of |ea|
//   stats_finish   selects the median among the gathered keys; the correctly rounded mean
//                  (multi-word integer arithmetic); both thresholds
// If the bracket misses the median (the sample misrepresents the tensor), that tensor takes
// the histogram path -- two more sweeps: a histogram of the top 13 key bits, then a gather of
// the median's bin and a select inside it.  Its kernels are always launched and return at
// once for tensors that do not need them.
//
// Every reduction is over integers, so the result does not depend on the
// order in which blocks or warps run.
#include "excp_common.cuh"
#include "warp_ring.cuh"
#include <type_traits>

namespace excp {

// alpha * median, the right-hand side of Eq. (rw).  A negative alpha is how the launcher passes
// "the threshold is set": then |alpha| itself is the threshold and the median is not used.
__device__ __forceinline__ float weight_threshold(float alpha, float median) {
    return alpha < 0.f || (alpha == 0.f && signbit(alpha)) ? -alpha : __fmul_rn(alpha, median);
}

// ---------------------------------------------------------------------------
// Find the bin that holds rank k (0-based) in a histogram in shared memory.
// Threads 0..255 each own BINS/256 consecutive bins.  All threads of the block
// must call.  Results are valid in every thread.
template <int BINS>
__device__ void find_rank_block(const u32* hist, u32 k, u32& bin, u32& rank_in, u32& cnt) {
    constexpr int PER = BINS / 256;
    __shared__ u32 warp_tot[8];
    __shared__ u32 res[3];
    const int tid = threadIdx.x;
    u32 local = 0;
    if (tid < 256) {
#pragma unroll 4
        for (int i = 0; i < PER; ++i) local += hist[tid * PER + i];
    }
    u32 incl = local;
    if (tid < 256) {
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            u32 v = __shfl_up_sync(0xffffffffu, incl, o);
            if ((tid & 31) >= o) incl += v;
        }
        if ((tid & 31) == 31) warp_tot[tid >> 5] = incl;
    }
    __syncthreads();
    if (tid < 256) {
        u32 base = 0;
        for (int w = 0; w < (tid >> 5); ++w) base += warp_tot[w];
        u32 excl = base + incl - local;
        if (k >= excl && k < excl + local) {
            u32 run = excl;
            for (int i = 0; i < PER; ++i) {
                u32 h = hist[tid * PER + i];
                if (k < run + h) { res[0] = tid * PER + i; res[1] = k - run; res[2] = h; break; }
                run += h;
            }
        }
    }
    __syncthreads();
    bin = res[0]; rank_in = res[1]; cnt = res[2];
    __syncthreads();
}

// ---------------------------------------------------------------------------
// Histogram path, sweep 1: top 13 key bits, per block in shared memory, merged with integer
// atomics.  Only tensors flagged need_hist.
template <typename WT>
__global__ void __launch_bounds__(TPB) hist1_kernel(const TensorDesc* __restrict__ descs,
                                                    TensorState* __restrict__ st, int nt, u32 tiles,
                                                    int residual_median) {
    __shared__ u32 hist[HIST1_BINS];
    const int tid = threadIdx.x;
    for (int i = tid; i < HIST1_BINS; i += TPB) hist[i] = 0;
    __syncthreads();
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u64 n = 0;
    bool active = false;
    const WT *w_t = nullptr, *w_prev = nullptr;
    auto flush_hist = [&](int t) {
        __syncthreads();
        for (int i = tid; i < HIST1_BINS; i += TPB) {
            u32 v = hist[i];
            if (v) { atomicAdd(&st[t].hist1[i], v); hist[i] = 0; }
        }
        __syncthreads();
    };
    for (u32 tile = lo; tile < hi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            if (cur >= 0 && active) flush_hist(cur);
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles; n = descs[cur].numel;
            w_t = static_cast<const WT*>(descs[cur].w_t); w_prev = static_cast<const WT*>(descs[cur].w_prev);
            active = st[cur].need_hist != 0;
            if (!active) tile = tb + ntl - 1;          // nothing to do for this tensor
        }
        if (!active) continue;
        const u64 base = (u64)(tile - tb) * TILE;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const u64 i0 = base + (u64)r * (TPB * 4) + (u64)tid * 4;
            float a[4], b[4];
            const int nv = load4(w_t, i0, n, a);
            if (residual_median) {
                load4(w_prev, i0, n, b);
#pragma unroll
                for (int k = 0; k < 4; ++k) a[k] = __fsub_rn(a[k], b[k]);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < nv) atomicAdd(&hist[(__float_as_uint(a[k]) & 0x7fffffffu) >> HIST1_SHIFT], 1u);
        }
    }
    if (cur >= 0 && active) flush_hist(cur);
}

// ---------------------------------------------------------------------------
// Correctly rounded fp32 of (sum |ea|) / n from the three tables.
// X = sum in units of 2^-173 held in twelve 32-bit limbs.
__device__ static void big_add(u32* x, int limb, u32 val) {
    u64 c = val;
    for (int i = limb; c && i < 12; ++i) { c += x[i]; x[i] = (u32)c; c >>= 32; }
}
__device__ static void big_add_shifted(u32* x, u64 v, int shift) {
    if (!v) return;
    const int limb = shift >> 5, s = shift & 31;
    const u64 v0 = (u64)(u32)v << s;          // low half shifted: 64 bits
    const u64 v1 = (u64)(u32)(v >> 32) << s;  // high half
    big_add(x, limb, (u32)v0);
    big_add(x, limb + 1, (u32)(v0 >> 32));
    big_add(x, limb + 1, (u32)v1);
    big_add(x, limb + 2, (u32)(v1 >> 32));
}
__device__ static u32 big_bit(const u32* q, int pos) { return (q[pos >> 5] >> (pos & 31)) & 1u; }

__device__ static float exact_mean_from_tables(const u64* lo, const u64* hi, const u64* low, u64 n) {
    u32 x[12];
    for (int i = 0; i < 12; ++i) x[i] = 0;
    for (int e = 1; e < 256; ++e) {
        big_add_shifted(x, lo[e], e - 1);
        big_add_shifted(x, hi[e], e - 1 + 32);
        big_add_shifted(x, low[e], e + 23);
    }
    // q = floor(X / n), r = X mod n   (n < 2^32)
    u32 q[12];
    u64 rem = 0;
    for (int i = 11; i >= 0; --i) {
        const u64 cur = (rem << 32) | x[i];
        q[i] = (u32)(cur / n);
        rem = cur % n;
    }
    int top = -1;
    for (int i = 11; i >= 0; --i) if (q[i]) { top = i * 32 + 31 - __clz(q[i]); break; }
    if (top < 0) return 0.f;                       // below 2^-173: rounds to zero
    const int ev = top - 173;                      // floor(log2(mean))
    const int u = max(ev - 23, -149);              // exponent of the last kept bit
    const int sh = u + 173;                        // >= 24
    u32 m = 0;
    for (int b = 24; b >= 0; --b) {
        const int pos = sh + b;
        m = (m << 1) | (pos < 384 ? big_bit(q, pos) : 0u);
    }
    const u32 round = big_bit(q, sh - 1);
    bool sticky = rem != 0;
    for (int pos = 0; pos < sh - 1 && !sticky; ++pos) sticky = big_bit(q, pos);
    if (round && (sticky || (m & 1u))) ++m;
    return __uint_as_float((u32)((u + 150) << 23) + m - 0x800000u);
}

// Histogram path: the bin that holds the median rank.  One block per flagged tensor.
__global__ void __launch_bounds__(TPB) hist1_finish_kernel(const TensorDesc* __restrict__ descs,
                                                           TensorState* __restrict__ st) {
    __shared__ u32 hist[HIST1_BINS];
    const int t = blockIdx.x, tid = threadIdx.x;
    TensorState& s = st[t];
    if (!s.need_hist) return;
    const u64 n = descs[t].numel;
    for (int i = tid; i < HIST1_BINS; i += TPB) hist[i] = s.hist1[i];
    __syncthreads();
    u32 bin, rank_in, cnt;
    find_rank_block<HIST1_BINS>(hist, (u32)((n - 1) / 2), bin, rank_in, cnt);
    if (tid == 0) { s.bin1 = bin; s.rank_in_bin = rank_in; s.bin_count = cnt; s.cand_count = 0; }
}

// ---------------------------------------------------------------------------
// Histogram path, sweep 2: keys of the selected bin -> candidate list (kept in the tensor's own
// survivor segment, which the mask sweep overwrites afterwards).  Only flagged tensors.
template <typename WT>
__global__ void __launch_bounds__(TPB) hist2_kernel(const TensorDesc* __restrict__ descs,
                                                     TensorState* __restrict__ st, int nt, u32 tiles,
                                                     Workspace ws, int residual_median) {
    const int tid = threadIdx.x, lane = tid & 31;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0, bin1 = 0;
    u64 n = 0;
    bool active = false;
    const WT *w_t = nullptr, *w_prev = nullptr;
    u32* cand = nullptr;
    for (u32 tile = lo; tile < hi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles; n = descs[cur].numel;
            w_t = static_cast<const WT*>(descs[cur].w_t); w_prev = static_cast<const WT*>(descs[cur].w_prev);
            bin1 = st[cur].bin1;
            cand = reinterpret_cast<u32*>(ws.surv[0] + (u64)tb * TILE);
            active = st[cur].need_hist != 0;
            if (!active) tile = tb + ntl - 1;          // nothing to do for this tensor
        }
        if (!active) continue;
        const u64 base = (u64)(tile - tb) * TILE;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const u64 i0 = base + (u64)r * (TPB * 4) + (u64)tid * 4;
            float a[4], b[4];
            const int nv = load4(w_t, i0, n, a);
            if (residual_median) {
                load4(w_prev, i0, n, b);
#pragma unroll
                for (int k = 0; k < 4; ++k) a[k] = __fsub_rn(a[k], b[k]);
            }
            u32 key[4];
            int mine = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                key[k] = __float_as_uint(a[k]) & 0x7fffffffu;
                if (k < nv && (key[k] >> HIST1_SHIFT) == bin1) ++mine;
            }
            if (__any_sync(0xffffffffu, mine)) {
                int incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                u32 start = 0;
                if (lane == 31) start = atomicAdd(&st[cur].cand_count, (u32)incl);
                start = __shfl_sync(0xffffffffu, start, 31) + incl - mine;
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (k < nv && (key[k] >> HIST1_SHIFT) == bin1) cand[start++] = key[k];
            }
        }
    }
}

// Histogram path: select inside the bin's keys; the weight threshold.
__global__ void __launch_bounds__(1024) hist2_finish_kernel(const TensorDesc* __restrict__ descs,
                                                            TensorState* __restrict__ st, Workspace ws,
                                                            float alpha) {
    __shared__ u32 hist[512];
    const int t = blockIdx.x, tid = threadIdx.x;
    TensorState& s = st[t];
    if (!s.need_hist) return;
    const u32 c = s.cand_count;
    const u32* cand = reinterpret_cast<const u32*>(ws.surv[0] + (u64)descs[t].tile_begin * TILE);
    u32 k = s.rank_in_bin;
    if (tid < 512) hist[tid] = 0;
    __syncthreads();
    for (u32 i = tid; i < c; i += 1024) atomicAdd(&hist[(cand[i] >> 9) & 511u], 1u);
    __syncthreads();
    u32 a, ka, ca;
    find_rank_block<512>(hist, k, a, ka, ca);
    if (tid < 512) hist[tid] = 0;
    __syncthreads();
    for (u32 i = tid; i < c; i += 1024) {
        const u32 key = cand[i];
        if (((key >> 9) & 511u) == a) atomicAdd(&hist[key & 511u], 1u);
    }
    __syncthreads();
    u32 b, kb, cb;
    find_rank_block<512>(hist, ka, b, kb, cb);
    if (tid == 0) {
        const u32 bits = (s.bin1 << HIST1_SHIFT) | (a << 9) | b;
        s.median_bits = bits;
        s.thr_w = weight_threshold(alpha, __uint_as_float(bits));
        if (c != s.bin_count) s.flags |= FLAG_INTERNAL;
    }
}


// ---------------------------------------------------------------------------
// The element of rank `rank` (0-based, ascending) among cnt keys that all lie in
// [base, base + width], by digit passes of at most 8 bits over key - base, from the top bit of
// width down: the digits of a narrow range spread over the bins, so the shared-memory atomics
// do not pile up on one counter.  Whole block (at least 256 threads); hist: 256 words.
__device__ static u32 block_select(const u32* __restrict__ keys, u32 cnt, u32 rank, u32* hist,
                                   u32 base, u32 width) {
    int hs = 32 - __clz(width | 1u);         // bits of key - base above hs equal `prefix`
    u32 prefix = 0;
    while (hs > 0) {
        const int ls = max(hs - 8, 0);
        const u32 dmask = (1u << (hs - ls)) - 1u;
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
        for (u32 i = threadIdx.x; i < cnt; i += blockDim.x) {
            const u32 d = keys[i] - base;
            if ((u32)((u64)d >> hs) == prefix) atomicAdd(&hist[(d >> ls) & dmask], 1u);
        }
        __syncthreads();
        u32 bin, rin, c;
        find_rank_block<256>(hist, rank, bin, rin, c);
        prefix = (prefix << (hs - ls)) | bin;
        rank = rin;
        hs = ls;
    }
    return base + prefix;
}

constexpr u32 MEDIAN_SAMPLE = 65536;         // evenly spaced elements that bracket the median
constexpr int SAMPLE_BINS = 2048;            // steps of the sample's histogram that places the bracket
constexpr u32 MEDIAN_MARGIN = MEDIAN_SAMPLE / 80;   // +-1.25 % of the sample: about six standard deviations

// One block per tensor.  The sample's keys go to the tensor's second survivor segment (free
// until the mask sweep); a tensor no larger than the sample gets its exact median here.
template <typename WT>
__global__ void __launch_bounds__(1024) median_sample_kernel(const TensorDesc* __restrict__ descs,
                                                             TensorState* __restrict__ st, Workspace ws,
                                                             int residual_median) {
    __shared__ u32 hist[256];
    __shared__ u32 fine[SAMPLE_BINS];
    __shared__ u32 range[2];
    const int t = blockIdx.x, tid = threadIdx.x;
    TensorState& s = st[t];
    const u64 n = descs[t].numel;
    if (n == 0) {
        if (tid == 0) { s.med_done = 1; s.median_bits = 0; }
        return;
    }
    if (tid == 0) { range[0] = 0xffffffffu; range[1] = 0; }
    __syncthreads();
    u32 kmin = 0xffffffffu, kmax = 0;
    const u32 m = (u32)min((u64)MEDIAN_SAMPLE, n);
    u32* keys = reinterpret_cast<u32*>(ws.surv[1] + (u64)descs[t].tile_begin * TILE);
    const WT* w_t = static_cast<const WT*>(descs[t].w_t);
    const WT* w_prev = static_cast<const WT*>(descs[t].w_prev);
    for (u32 j = tid; j < m; j += 1024) {
        const u64 i = ((u64)j * n) / m;
        float a = wget(w_t, i);
        if (residual_median) a = __fsub_rn(a, wget(w_prev, i));
        const u32 key = __float_as_uint(a) & 0x7fffffffu;
        keys[j] = key;
        kmin = min(kmin, key);
        kmax = max(kmax, key);
    }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if ((tid & 31) == 0) { atomicMin(&range[0], kmin); atomicMax(&range[1], kmax); }
    __syncthreads();
    kmin = range[0];
    const u32 width = range[1] - kmin;
    if (n <= MEDIAN_SAMPLE) {
        const u32 med = block_select(keys, m, (u32)((n - 1) / 2), hist, kmin, width);
        if (tid == 0) { s.median_bits = med; s.med_done = 1; }
        return;
    }
    // The bracket only has to hold the two sample ranks, not to be them: one histogram of the
    // sample over 2048 equal steps of its range, and the bracket runs from the lower edge of the
    // step that holds rank m/2 - margin to the upper edge of the step that holds rank m/2 + margin.
    const int shift = max(32 - __clz(width | 1u) - 11, 0);
    for (int i = tid; i < SAMPLE_BINS; i += 1024) fine[i] = 0;
    __syncthreads();
    for (u32 j = tid; j < m; j += 1024) atomicAdd(&fine[(keys[j] - kmin) >> shift], 1u);
    __syncthreads();
    u32 bin_lo, bin_hi, rin, cnt;
    find_rank_block<SAMPLE_BINS>(fine, m / 2 - MEDIAN_MARGIN, bin_lo, rin, cnt);
    find_rank_block<SAMPLE_BINS>(fine, m / 2 + MEDIAN_MARGIN, bin_hi, rin, cnt);
    if (tid == 0) {
        s.lo_key = kmin + (bin_lo << shift);
        s.hi_key = (u32)min((u64)kmin + (((u64)bin_hi + 1) << shift) - 1, (u64)range[1]);
    }
}

// ---------------------------------------------------------------------------
// The statistics sweep.  Every warp walks its own run of tiles; 512-value chunks of the
// median's source stream(s) and of ea arrive in its ring of stages.
constexpr int SCH = 512;             // values per stream per staged chunk
constexpr int SST = 2;               // chunks in flight per warp
constexpr int SWARPS = TPB / 32;
constexpr int QCAP = 16;             // bracket keys a lane can hold before the warp hands them over

struct SweepSmem {
    float buf[SWARPS][SST][3][SCH];
    unsigned long long bar[SWARPS][SST];
    u32 q[SWARPS][QCAP][32];         // per-lane queues of bracket keys waiting for their place in the tensor's list
};

template <typename WT>
__global__ void __launch_bounds__(TPB, 2) stats_sweep_kernel(const TensorDesc* __restrict__ descs,
                                                             TensorState* __restrict__ st, int nt, u32 tiles,
                                                             Workspace ws, int residual_median, CallState* call, u64 wait_ns) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    SweepSmem& sm = *reinterpret_cast<SweepSmem*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    WarpRing<3, SCH, SST> ring;
    ring.init(&sm.buf[warp][0][0][0], sm.bar[warp], lane, wait_ns);
    const u32 gw = blockIdx.x * SWARPS + warp, nw = gridDim.x * SWARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    TileWalk<SCH> ic, cc;
    ic.start(wlo); cc.start(wlo);
    constexpr u32 WPER = 16 / sizeof(WT);      // weights per 16 bytes: a bulk copy moves whole 16-byte units
    const WT* iw[2] = {nullptr, nullptr};      // issue side: the weight streams, and ea
    const float* iea = nullptr;
    const WT* cw[2] = {nullptr, nullptr};      // consume side
    const float* cea = nullptr;
    u32 lo_key = 0, span = 0;        // bracket [lo_key, lo_key + span]
    bool want_median = false;
    u32* cand = nullptr;
    u32* const q = &sm.q[warp][0][lane];   // this lane's queue: q[32 * j]
    u32 nq = 0;                      // keys in it
    u32 below = 0;                   // this thread's count of keys under the bracket
    u64 acc = 0;                     // this thread's share of sum |ea|, unit 2^(ecur-174)
    int ecur = 1;                    // biased exponent the unit is tied to (warp uniform)
    int since = 0;
    int prev = -1;

    auto flush_acc = [&](int t) {
        const u64 s = warp_sum_u64(acc);
        if (lane == 0 && s) {
            atomicAdd(&st[t].sum_lo[ecur], s & 0xffffffffull);
            atomicAdd(&st[t].sum_hi[ecur], s >> 32);
        }
        acc = 0;
        since = 0;
    };
    auto flush_below = [&](int t) {
        const u32 b = __reduce_add_sync(0xffffffffu, below);
        if (lane == 0 && b) atomicAdd(&st[t].count_below, b);
        below = 0;
    };

    auto flush_cand = [&](int t) {   // one atomic for the warp's queued keys
        u32 incl = nq;
#pragma unroll
        for (int w = 1; w < 32; w <<= 1) {
            const u32 v = __shfl_up_sync(0xffffffffu, incl, w);
            if (lane >= w) incl += v;
        }
        u32 base = 0;
        if (lane == 31 && incl) base = atomicAdd(&st[t].cand_count, incl);
        base = __shfl_sync(0xffffffffu, base, 31) + incl - nq;
        for (u32 j = 0; j < nq; ++j)
            if (EXCP_IN_BOUNDS(call, (u64)base + j < (u64)descs[t].num_tiles * TILE)) cand[base + j] = q[32 * j];
        nq = 0;
    };

    while (cc.tile < whi) {
        while (ic.tile < whi && ring.can_issue()) {
            if (ic.chunk == 0 && ic.enter_tile(descs, nt)) {
                iw[0] = static_cast<const WT*>(descs[ic.tns].w_t);
                iw[1] = residual_median ? static_cast<const WT*>(descs[ic.tns].w_prev) : nullptr;
                iea = descs[ic.tns].ea;
            }
            const u64 e0 = ic.elem0();
            const void* src[3] = {iw[0] + e0, iw[1] ? iw[1] + e0 : nullptr, iea + e0};
            const u32 v = ic.valid();
            const u32 wb = (v & ~(WPER - 1u)) * (u32)sizeof(WT);
            const u32 bytes[3] = {wb, wb, (v & ~3u) * 4u};
            ring.issue_bytes(lane, src, bytes);
            ic.next();
        }
        if (cc.chunk == 0 && cc.enter_tile(descs, nt)) {
            if (prev >= 0) { flush_acc(prev); flush_below(prev); flush_cand(prev); }
            prev = cc.tns;
            ecur = 1;
            cw[0] = static_cast<const WT*>(descs[cc.tns].w_t); cw[1] = static_cast<const WT*>(descs[cc.tns].w_prev);
            cea = descs[cc.tns].ea;
            want_median = st[cc.tns].med_done == 0;
            lo_key = st[cc.tns].lo_key;
            span = st[cc.tns].hi_key - lo_key;
            cand = reinterpret_cast<u32*>(ws.surv[0] + (u64)cc.tb * TILE);
        }
        const u32 valid = cc.valid(), nbulk = valid & ~3u, nbulk_w = valid & ~(WPER - 1u);
        const u64 e0 = cc.elem0();
        if (!ring.wait()) {
            if (lane == 0) atomicOr(&call->flags, FLAG_TIMEOUT);
            ring.drain();
            return;
        }
        const float* stg = ring.stage();
        auto weights4 = [&](int k, u32 o, bool full, float out[4]) {     // four weights of stream k at offset o
            if constexpr (sizeof(WT) == 4) {
                if (full) {
                    const float4 t = *reinterpret_cast<const float4*>(stg + k * SCH + o);
                    out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
                } else {
                    fetch4(stg + k * SCH, reinterpret_cast<const float*>(cw[k]) + e0, o, nbulk, valid, out);
                }
            } else {
                fetch4w<WT>(stg + k * SCH, cw[k] + e0, o, full ? (u32)SCH : nbulk_w, valid, out);
            }
        };
        // exact sum of |ea|: every lane adds its 16 values of the chunk in fp64 (exact: they span at most
        // 52 bits, see below), and the chunk's sums join a 64-bit integer whose unit 2^(ecur-174) is tied to
        // the largest exponent this warp has met in this tensor
        double dsum = 0.0;
        u32 kmax = 0;
        u32 lowkey = 0xffffffffu;            // smallest non-zero key, minus one
        auto sweep_chunk = [&](auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;     // the whole chunk came by bulk copy
#pragma unroll
            for (int r = 0; r < SCH / 128; ++r) {
                const u32 o = r * 128 + lane * 4;
                float a[4], b[4], e[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) e[k] = 0.f;
                if (FULL || (u32)r * 128u < valid) {
                    if (FULL) {
                        const float4 t = *reinterpret_cast<const float4*>(stg + 2 * SCH + o);
                        e[0] = t.x; e[1] = t.y; e[2] = t.z; e[3] = t.w;
                    } else {
                        fetch4(stg + 2 * SCH, cea + e0, o, nbulk, valid, e);
                    }
                    if (want_median) {
                        weights4(0, o, FULL, a);
                        if (residual_median) {
                            weights4(1, o, FULL, b);
#pragma unroll
                            for (int k = 0; k < 4; ++k) a[k] = __fsub_rn(a[k], b[k]);
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const u32 key = __float_as_uint(a[k]) & 0x7fffffffu;
                            const bool real = FULL || o + k < valid;
                            below += real && key < lo_key;
                            if (real && key - lo_key <= span) {      // unsigned: false below lo_key
                                q[32 * nq] = key;
                                ++nq;
                            }
                        }
                        if (__any_sync(0xffffffffu, nq > (u32)QCAP - 4u)) flush_cand(cc.tns);
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const u32 kk = __float_as_uint(e[k]) & 0x7fffffffu;
                    kmax = max(kmax, kk);
                    lowkey = min(lowkey, kk - 1u);
                    dsum += (double)__uint_as_float(kk);
                }
            }
        };
        if (valid == (u32)SCH) sweep_chunk(std::true_type{});
        else sweep_chunk(std::false_type{});
        const int emax = max((int)(__reduce_max_sync(0xffffffffu, kmax) >> 23), 1);
        if (emax > ecur) { flush_acc(cc.tns); ecur = emax; }
        const int bias = 24 - ecur;
        // A value is a whole number of units iff its exponent is within 24 binades of ecur; then a lane's 16
        // values (each below 2^(ecur-126), the unit 2^(ecur-174)) add up to less than 2^52 units: exact in fp64.
        const bool has_low = lowkey != 0xffffffffu && (int)max((lowkey + 1u) >> 23, 1u) + bias < 0;
        if (!__any_sync(0xffffffffu, has_low)) {
            const double unit_inv = __longlong_as_double((s64)(1197 - ecur) << 52);          // 2^(174-ecur)
            acc += (u64)__double2ull_rz(dsum * unit_inv);
        } else {
            // rare: some non-zero value lies more than 24 binades under the unit.  Redo the chunk in integers:
            // mantissas shifted to the unit, the small ones into the table of their own
            for (u32 o = lane; o < valid; o += 32) {
                const u32 kk = __float_as_uint(o < nbulk ? stg[2 * SCH + o] : __ldg(cea + e0 + o)) & 0x7fffffffu;
                const u32 e1 = max(kk >> 23, 1u);
                const u32 m = kk - ((e1 - 1u) << 23);                    // mantissa with its implicit bit (none below 2^-126)
                if ((int)e1 + bias >= 0) acc += (u64)m << (e1 + bias);
                else if (kk) atomicAdd(&st[cc.tns].sum_low[e1], (u64)m);
            }
        }
        if (++since >= 32) flush_acc(cc.tns);
        ring.release();
        cc.next();
    }
    if (prev >= 0) { flush_acc(prev); flush_below(prev); flush_cand(prev); }
}

// The correctly rounded mean and its threshold; then, per tensor, either the flag for the
// histogram path (the bracket missed the median) or the start of the select among the
// bracket's keys.  One block per tensor.
__global__ void __launch_bounds__(TPB) stats_finish_kernel(const TensorDesc* __restrict__ descs,
                                                           TensorState* __restrict__ st, float alpha, float beta,
                                                           const CallState* call) {
    __shared__ u64 tab[3][256];
    if (call_aborted(call)) return;
    const int t = blockIdx.x, tid = threadIdx.x;
    TensorState& s = st[t];
    const u64 n = descs[t].numel;
    if (n == 0) {
        if (tid == 0) {
            s.mean_abs_ea = 0.f;
            s.thr_w = weight_threshold(alpha, 0.f);
            s.thr_o = __fmul_rn(beta, 0.f);
        }
        return;
    }
    tab[0][tid] = s.sum_lo[tid]; tab[1][tid] = s.sum_hi[tid]; tab[2][tid] = s.sum_low[tid];
    __syncthreads();
    if (tid != 0) return;
    const float mean = exact_mean_from_tables(tab[0], tab[1], tab[2], n);
    s.mean_abs_ea = mean;
    s.thr_o = __fmul_rn(beta, mean);                                  // beta * mean, Eq. (ro)
    if (s.med_done) {
        s.thr_w = weight_threshold(alpha, __uint_as_float(s.median_bits));
        return;
    }
    const u32 k = (u32)((n - 1) / 2), below = s.count_below, c = s.cand_count;
    if (k < below || k - below >= c) { s.need_hist = 1; return; }
    s.sel_hs = 32 - __clz((s.hi_key - s.lo_key) | 1u);
    s.sel_prefix = 0;
    s.sel_rank = k - below;
}

// One digit pass (at most 8 bits, from the top bit of the bracket's width down) of the select
// among a tensor's bracket keys.  grid = (SEL_SLICES, tensors): every block counts the digits
// of its slice of the keys that share the bits fixed so far, adds them to the tensor's table,
// and the block that arrives last picks the digit.  The pass that fixes the lowest bit writes
// the median and alpha * median (Eq. (rw)).  A tensor whose median is known returns at once.
constexpr int SEL_SLICES = 64;

__global__ void __launch_bounds__(TPB) median_digit_kernel(TensorState* __restrict__ st,
                                                           const TensorDesc* __restrict__ descs, Workspace ws,
                                                           int pass, float alpha, const CallState* call) {
    __shared__ u32 hist[256];
    __shared__ u32 is_last;
    if (call_aborted(call)) return;
    const int t = blockIdx.y, tid = threadIdx.x;
    TensorState& s = st[t];
    if (s.med_done | s.need_hist) return;
    const int hs = (int)s.sel_hs;
    if (hs == 0 || descs[t].numel == 0) return;
    const int ls = max(hs - 8, 0);
    const u32 dmask = (1u << (hs - ls)) - 1u;
    const u32 prefix = s.sel_prefix, base = s.lo_key, c = s.cand_count, rank = s.sel_rank;
    const u32* __restrict__ cand = reinterpret_cast<const u32*>(ws.surv[0] + (u64)descs[t].tile_begin * TILE);
    const u32 i0 = (u32)(((u64)c * blockIdx.x) / gridDim.x), i1 = (u32)(((u64)c * (blockIdx.x + 1)) / gridDim.x);
    hist[tid] = 0;
    __syncthreads();
    u32 i = i0 + tid;
    for (; i + 3 * TPB < i1; i += 4 * TPB) {
        u32 d[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) d[k] = __ldcg(cand + i + k * TPB) - base;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if ((u32)((u64)d[k] >> hs) == prefix) atomicAdd(&hist[(d[k] >> ls) & dmask], 1u);
    }
    for (; i < i1; i += TPB) {
        const u32 d = __ldcg(cand + i) - base;
        if ((u32)((u64)d >> hs) == prefix) atomicAdd(&hist[(d >> ls) & dmask], 1u);
    }
    __syncthreads();
    if (hist[tid]) atomicAdd(&s.sel_hist[pass][tid], hist[tid]);
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(&s.sel_done[pass], 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    hist[tid] = __ldcg(&s.sel_hist[pass][tid]);
    __syncthreads();
    u32 bin, rin, cnt;
    find_rank_block<256>(hist, rank, bin, rin, cnt);
    if (tid == 0) {
        const u32 np = (prefix << (hs - ls)) | bin;
        s.sel_prefix = np;
        s.sel_rank = rin;
        s.sel_hs = (u32)ls;
        if (ls == 0) {
            s.median_bits = base + np;
            s.med_done = 1;
            s.thr_w = weight_threshold(alpha, __uint_as_float(base + np));
        }
    }
}

void launch_stats(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                  const Workspace& ws, const Params& p, CallState* call) {
    const int resid = p.median_source == 1 && !(p.flags & OPT_NO_RESIDUAL);   // without the residual dW is W_t
    const float alpha = (p.flags & OPT_NO_M2W) ? -p.alpha : p.alpha;          // see weight_threshold
    auto run = [&](auto tag) {
        using WT = decltype(tag);
        median_sample_kernel<WT><<<nt, 1024, 0, cfg.stream>>>(descs, st, ws, resid);
        if (tiles) {
            const u32 grid = min((tiles + SWARPS - 1) / SWARPS, (u32)cfg.sms * 2u);
            cudaFuncSetAttribute(stats_sweep_kernel<WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SweepSmem));
            stats_sweep_kernel<WT><<<grid, TPB, sizeof(SweepSmem), cfg.stream>>>(descs, st, nt, tiles, ws, resid, call, p.wait_ns);
        }
        stats_finish_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, alpha, p.beta, call);
        if (tiles)
            for (int pass = 0; pass < 4; ++pass)
                median_digit_kernel<<<dim3(SEL_SLICES, nt), TPB, 0, cfg.stream>>>(st, descs, ws, pass, alpha, call);
        prof_mark(cfg, ST_STATS1, tiles ? 7 : 2);
        if (tiles) {          // the histogram path: returns at once unless a bracket missed
            hist1_kernel<WT><<<min(tiles, (u32)cfg.sms * 4u), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, resid);
            hist1_finish_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st);
            hist2_kernel<WT><<<min(tiles, (u32)cfg.sms * 8u), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, resid);
            hist2_finish_kernel<<<nt, 1024, 0, cfg.stream>>>(descs, st, ws, alpha);
            prof_mark(cfg, ST_STATS2, 4);
        }
    };
    if (p.wfmt == WF_F16) run(__half{});
    else if (p.wfmt == WF_BF16) run(__nv_bfloat16{});
    else run(float{});
}

}  // namespace excp
