// Per-tensor statistics behind the two thresholds of Section 3.2:
//   the lower median of |W_t| or |dW_t| (Eq. rw) by a radix select on fp32 bit
//   patterns, and the exact mean of |ea| (Eq. ro) by integer accumulation.
//
// Sweep 1 (stats1): histogram of the top 13 key bits (per-block in shared
//   memory, merged with integer atomics) + exact fixed-point sum of |ea|.
// finish1:          pick the bin holding the median rank; turn the sum tables
//   into the correctly rounded mean (multi-word integer arithmetic).
// Sweep 2 (stats2): gather the keys of that bin (about 1 % of the tensor).
// finish2:          select inside the candidates (two 9-bit levels); thresholds.
//
// Every reduction is over integers, so the result does not depend on the
// order in which blocks or warps run.
#include "excp_common.cuh"

namespace excp {

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
// Sweep 1.
__global__ void __launch_bounds__(TPB) stats1_kernel(const TensorDesc* __restrict__ descs,
                                                     TensorState* __restrict__ st, int nt, u32 tiles,
                                                     int residual_median) {
    __shared__ u32 hist[HIST1_BINS];
    const int tid = threadIdx.x, lane = tid & 31;
    for (int i = tid; i < HIST1_BINS; i += TPB) hist[i] = 0;
    __syncthreads();

    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u64 n = 0;
    const float *w_t = nullptr, *w_prev = nullptr, *ea = nullptr;
    u64 acc = 0;          // this thread's share of sum |ea|, unit 2^(ecur-174)
    int ecur = 1;         // biased exponent the unit is tied to (warp uniform)
    int since = 0;

    auto flush_acc = [&](int t) {
        u64 s = warp_sum_u64(acc);
        if (lane == 0 && s) {
            atomicAdd(&st[t].sum_lo[ecur], s & 0xffffffffull);
            atomicAdd(&st[t].sum_hi[ecur], s >> 32);
        }
        acc = 0;
        since = 0;
    };
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
            if (cur >= 0) { flush_hist(cur); flush_acc(cur); }
            ecur = 1;
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles; n = descs[cur].numel;
            w_t = descs[cur].w_t; w_prev = descs[cur].w_prev; ea = descs[cur].ea;
        }
        const u64 base = (u64)(tile - tb) * TILE;
        u32 ke[4 * ROUNDS];
        u32 kmax = 0;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const u64 i0 = base + (u64)r * (TPB * 4) + (u64)tid * 4;
            float a[4], b[4], e[4];
            const int nv = load4(w_t, i0, n, a);
            if (residual_median) {
                load4(w_prev, i0, n, b);
#pragma unroll
                for (int k = 0; k < 4; ++k) a[k] = __fsub_rn(a[k], b[k]);
            }
            load4(ea, i0, n, e);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (k < nv) atomicAdd(&hist[(__float_as_uint(a[k]) & 0x7fffffffu) >> HIST1_SHIFT], 1u);
                const u32 kk = __float_as_uint(e[k]) & 0x7fffffffu;
                ke[r * 4 + k] = kk;
                kmax = max(kmax, kk);
            }
        }
        // exact sum of |ea|: integer mantissas shifted to a common unit tied to
        // the largest exponent this warp has met
        const int emax = max((int)(__reduce_max_sync(0xffffffffu, kmax) >> 23), 1);
        if (emax > ecur) { flush_acc(cur); ecur = emax; }
#pragma unroll
        for (int j = 0; j < 4 * ROUNDS; ++j) {
            const u32 kk = ke[j];
            const int e = (int)(kk >> 23);
            const u32 m = (kk & 0x7fffffu) | (e ? 0x800000u : 0u);
            const int e1 = max(e, 1);
            const int sh = e1 - ecur + 24;
            if (sh >= 0) acc += (u64)m << sh;
            else if (m) atomicAdd(&st[cur].sum_low[e1], (u64)m);
        }
        if (++since >= 32) flush_acc(cur);
    }
    if (cur >= 0) { flush_hist(cur); flush_acc(cur); }
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

__global__ void __launch_bounds__(TPB) stats1_finish_kernel(const TensorDesc* __restrict__ descs,
                                                            TensorState* __restrict__ st) {
    __shared__ u32 hist[HIST1_BINS];
    __shared__ u64 tab[3][256];
    const int t = blockIdx.x, tid = threadIdx.x;
    TensorState& s = st[t];
    const u64 n = descs[t].numel;
    if (n == 0) {
        if (tid == 0) { s.bin1 = 0; s.rank_in_bin = 0; s.bin_count = 0; s.mean_abs_ea = 0.f; }
        return;
    }
    for (int i = tid; i < HIST1_BINS; i += TPB) hist[i] = s.hist1[i];
    tab[0][tid] = s.sum_lo[tid];
    tab[1][tid] = s.sum_hi[tid];
    tab[2][tid] = s.sum_low[tid];
    __syncthreads();
    u32 bin, rank_in, cnt;
    find_rank_block<HIST1_BINS>(hist, (u32)((n - 1) / 2), bin, rank_in, cnt);
    if (tid == 0) {
        s.bin1 = bin; s.rank_in_bin = rank_in; s.bin_count = cnt;
        s.mean_abs_ea = exact_mean_from_tables(tab[0], tab[1], tab[2], n);
    }
}

// ---------------------------------------------------------------------------
// Sweep 2: keys of the selected bin -> candidate list (kept in the tensor's own
// survivor segment, which the mask sweep overwrites afterwards).
__global__ void __launch_bounds__(TPB) stats2_kernel(const TensorDesc* __restrict__ descs,
                                                     TensorState* __restrict__ st, int nt, u32 tiles,
                                                     Workspace ws, int residual_median) {
    const int tid = threadIdx.x, lane = tid & 31;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0, bin1 = 0;
    u64 n = 0;
    const float *w_t = nullptr, *w_prev = nullptr;
    u32* cand = nullptr;
    for (u32 tile = lo; tile < hi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles; n = descs[cur].numel;
            w_t = descs[cur].w_t; w_prev = descs[cur].w_prev;
            bin1 = st[cur].bin1;
            cand = reinterpret_cast<u32*>(ws.surv[0] + (u64)tb * TILE);
        }
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

// Select inside the candidates and set both thresholds.
__global__ void __launch_bounds__(1024) stats2_finish_kernel(const TensorDesc* __restrict__ descs,
                                                             TensorState* __restrict__ st, Workspace ws,
                                                             float alpha, float beta) {
    __shared__ u32 hist[512];
    const int t = blockIdx.x, tid = threadIdx.x;
    TensorState& s = st[t];
    const u64 n = descs[t].numel;
    if (n == 0) {
        if (tid == 0) {
            s.median_bits = 0;
            s.thr_w = __fmul_rn(alpha, 0.f);
            s.thr_o = __fmul_rn(beta, 0.f);
        }
        return;
    }
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
        s.thr_w = __fmul_rn(alpha, __uint_as_float(bits));      // alpha * median, Eq. (rw)
        s.thr_o = __fmul_rn(beta, s.mean_abs_ea);               // beta * mean, Eq. (ro)
        if (c != s.bin_count) s.flags |= FLAG_INTERNAL;
    }
}

void launch_stats(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                  const Workspace& ws, const Params& p) {
    const int resid = p.median_source == 1;
    if (tiles) {
        const u32 grid = min(tiles, (u32)cfg.sms * 4u);
        stats1_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, resid);
    }
    stats1_finish_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st);
    prof_mark(cfg, ST_STATS1, tiles ? 2 : 1);
    if (tiles) {
        const u32 grid = min(tiles, (u32)cfg.sms * 8u);
        stats2_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, resid);
    }
    stats2_finish_kernel<<<nt, 1024, 0, cfg.stream>>>(descs, st, ws, p.alpha, p.beta);
    prof_mark(cfg, ST_STATS2, tiles ? 2 : 1);
}

}  // namespace excp
