// Non-uniform quantisation of the survivors (Section 3.3): Lloyd's algorithm in
// one dimension, K = 15 centres, per tensor and per stream.
//
//   start    K equal-mass quantiles of a seeded, index-stratified sample
//   assign   cluster(x) = #{ j : x > thr_j },  thr_j = largest fp32 not above the
//            fp64 mid-point of centres j and j+1 (so the comparison is exactly
//            "2x > c_j + c_j+1" in fp64); a 4-step binary search, no distances
//   sums     Q(x) = rint(x * 2^(30-E)) in int32, accumulated as integers: each
//            thread owns a private row of 16 shared-memory cells (count in the
//            top 16 bits, sum below), so there are no atomics in the sweep and
//            the result is independent of the order of summation
//   update   mean = fp32(fp64(sum)/fp64(count) * 2^(E-30)); empty clusters keep
//            their centre; centres re-sorted; new thresholds
#include "excp_common.cuh"

namespace excp {

__device__ inline u64 mix64(u64 z) {   // SplitMix64 output function
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ inline void set_thresholds(StreamState& s, int lane) {
    // lanes 0..15 of one warp; centres already final and sorted
    if (lane < KPAD) {
        float t = __uint_as_float(0x7f800000u);
        if (lane < KMAX - 1)
            t = __double2float_rd(((double)s.cent[lane] + (double)s.cent[lane + 1]) * 0.5);
        s.thr[lane] = t;
    }
}

// One block per (tensor, stream).
__global__ void __launch_bounds__(SAMPLE_MAX) kmeans_start_kernel(const TensorDesc* __restrict__ descs,
                                                                  TensorState* __restrict__ st,
                                                                  Workspace ws, u64 seed) {
    __shared__ float smp[SAMPLE_MAX];
    const int t = blockIdx.x, stream = blockIdx.y, tid = threadIdx.x;
    StreamState& s = st[t].s[stream];
    const u32 nnz = stream == 0 ? st[t].nnz_w : st[t].nnz_o;
    const u32 tb = descs[t].tile_begin, ntl = descs[t].num_tiles;
    const u32* toff = (stream == 0 ? ws.tile_off_w : ws.tile_off_o) + tb;
    const float* data = ws.surv[stream] + (u64)tb * TILE;
    if (tid < KPAD) { s.acc_sum[tid] = 0; s.acc_cnt[tid] = 0; }
    if (nnz == 0) {
        if (tid < KPAD) { s.cent[tid] = 0.f; s.thr[tid] = __uint_as_float(0x7f800000u); }
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
    __syncthreads();
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
    if (tid < KPAD) s.cent[tid] = tid < KMAX ? smp[((2 * tid + 1) * m) / (2 * KMAX)] : 0.f;
    __syncthreads();
    if (tid < 32) set_thresholds(s, tid);
}

// One Lloyd sweep of one stream over every tile of the group.
__global__ void __launch_bounds__(TPB) lloyd_pass_kernel(const TensorDesc* __restrict__ descs,
                                                         TensorState* __restrict__ st, int nt, u32 tiles,
                                                         const float* __restrict__ surv,
                                                         const u32* __restrict__ tile_cnt, int stream) {
    __shared__ u64 acc[KPAD][TPB];       // [cluster][thread]: bank = thread, conflict free
    __shared__ float thr[KPAD];
    __shared__ s64 red_sum[8][KPAD];
    __shared__ u32 red_cnt[8][KPAD];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int j = 0; j < KPAD; ++j) acc[j][tid] = 0;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    float s1 = 0.f, s2 = 0.f;
    int since = 0;

    auto flush = [&](int t) {
        // per-thread cells -> block totals -> one integer atomic per cluster
#pragma unroll
        for (int j = 0; j < KMAX; ++j) {
            const s64 v = (s64)acc[j][tid];
            acc[j][tid] = 0;
            s64 c = (v + (1ll << 47)) >> 48;          // count sits above a 48-bit signed sum
            s64 sm = v - (c << 48);
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                c += __shfl_xor_sync(0xffffffffu, c, o);
                sm += __shfl_xor_sync(0xffffffffu, sm, o);
            }
            if (lane == 0) { red_sum[warp][j] = sm; red_cnt[warp][j] = (u32)c; }
        }
        __syncthreads();
        if (tid < KMAX) {
            s64 sm = 0; u64 c = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) { sm += red_sum[w][tid]; c += red_cnt[w][tid]; }
            if (c) {
                atomicAdd(reinterpret_cast<u64*>(&st[t].s[stream].acc_sum[tid]), (u64)sm);
                atomicAdd(&st[t].s[stream].acc_cnt[tid], c);
            }
        }
        __syncthreads();
        since = 0;
    };

    for (u32 tile = lo; tile < hi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            if (cur >= 0) flush(cur);
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            const StreamState& s = st[cur].s[stream];
            __syncthreads();
            if (tid < KPAD) thr[tid] = s.thr[tid];
            s1 = s.scale1; s2 = s.scale2;
            __syncthreads();
        }
        const u32 cnt = tile_cnt[tile];
        const float* data = surv + (u64)tile * TILE;
        for (u32 i = tid; i < cnt; i += TPB) {
            const float x = data[i];
            int p = (x > thr[7]) ? 8 : 0;
            p += (x > thr[p + 3]) ? 4 : 0;
            p += (x > thr[p + 1]) ? 2 : 0;
            p += (x > thr[p]) ? 1 : 0;
            const int q = __float2int_rn(__fmul_rn(__fmul_rn(x, s1), s2));
            acc[p][tid] += (u64)((s64)q + (1ll << 48));
        }
        if (++since >= 1024) flush(cur);
    }
    if (cur >= 0) flush(cur);
}

// New centres from the sums of the finished sweep; one block per tensor, one
// warp per stream.
__global__ void __launch_bounds__(96) kmeans_update_kernel(TensorState* __restrict__ st) {
    const int t = blockIdx.x, stream = threadIdx.x >> 5, lane = threadIdx.x & 31;
    StreamState& s = st[t].s[stream];
    float c = __uint_as_float(0x7f800000u);
    if (lane < KMAX) {
        c = s.cent[lane];
        const u64 n = s.acc_cnt[lane];
        if (n) {
            const double mean = __ll2double_rn(s.acc_sum[lane]) / __ull2double_rn(n);
            const double scale = __longlong_as_double((s64)(s.e - 30 + 1023) << 52);
            c = __double2float_rn(mean * scale);
        }
        s.acc_sum[lane] = 0;
        s.acc_cnt[lane] = 0;
    }
    // sort ascending: rank of each centre among the 15 (ties by lane)
    int rank = 0;
    for (int j = 0; j < KMAX; ++j) {
        const float o = __shfl_sync(0xffffffffu, c, j);
        rank += (o < c) || (o == c && j < lane);
    }
    __syncwarp();
    if (lane < KMAX) s.cent[rank] = c;
    __syncwarp();
    set_thresholds(s, lane);
}

void launch_kmeans(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                   const Workspace& ws, const Params& p) {
    kmeans_start_kernel<<<dim3(nt, 3), SAMPLE_MAX, 0, cfg.stream>>>(descs, st, ws, p.seed);
    prof_mark(cfg, ST_KMEANS_START, 1);
    if (!tiles) return;
    const u32 grid = min(tiles, (u32)cfg.sms * 4u);
    for (int it = 0; it < p.kmeans_iters; ++it) {
        lloyd_pass_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws.surv[0], ws.tile_cnt_w, 0);
        prof_mark(cfg, ST_LLOYD_W, 1);
        lloyd_pass_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws.surv[1], ws.tile_cnt_o, 1);
        prof_mark(cfg, ST_LLOYD_EA, 1);
        lloyd_pass_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws.surv[2], ws.tile_cnt_o, 2);
        prof_mark(cfg, ST_LLOYD_EAS, 1);
        kmeans_update_kernel<<<nt, 96, 0, cfg.stream>>>(st);
        prof_mark(cfg, ST_KMEANS_UPDATE, 1);
    }
}

}  // namespace excp
