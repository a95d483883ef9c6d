// Non-uniform quantisation of the survivors (Section 3.3): Lloyd's algorithm in
// one dimension, K = 15 centres, per tensor and per stream.
//
//   start    K equal-mass quantiles of a seeded, index-stratified sample
//   assign   cluster(x) = #{ j : x > thr_j },  thr_j = largest fp32 not above the
//            fp64 mid-point of centres j and j+1 (so the comparison is exactly
//            "2x > c_j + c_j+1" in fp64); a 4-step binary search, no distances
//   sums     Q(x) = rint(x * 2^(30-E)) in int32, accumulated as integers: each
//            thread owns a private row of 15 shared-memory cells (48-bit sum above
//            a 16-bit count), so there are no atomics in the sweep and
//            the result is independent of the order of summation
//   update   mean = fp32(fp64(sum)/fp64(count) * 2^(E-30)); empty clusters keep
//            their centre; centres re-sorted; new thresholds
#include "excp_common.cuh"
#include "seg_ring.cuh"

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
            t = __double2float_rd(((double)s.cent[lane] + (double)s.cent[lane + 1]) * 0.5) + 0.f;   // -0 -> +0
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

// One Lloyd sweep over every tile of the group: NS = 1 for the dW stream, NS = 2 for the two
// moment streams together (they share the mask M_o, hence their tile counts).
//
// Every warp works alone on a contiguous run of tiles: lane 0 streams the tiles' survivor
// segments into the warp's own ring of shared-memory stages with bulk asynchronous copies,
// the warp consumes them as float4, and nothing in the sweep synchronises the block.
constexpr int LST = 2;               // stages per warp
constexpr int LWARPS = TPB / 32;

template <int NS, int CH>
struct LloydSmem {
    float buf[LWARPS][LST][NS][CH];
    u64 acc[NS][KMAX][TPB];          // [stream][cluster][thread]: a private cell per thread, bank = thread
    unsigned long long bar[LWARPS][LST];
    float thr[LWARPS][NS][KPAD];     // each warp's copy of its tensor's thresholds
};

template <int NS, int CH>
__global__ void __launch_bounds__(TPB, NS == 1 ? 3 : 2)
lloyd_pass_kernel(const TensorDesc* __restrict__ descs, TensorState* __restrict__ st, int nt, u32 tiles,
                  Workspace ws, int stream0, CallState* call) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    LloydSmem<NS, CH>& sm = *reinterpret_cast<LloydSmem<NS, CH>*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int k = 0; k < NS; ++k)
#pragma unroll
        for (int j = 0; j < KMAX; ++j) sm.acc[k][j][tid] = 0;

    const u32 gw = blockIdx.x * LWARPS + warp, nw = gridDim.x * LWARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    SegRing<NS, CH, LST> ring;
    ring.init(&sm.buf[warp][0][0][0], sm.bar[warp], lane, wlo, whi);
    const u32* tile_cnt = stream0 == 0 ? ws.tile_cnt_w : ws.tile_cnt_o;
    const float* surv[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) surv[k] = ws.surv[stream0 + k];

    int cur = -1;
    u32 tb = 0, ntl = 0, since = 0;
    float t3[NS], t7[NS], t11[NS], s1[NS], s2[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) t3[k] = t7[k] = t11[k] = s1[k] = s2[k] = 0.f;
    char* const cell0 = reinterpret_cast<char*>(&sm.acc[0][0][tid]);

    auto flush = [&](int tns) {      // this warp's cells -> one integer atomic per cluster
#pragma unroll
        for (int k = 0; k < NS; ++k) {
#pragma unroll
            for (int j = 0; j < KMAX; ++j) {
                const s64 v = (s64)sm.acc[k][j][tid];
                sm.acc[k][j][tid] = 0;
                s64 c, q;
                cell_split((u64)v, q, c);
#pragma unroll
                for (int o = 16; o; o >>= 1) {
                    c += __shfl_xor_sync(0xffffffffu, c, o);
                    q += __shfl_xor_sync(0xffffffffu, q, o);
                }
                if (lane == 0 && c) {
                    atomicAdd(reinterpret_cast<u64*>(&st[tns].s[stream0 + k].acc_sum[j]), (u64)q);
                    atomicAdd(&st[tns].s[stream0 + k].acc_cnt[j], (u64)c);
                }
            }
        }
        since = 0;
    };

    for (bool first = true; ring.next_window(tile_cnt, lane, first); first = false) {
        while (ring.have()) {
            ring.issue_ahead(lane, surv);
            const u32 tile = ring.tile();
            if (cur < 0 || tile >= tb + ntl) {
                if (cur >= 0) flush(cur);
                cur = find_tensor(descs, nt, tile);
                tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
                __syncwarp();
#pragma unroll
                for (int k = 0; k < NS; ++k) {
                    const StreamState& ss = st[cur].s[stream0 + k];
                    if (lane < KPAD) sm.thr[warp][k][lane] = ss.thr[lane];
                    s1[k] = ss.scale1; s2[k] = ss.scale2;
                }
                __syncwarp();
#pragma unroll
                for (int k = 0; k < NS; ++k) {
                    t3[k] = sm.thr[warp][k][3]; t7[k] = sm.thr[warp][k][7]; t11[k] = sm.thr[warp][k][11];
                }
            }
            const u32 nel = ring.nel();
            if (!ring.wait()) {
                if (lane == 0) atomicOr(&call->flags, FLAG_TIMEOUT);
                return;
            }
#pragma unroll
            for (int k = 0; k < NS; ++k) {
                const float4* b4 = reinterpret_cast<const float4*>(ring.stage() + k * CH);
                const char* thr_row = reinterpret_cast<const char*>(sm.thr[warp][k]);
                char* const cells = cell0 + k * (KMAX * TPB * 8);
                auto find = [&](float x) { return find_cluster4(x, t3[k], t7[k], t11[k], thr_row); };
                auto add = [&](u32 p, float x) {
                    const int q = __float2int_rn(__fmul_rn(__fmul_rn(x, s1[k]), s2[k]));
                    cell_add(reinterpret_cast<u64*>(cells + p * (TPB * 2u)), q);
                };
                if (nel == (u32)CH) {
                    // all searches of a batch first (they only read), then the read-modify-writes
#pragma unroll
                    for (int f = 0; f < CH / 128; f += 2) {
                        const float4 u4 = b4[lane + 32 * f], v4 = b4[lane + 32 * (f + 1)];
                        const u32 p0 = find(u4.x), p1 = find(u4.y), p2 = find(u4.z), p3 = find(u4.w);
                        const u32 p4 = find(v4.x), p5 = find(v4.y), p6 = find(v4.z), p7 = find(v4.w);
                        add(p0, u4.x); add(p1, u4.y); add(p2, u4.z); add(p3, u4.w);
                        add(p4, v4.x); add(p5, v4.y); add(p6, v4.z); add(p7, v4.w);
                    }
                } else {
                    for (u32 f = lane; 4 * f < nel; f += 32) {
                        const float4 v4 = b4[f];
                        const u32 p0 = find(v4.x), p1 = find(v4.y), p2 = find(v4.z), p3 = find(v4.w);
                        add(p0, v4.x);
                        if (4 * f + 1 < nel) add(p1, v4.y);
                        if (4 * f + 2 < nel) add(p2, v4.z);
                        if (4 * f + 3 < nel) add(p3, v4.w);
                    }
                }
            }
            ring.advance();
            if (++since >= 1024) flush(cur);
        }
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
                   const Workspace& ws, const Params& p, CallState* call) {
    kmeans_start_kernel<<<dim3(nt, 3), SAMPLE_MAX, 0, cfg.stream>>>(descs, st, ws, p.seed);
    prof_mark(cfg, ST_KMEANS_START, 1);
    if (!tiles) return;
    const u32 grid1 = min((tiles + LWARPS - 1) / LWARPS, (u32)cfg.sms * 3u);
    const u32 grid2 = min((tiles + LWARPS - 1) / LWARPS, (u32)cfg.sms * 2u);
    const size_t smem1 = sizeof(LloydSmem<1, 512>), smem2 = sizeof(LloydSmem<2, 256>);
    cudaFuncSetAttribute(lloyd_pass_kernel<1, 512>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
    cudaFuncSetAttribute(lloyd_pass_kernel<2, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
    for (int it = 0; it < p.kmeans_iters; ++it) {
        lloyd_pass_kernel<1, 512><<<grid1, TPB, smem1, cfg.stream>>>(descs, st, nt, tiles, ws, 0, call);
        prof_mark(cfg, ST_LLOYD_W, 1);
        lloyd_pass_kernel<2, 256><<<grid2, TPB, smem2, cfg.stream>>>(descs, st, nt, tiles, ws, 1, call);
        prof_mark(cfg, ST_LLOYD_EA, 1);
        kmeans_update_kernel<<<nt, 96, 0, cfg.stream>>>(st);
        prof_mark(cfg, ST_KMEANS_UPDATE, 1);
    }
}

}  // namespace excp
