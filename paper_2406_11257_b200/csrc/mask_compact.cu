// The one sweep over all four streams (Algorithm 1, steps 1-2):
//   dW = W_t - W^_(t-1)                                   Eq. (ckpt_res)
//   M_w = [ |dW| * sqrt(eas) > alpha * median ]           Eq. (rw), product form
//   M_o = [ |ea| > beta * mean ] and M_w                  Eq. (ro)
// and, fused with it, the bitmaps (warp ballots re-ordered to element order)
// and the compaction of the survivors: each tile's survivors are written, in
// index order, at the start of the tile's own 4096-element segment, with the
// count beside it.  No block waits for another; the tensor-wide offsets come
// from a small scan afterwards and are only needed when the codes are packed.
#include "excp_common.cuh"
#include "warp_ring.cuh"

namespace excp {

__device__ inline u32 spread8(u32 b) {   // bit i of an 8-bit value -> bit 4 i
    b = (b | (b << 12)) & 0x000F000Fu;
    b = (b | (b << 6)) & 0x03030303u;
    b = (b | (b << 3)) & 0x11111111u;
    return b;
}

constexpr int MCH = 256;             // values per stream per staged chunk
constexpr int MST = 3;               // chunks in flight per warp
constexpr int MWARPS = TPB / 32;

struct MaskSmem {
    float buf[MWARPS][MST][4][MCH];
    unsigned long long bar[MWARPS][MST];
};

// Every warp owns a contiguous run of tiles and walks it alone: 256-value chunks of the four
// streams arrive in its ring of stages, a tile's survivor offset is a running count in the
// warp, and nothing in the sweep synchronises the block.
__global__ void __launch_bounds__(TPB, 2) mask_compact_kernel(const TensorDesc* __restrict__ descs,
                                                              TensorState* __restrict__ st, int nt,
                                                              u32 tiles, Workspace ws, CallState* call) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    MaskSmem& sm = *reinterpret_cast<MaskSmem*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u32 lt = (1u << lane) - 1u;
    WarpRing<4, MCH, MST> ring;
    ring.init(&sm.buf[warp][0][0][0], sm.bar[warp], lane);

    const u32 gw = blockIdx.x * MWARPS + warp, nw = gridDim.x * MWARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    DenseCursor<MCH> ic, cc;
    ic.start(wlo); cc.start(wlo);
    const float* ip[4] = {nullptr, nullptr, nullptr, nullptr};      // issue side: the tensor's streams
    const float* cp[4] = {nullptr, nullptr, nullptr, nullptr};      // consume side
    float thr_w = 0.f, thr_o = 0.f;
    u32 rw = 0, ro = 0;               // survivors of the current tile so far (warp uniform)
    u32 mk0 = 0, mk1 = 0, mk2 = 0;    // running max |x| patterns of the survivors
    u32 bad = 0;
    int prev = -1;

    auto flush_max = [&](int t) {
        mk0 = __reduce_max_sync(0xffffffffu, mk0);
        mk1 = __reduce_max_sync(0xffffffffu, mk1);
        mk2 = __reduce_max_sync(0xffffffffu, mk2);
        if (lane == 0) {
            if (mk0) atomicMax(&st[t].s[0].maxkey, mk0);
            if (mk1) atomicMax(&st[t].s[1].maxkey, mk1);
            if (mk2) atomicMax(&st[t].s[2].maxkey, mk2);
        }
        mk0 = mk1 = mk2 = 0;
    };

    while (cc.tile < whi) {
        while (ic.tile < whi && ring.can_issue()) {
            if (ic.locate(descs, nt)) {
                ip[0] = descs[ic.tns].w_t; ip[1] = descs[ic.tns].w_prev;
                ip[2] = descs[ic.tns].ea; ip[3] = descs[ic.tns].eas;
            }
            const u64 e0 = ic.elem0();
            const float* src[4] = {ip[0] + e0, ip[1] + e0, ip[2] + e0, ip[3] + e0};
            ring.issue(lane, src, ic.valid() & ~3u);
            ic.next();
        }
        if (cc.locate(descs, nt)) {
            if (prev >= 0) flush_max(prev);
            prev = cc.tns;
            cp[0] = descs[cc.tns].w_t; cp[1] = descs[cc.tns].w_prev;
            cp[2] = descs[cc.tns].ea; cp[3] = descs[cc.tns].eas;
            thr_w = st[cc.tns].thr_w; thr_o = st[cc.tns].thr_o;
        }
        const u32 valid = cc.valid(), nbulk = valid & ~3u;
        const u64 e0 = cc.elem0();
        if (!ring.wait()) {
            if (lane == 0) atomicOr(&call->flags, FLAG_TIMEOUT);
            return;
        }
        if (cc.chunk == 0) { rw = 0; ro = 0; }
        const float* stg = ring.stage();
        float* sw = ws.surv[0] + (u64)cc.tile * TILE;
        float* sea = ws.surv[1] + (u64)cc.tile * TILE;
        float* seas = ws.surv[2] + (u64)cc.tile * TILE;
#pragma unroll
        for (int step = 0; step < MCH / 128; ++step) {
            if ((u32)step * 128u < valid) {
                const u32 o = step * 128 + lane * 4;
                float a[4], b[4], e[4], v[4];
                fetch4(stg, cp[0] + e0, o, nbulk, valid, a);
                fetch4(stg + MCH, cp[1] + e0, o, nbulk, valid, b);
                fetch4(stg + 2 * MCH, cp[2] + e0, o, nbulk, valid, e);
                fetch4(stg + 3 * MCH, cp[3] + e0, o, nbulk, valid, v);
                u32 bw[4], bo[4];
                float dwv[4];
                u32 mw = 0, mo = 0;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const u32 vb = __float_as_uint(v[k]);
                    bad |= ((__float_as_uint(a[k]) & 0x7fffffffu) >= 0x7f800000u) |
                           ((__float_as_uint(b[k]) & 0x7fffffffu) >= 0x7f800000u) |
                           ((__float_as_uint(e[k]) & 0x7fffffffu) >= 0x7f800000u) |
                           ((vb & 0x7fffffffu) >= 0x7f800000u) | (vb > 0x80000000u);
                    const float dw = __fsub_rn(a[k], b[k]);                      // Eq. (ckpt_res)
                    const float lhs = __fmul_rn(fabsf(dw), __fsqrt_rn(v[k]));
                    const bool kw = lhs > thr_w;                                 // Eq. (rw); past numel: 0 > thr is false
                    const bool ko = kw && (fabsf(e[k]) > thr_o);                 // Eq. (ro)
                    bw[k] = __ballot_sync(0xffffffffu, kw);
                    bo[k] = __ballot_sync(0xffffffffu, ko);
                    dwv[k] = dw;
                    mw |= (u32)kw << k;
                    mo |= (u32)ko << k;
                }
                if (lane < 4) {   // lane j assembles bitmap word j of these 128 values
                    const int sh = 8 * lane;
                    const u32 ww = spread8((bw[0] >> sh) & 0xffu) | (spread8((bw[1] >> sh) & 0xffu) << 1) |
                                   (spread8((bw[2] >> sh) & 0xffu) << 2) | (spread8((bw[3] >> sh) & 0xffu) << 3);
                    const u32 wo = spread8((bo[0] >> sh) & 0xffu) | (spread8((bo[1] >> sh) & 0xffu) << 1) |
                                   (spread8((bo[2] >> sh) & 0xffu) << 2) | (spread8((bo[3] >> sh) & 0xffu) << 3);
                    const u64 wi = (u64)cc.tile * TILE_WORDS + cc.chunk * (MCH / 32) + step * 4 + lane;
                    ws.bm_w[wi] = ww;
                    ws.bm_o[wi] = wo;
                }
                u32 pw = rw + __popc(bw[0] & lt) + __popc(bw[1] & lt) + __popc(bw[2] & lt) + __popc(bw[3] & lt);
                u32 po = ro + __popc(bo[0] & lt) + __popc(bo[1] & lt) + __popc(bo[2] & lt) + __popc(bo[3] & lt);
                rw += __popc(bw[0]) + __popc(bw[1]) + __popc(bw[2]) + __popc(bw[3]);
                ro += __popc(bo[0]) + __popc(bo[1]) + __popc(bo[2]) + __popc(bo[3]);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if ((mw >> k) & 1u) {
                        sw[pw++] = dwv[k];
                        mk0 = max(mk0, __float_as_uint(dwv[k]) & 0x7fffffffu);
                    }
                    if ((mo >> k) & 1u) {
                        sea[po] = e[k];
                        seas[po] = v[k];
                        ++po;
                        mk1 = max(mk1, __float_as_uint(e[k]) & 0x7fffffffu);
                        mk2 = max(mk2, __float_as_uint(v[k]) & 0x7fffffffu);
                    }
                }
            }
        }
        ring.release();
        if (cc.chunk == DenseCursor<MCH>::CHUNKS_PER_TILE - 1 && lane == 0) {
            ws.tile_cnt_w[cc.tile] = rw;
            ws.tile_cnt_o[cc.tile] = ro;
        }
        cc.next();
    }
    if (prev >= 0) flush_max(prev);
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(&call->flags, FLAG_NONFINITE);
}

// Exclusive prefix of the tile counts inside each tensor; totals; the
// fixed-point scale of each stream's sums.
__global__ void __launch_bounds__(TPB) tile_scan_kernel(const TensorDesc* __restrict__ descs,
                                                        TensorState* __restrict__ st, Workspace ws) {
    const int t = blockIdx.x, tid = threadIdx.x;
    u32 carry_w, carry_o;
    scan_tile_counts(descs[t].tile_begin, descs[t].num_tiles, ws, carry_w, carry_o);
    if (tid == 0) { st[t].nnz_w = carry_w; st[t].nnz_o = carry_o; }
    if (tid < 3) {
        StreamState& s = st[t].s[tid];
        const u32 mk = s.maxkey;
        const int e = mk ? max((int)(mk >> 23), 1) - 127 : 0;   // floor(log2(max)), not below -126
        const int sc = 30 - e;                                  // 2^sc as two exact factors
        const int s1 = sc >> 1, s2 = sc - s1;
        s.e = e;
        s.scale1 = __uint_as_float((u32)(s1 + 127) << 23);
        s.scale2 = __uint_as_float((u32)(s2 + 127) << 23);
    }
}

// Record sizes -> record offsets in the blob (prefix over the group's tensors,
// continuing from the previous group), capacity check.
__global__ void __launch_bounds__(MAX_GROUP_TENSORS) layout_kernel(const TensorDesc* __restrict__ descs,
                                                                   TensorState* __restrict__ st, int nt,
                                                                   int bits, CallState* call,
                                                                   u64 blob_capacity) {
    __shared__ u64 wtot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u64 bytes = 0;
    if (tid < nt) bytes = record_bytes(descs[tid].numel, st[tid].nnz_w, st[tid].nnz_o, bits);
    u64 incl = bytes;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        u64 x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
    }
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    u64 base = 0, total = 0;
    for (int w = 0; w < 32; ++w) {
        if (w < warp) base += wtot[w];
        total += wtot[w];
    }
    const u64 cursor = call->blob_cursor;
    __syncthreads();
    if (tid < nt) {
        st[tid].blob_off = cursor + base + incl - bytes;
        st[tid].blob_bytes = bytes;
    }
    if (tid == 0) {
        call->blob_cursor = cursor + total;
        if (cursor + total > blob_capacity) call->flags |= FLAG_BLOB_FULL;
    }
}

void launch_mask_compact(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                         const Workspace& ws, const Params& p, CallState* call, u64 blob_capacity) {
    if (tiles) {
        const u32 grid = min((tiles + MWARPS - 1) / MWARPS, (u32)cfg.sms * 2u);
        cudaFuncSetAttribute(mask_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(MaskSmem));
        mask_compact_kernel<<<grid, TPB, sizeof(MaskSmem), cfg.stream>>>(descs, st, nt, tiles, ws, call);
        prof_mark(cfg, ST_MASK_COMPACT, 1);
    }
    tile_scan_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, ws);
    layout_kernel<<<1, MAX_GROUP_TENSORS, 0, cfg.stream>>>(descs, st, nt, p.bits, call, blob_capacity);
    prof_mark(cfg, ST_SCAN_LAYOUT, 2);
}

}  // namespace excp
