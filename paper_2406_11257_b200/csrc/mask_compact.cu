// The one sweep over all four streams (Algorithm 1, steps 1-2):
//   dW = W_t - W^_(t-1)                                   Eq. (ckpt_res)
//   M_w = [ |dW| * sqrt(eas) > alpha * median ]           Eq. (rw), product form
//   M_o = [ |ea| > beta * mean ] and M_w                  Eq. (ro)
// and, fused with it, the bitmaps (each warp ballot is one bitmap word)
// and the compaction of the survivors: each tile's survivors are written, in
// index order, at the start of the tile's own 4096-element segment, with the
// count beside it.  No block waits for another; the tensor-wide offsets come
// from a small scan afterwards and are only needed when the codes are packed.
#include "excp_common.cuh"
#include "warp_ring.cuh"
#include <type_traits>

namespace excp {

#ifndef EXCP_MC_CH
#define EXCP_MC_CH 512
#endif
#ifndef EXCP_MC_ST
#define EXCP_MC_ST 2
#endif
#ifndef EXCP_MC_WARPS
#define EXCP_MC_WARPS 7
#endif
#ifndef EXCP_MC_BLOCKS
#define EXCP_MC_BLOCKS 2
#endif
constexpr int MCH = EXCP_MC_CH;      // values per stream per staged chunk
constexpr int MST = EXCP_MC_ST;      // chunks in flight per warp
constexpr int MWARPS = EXCP_MC_WARPS;   // 7 warps x 16 KB of stages: two blocks per SM
constexpr int MBLOCKS = EXCP_MC_BLOCKS; // resident blocks per SM
constexpr int MTPB = MWARPS * 32;

// sqrt(x) to within a few units in the last place (the hardware's approximation; its documented
// relative error is 2^-23).  Used only to decide the elements that are far from the threshold.
__device__ __forceinline__ float sqrt_fast(float x) {
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// Eq. (rw) is decided on lhs = |dW| (x) sqrt_rn(eas) in fp32.  With the approximate root the product
// differs from lhs by well under 2^-20 of its value (plus a subnormal's spacing), so outside the band
// [lo, hi] around the threshold the approximate product decides exactly as lhs would; inside it the
// warp recomputes with the correctly rounded root.
constexpr float BAND = 1.f / 262144.f;        // 2^-18
constexpr float TINY = 7.174648e-43f;         // 2^-140

struct MaskSmem {
    float buf[MWARPS][MST][4][MCH];
    unsigned long long bar[MWARPS][MST];
};

// Every warp owns a contiguous run of tiles and walks it alone: 256-value chunks of the four
// streams arrive in its ring of stages, a tile's survivor offset is a running count in the
// warp, and nothing in the sweep synchronises the block.
// VARIANT = false is the method; VARIANT = true adds the ablation switches `opt` (OPT_*), kept
// out of the method's own instruction stream.
template <bool VARIANT, typename WT>
__global__ void __launch_bounds__(MTPB, MBLOCKS) mask_compact_kernel(const TensorDesc* __restrict__ descs,
                                                              TensorState* __restrict__ st, int nt,
                                                              u32 tiles, Workspace ws, CallState* call, u32 opt, u64 wait_ns) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    MaskSmem& sm = *reinterpret_cast<MaskSmem*>(smem_raw);
    if (call_aborted(call)) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u32 lt = (1u << lane) - 1u;
    WarpRing<4, MCH, MST> ring;
    ring.init(&sm.buf[warp][0][0][0], sm.bar[warp], lane, wait_ns);

    const u32 gw = blockIdx.x * MWARPS + warp, nw = gridDim.x * MWARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    TileWalk<MCH> ic, cc;
    ic.start(wlo); cc.start(wlo);
    constexpr u32 BULK_ALIGN = sizeof(WT) == 4 ? 4u : 8u;           // values per bulk-copied unit: 16 bytes of the narrowest stream
    const float* ip[4] = {nullptr, nullptr, nullptr, nullptr};      // issue side: the tensor's moment streams ([2], [3])
    const float* cp[4] = {nullptr, nullptr, nullptr, nullptr};      // consume side
    const WT* ipw[2] = {nullptr, nullptr};                          // and its weight streams W_t, W^_(t-1)
    const WT* cpw[2] = {nullptr, nullptr};
    float thr_w = 0.f, thr_o = 0.f;
    float thr_lo = 0.f, thr_hi = 0.f;        // the band around thr_w (non-variant path)
    u32 rw = 0, ro = 0;               // survivors of the current tile so far (warp uniform)
    float mk0 = 0.f, mk1 = 0.f, mk2 = 0.f;   // running max magnitudes of the survivors
    float nanacc = 0.f;                      // turns NaN once any input is NaN or infinite
    float minv = 0.f;                        // goes negative with a negative second moment
    int prev = -1;

    auto flush_max = [&](int t) {            // non-negative floats order like their bit patterns
        const u32 m0 = __reduce_max_sync(0xffffffffu, __float_as_uint(mk0));
        const u32 m1 = __reduce_max_sync(0xffffffffu, __float_as_uint(mk1));
        const u32 m2 = __reduce_max_sync(0xffffffffu, __float_as_uint(mk2));
        if (lane == 0) {
            if (m0) atomicMax(&st[t].s[0].maxkey, m0);
            if (m1) atomicMax(&st[t].s[1].maxkey, m1);
            if (m2) atomicMax(&st[t].s[2].maxkey, m2);
        }
        mk0 = mk1 = mk2 = 0.f;
    };

    while (cc.tile < whi) {
        while (ic.tile < whi && ring.can_issue()) {
            if (ic.chunk == 0 && ic.enter_tile(descs, nt)) {
                ipw[0] = static_cast<const WT*>(descs[ic.tns].w_t); ipw[1] = static_cast<const WT*>(descs[ic.tns].w_prev);
                ip[2] = descs[ic.tns].ea; ip[3] = descs[ic.tns].eas;
                if (VARIANT && (opt & OPT_NO_RESIDUAL)) ipw[1] = nullptr;    // W^_(t-1) is not read
            }
            const u64 e0 = ic.elem0();
            const void* src[4] = {ipw[0] + e0, VARIANT && !ipw[1] ? nullptr : ipw[1] + e0, ip[2] + e0, ip[3] + e0};
            const u32 nb = ic.valid() & ~(BULK_ALIGN - 1u);
            const u32 bytes[4] = {nb * (u32)sizeof(WT), nb * (u32)sizeof(WT), nb * 4u, nb * 4u};
            ring.issue_bytes(lane, src, bytes);
            ic.next();
        }
        if (cc.chunk == 0 && cc.enter_tile(descs, nt)) {
            if (prev >= 0) flush_max(prev);
            prev = cc.tns;
            cpw[0] = static_cast<const WT*>(descs[cc.tns].w_t); cpw[1] = static_cast<const WT*>(descs[cc.tns].w_prev);
            cp[2] = descs[cc.tns].ea; cp[3] = descs[cc.tns].eas;
            thr_w = st[cc.tns].thr_w; thr_o = st[cc.tns].thr_o;
            thr_lo = __fsub_rd(__fmul_rd(thr_w, 1.f - BAND), TINY);
            thr_hi = __fadd_ru(__fmul_ru(thr_w, 1.f + BAND), TINY);
        }
        const u32 valid = cc.valid(), nbulk = valid & ~(BULK_ALIGN - 1u);
        const u64 e0 = cc.elem0();
        if (!ring.wait()) {
            if (lane == 0) atomicOr(&call->flags, FLAG_TIMEOUT);
            ring.drain();
            return;
        }
        if (cc.chunk == 0) { rw = 0; ro = 0; }
        const float* stg = ring.stage();
        const WT* stw = reinterpret_cast<const WT*>(stg);              // W_t's slot; W^_(t-1)'s starts MCH floats on
        const WT* stp = reinterpret_cast<const WT*>(stg + MCH);
        float* sw = ws.surv[0] + (u64)cc.tile * TILE;
        float* sea = ws.surv[1] + (u64)cc.tile * TILE;
        float* seas = ws.surv[2] + (u64)cc.tile * TILE;
        // Lane l takes values l, l+32, l+64, l+96 of each run of 128, so that a ballot IS a
        // bitmap word and the survivors of one ballot go to consecutive addresses.
        auto sweep_chunk = [&](auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;     // the whole chunk came by bulk copy
#pragma unroll
        for (int step = 0; step < MCH / 128; ++step) {
            if (FULL || (u32)step * 128u < valid) {
                u32 bw[4], bo[4];
                float dwv[4], eav[4], easv[4];
                bool kwv[4], kov[4];
                bool amb = false;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const u32 i = step * 128 + k * 32 + lane;
                    float a, b, e, v;
                    const bool no_prev = VARIANT && (opt & OPT_NO_RESIDUAL);
                    if (FULL || i < nbulk) {
                        a = wget(stw, i); b = no_prev ? 0.f : wget(stp, i); e = stg[2 * MCH + i]; v = stg[3 * MCH + i];
                    } else if (i < valid) {          // ragged last values of a tensor
                        a = wget(cpw[0], e0 + i); b = no_prev ? 0.f : wget(cpw[1], e0 + i);
                        e = __ldg(cp[2] + e0 + i); v = __ldg(cp[3] + e0 + i);
                    } else {
                        a = b = e = v = 0.f;
                    }
                    const float dw = no_prev ? a : __fsub_rn(a, b);              // Eq. (ckpt_res)
                    bool kw, ko;
                    if (!VARIANT) {
                        // a NaN, an infinity or a negative second moment anywhere makes the product NaN or
                        // infinite; so can finite values that overflow, which the exact check at the end tells apart
                        const float lhs = __fmul_rn(fabsf(dw), sqrt_fast(v));
                        nanacc = __fmaf_rn(lhs, 0.f, nanacc);     // inf * 0 and NaN * 0 are NaN
                        nanacc = __fmaf_rn(e, 0.f, nanacc);
                        kw = lhs > thr_hi;                                       // Eq. (rw); past numel: 0 > thr is false
                        amb |= kw != (lhs >= thr_lo);
                        ko = fabsf(e) > thr_o;                                   // Eq. (ro), before the conjunction
                    } else {
                        nanacc = __fmaf_rn(a, 0.f, nanacc);
                        nanacc = __fmaf_rn(b, 0.f, nanacc);
                        nanacc = __fmaf_rn(e, 0.f, nanacc);
                        nanacc = __fmaf_rn(v, 0.f, nanacc);
                        minv = fminf(minv, v);
                        const bool real = FULL || i < valid;
                        const float lhs = (opt & OPT_NO_M2W) ? fabsf(dw) : __fmul_rn(fabsf(dw), __fsqrt_rn(v));
                        kw = real && ((opt & OPT_NO_PRUNE) || lhs > thr_w);
                        ko = real && ((opt & OPT_NO_PRUNE) || (fabsf(e) > thr_o && ((opt & OPT_NO_W2M) || kw)));
                    }
                    kwv[k] = kw; kov[k] = ko;
                    dwv[k] = dw; eav[k] = e; easv[k] = v;
                }
                if (!VARIANT) {
                    if (__any_sync(0xffffffffu, amb)) {          // rare: some product lies next to the threshold
#pragma unroll
                        for (int k = 0; k < 4; ++k) kwv[k] = __fmul_rn(fabsf(dwv[k]), __fsqrt_rn(easv[k])) > thr_w;
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k) kov[k] = kov[k] && kwv[k];       // the joint rule
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    bw[k] = __ballot_sync(0xffffffffu, kwv[k]);
                    bo[k] = __ballot_sync(0xffffffffu, kov[k]);
                }
                if (lane < 4) {
                    const u64 wi = (u64)cc.tile * TILE_WORDS + cc.chunk * (MCH / 32) + step * 4 + lane;
                    if (EXCP_IN_BOUNDS(call, wi < (u64)tiles * TILE_WORDS)) {
                        ws.bm_w[wi] = lane == 0 ? bw[0] : lane == 1 ? bw[1] : lane == 2 ? bw[2] : bw[3];
                        ws.bm_o[wi] = lane == 0 ? bo[0] : lane == 1 ? bo[1] : lane == 2 ? bo[2] : bo[3];
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (((bw[k] >> lane) & 1u) && EXCP_IN_BOUNDS(call, rw + __popc(bw[k] & lt) < (u32)TILE)) {
                        sw[rw + __popc(bw[k] & lt)] = dwv[k];
                        mk0 = fmaxf(mk0, fabsf(dwv[k]));
                    }
                    if (((bo[k] >> lane) & 1u) && EXCP_IN_BOUNDS(call, ro + __popc(bo[k] & lt) < (u32)TILE)) {
                        const u32 po = ro + __popc(bo[k] & lt);
                        sea[po] = eav[k];
                        seas[po] = easv[k];
                        mk1 = fmaxf(mk1, fabsf(eav[k]));
                        mk2 = fmaxf(mk2, easv[k]);
                    }
                    rw += __popc(bw[k]);
                    ro += __popc(bo[k]);
                }
            }
        }
        };
        if (valid == (u32)MCH) sweep_chunk(std::true_type{});
        else sweep_chunk(std::false_type{});
        ring.release();
        if (cc.chunk == TileWalk<MCH>::CHUNKS_PER_TILE - 1 && lane == 0) {
            ws.tile_cnt_w[cc.tile] = rw;
            ws.tile_cnt_o[cc.tile] = ro;
        }
        cc.next();
    }
    if (prev >= 0) flush_max(prev);
    bool bad = (nanacc != nanacc) || (minv < 0.f);
    if (!VARIANT && __any_sync(0xffffffffu, bad)) {
        // The products went NaN or infinite somewhere in this warp's run.  Tell an invalid input from
        // finite values that overflowed: look at the inputs themselves (plain loads; this path is cold).
        bad = false;
        TileWalk<MCH> rc;
        rc.start(wlo);
        while (rc.tile < whi) {
            rc.enter_tile(descs, nt);
            const TensorDesc& d = descs[rc.tns];
            const WT* wt = static_cast<const WT*>(d.w_t);
            const WT* wp = static_cast<const WT*>(d.w_prev);
            for (u32 i = lane; i < rc.tv; i += 32) {
                const u64 el = rc.toff + i;
                const float a = wget(wt, el), b = wget(wp, el), e = d.ea[el], v = d.eas[el];
                const float z = __fmaf_rn(a, 0.f, __fmaf_rn(b, 0.f, __fmaf_rn(e, 0.f, __fmul_rn(v, 0.f))));
                bad |= (z != z) || (v < 0.f);
            }
            ++rc.tile;
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(&call->flags, FLAG_NONFINITE);
}

// Exclusive prefix of the tile counts inside each tensor; totals; the
// fixed-point scale of each stream's sums.
__global__ void __launch_bounds__(TPB) tile_scan_kernel(const TensorDesc* __restrict__ descs,
                                                        TensorState* __restrict__ st, Workspace ws,
                                                        const CallState* call) {
    if (call_aborted(call)) return;
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
    if (call_aborted(call)) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u64 bytes = 0;
    if (tid < nt) bytes = record_bytes(descs[tid].numel, st[tid].nnz_w, st[tid].nnz_o, bits);   // bits = 32: raw survivors
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
        const u32 grid = min((tiles + MWARPS - 1) / MWARPS, (u32)cfg.sms * (u32)MBLOCKS);
        const u32 opt = p.flags & (OPT_NO_W2M | OPT_NO_M2W | OPT_NO_RESIDUAL | OPT_NO_PRUNE);
        auto run = [&](auto tag) {
            using WT = decltype(tag);
            cudaFuncSetAttribute(mask_compact_kernel<false, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(MaskSmem));
            cudaFuncSetAttribute(mask_compact_kernel<true, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(MaskSmem));
            if (opt) mask_compact_kernel<true, WT><<<grid, MTPB, sizeof(MaskSmem), cfg.stream>>>(descs, st, nt, tiles, ws, call, opt, p.wait_ns);
            else mask_compact_kernel<false, WT><<<grid, MTPB, sizeof(MaskSmem), cfg.stream>>>(descs, st, nt, tiles, ws, call, 0u, p.wait_ns);
        };
        if (p.wfmt == WF_F16) run(__half{});
        else if (p.wfmt == WF_BF16) run(__nv_bfloat16{});
        else run(float{});
        prof_mark(cfg, ST_MASK_COMPACT, 1);
    }
    tile_scan_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, ws, call);
    layout_kernel<<<1, MAX_GROUP_TENSORS, 0, cfg.stream>>>(descs, st, nt, stored_bits(p), call, blob_capacity);
    prof_mark(cfg, ST_SCAN_LAYOUT, 2);
}

}  // namespace excp
