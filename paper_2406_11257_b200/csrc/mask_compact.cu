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

namespace excp {

__device__ inline u32 spread8(u32 b) {   // bit i of an 8-bit value -> bit 4 i
    b = (b | (b << 12)) & 0x000F000Fu;
    b = (b | (b << 6)) & 0x03030303u;
    b = (b | (b << 3)) & 0x11111111u;
    return b;
}

__global__ void __launch_bounds__(TPB) mask_compact_kernel(const TensorDesc* __restrict__ descs,
                                                           TensorState* __restrict__ st, int nt,
                                                           u32 tiles, Workspace ws, CallState* call) {
    __shared__ u32 cnt_w[2][CHUNKS], cnt_o[2][CHUNKS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u32 lt = (1u << lane) - 1u;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u64 n = 0;
    const float *w_t = nullptr, *w_prev = nullptr, *ea = nullptr, *eas = nullptr;
    float thr_w = 0.f, thr_o = 0.f;
    u32 mk0 = 0, mk1 = 0, mk2 = 0;    // running max |x| patterns of the survivors
    u32 bad = 0;

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

    int par = 0;
    for (u32 tile = lo; tile < hi; ++tile, par ^= 1) {
        if (cur < 0 || tile >= tb + ntl) {
            if (cur >= 0) flush_max(cur);
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles; n = descs[cur].numel;
            w_t = descs[cur].w_t; w_prev = descs[cur].w_prev; ea = descs[cur].ea; eas = descs[cur].eas;
            thr_w = st[cur].thr_w; thr_o = st[cur].thr_o;
        }
        const u64 base = (u64)(tile - tb) * TILE;
        float dwv[4 * ROUNDS], eav[4 * ROUNDS], easv[4 * ROUNDS];
        u32 mw = 0, mo = 0;                 // this thread's 16 mask bits
        u32 prew[ROUNDS], preo[ROUNDS];     // survivors before this lane within its chunk
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const u64 i0 = base + (u64)r * (TPB * 4) + (u64)tid * 4;
            float a[4], b[4], e[4], v[4];
            load4(w_t, i0, n, a);
            load4(w_prev, i0, n, b);
            load4(ea, i0, n, e);
            load4(eas, i0, n, v);
            u32 bw[4], bo[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const u32 vb = __float_as_uint(v[k]);
                bad |= ((__float_as_uint(a[k]) & 0x7fffffffu) >= 0x7f800000u) |
                       ((__float_as_uint(b[k]) & 0x7fffffffu) >= 0x7f800000u) |
                       ((__float_as_uint(e[k]) & 0x7fffffffu) >= 0x7f800000u) |
                       ((vb & 0x7fffffffu) >= 0x7f800000u) | (vb > 0x80000000u);
                const float dw = __fsub_rn(a[k], b[k]);
                const float lhs = __fmul_rn(fabsf(dw), __fsqrt_rn(v[k]));
                const bool kw = lhs > thr_w;                       // elements past numel: 0 > thr is false
                const bool ko = kw && (fabsf(e[k]) > thr_o);
                bw[k] = __ballot_sync(0xffffffffu, kw);
                bo[k] = __ballot_sync(0xffffffffu, ko);
                dwv[r * 4 + k] = dw; eav[r * 4 + k] = e[k]; easv[r * 4 + k] = v[k];
                mw |= (u32)kw << (r * 4 + k);
                mo |= (u32)ko << (r * 4 + k);
            }
            prew[r] = __popc(bw[0] & lt) + __popc(bw[1] & lt) + __popc(bw[2] & lt) + __popc(bw[3] & lt);
            preo[r] = __popc(bo[0] & lt) + __popc(bo[1] & lt) + __popc(bo[2] & lt) + __popc(bo[3] & lt);
            const int chunk = r * (TPB / 32) + warp;
            if (lane < 4) {   // lane j assembles bitmap word j of this 128-element chunk
                const int sh = 8 * lane;
                const u32 ww = spread8((bw[0] >> sh) & 0xffu) | (spread8((bw[1] >> sh) & 0xffu) << 1) |
                               (spread8((bw[2] >> sh) & 0xffu) << 2) | (spread8((bw[3] >> sh) & 0xffu) << 3);
                const u32 wo = spread8((bo[0] >> sh) & 0xffu) | (spread8((bo[1] >> sh) & 0xffu) << 1) |
                               (spread8((bo[2] >> sh) & 0xffu) << 2) | (spread8((bo[3] >> sh) & 0xffu) << 3);
                const u64 wi = (u64)tile * TILE_WORDS + chunk * 4 + lane;
                ws.bm_w[wi] = ww;
                ws.bm_o[wi] = wo;
            }
            if (lane == 0) {
                cnt_w[par][chunk] = __popc(bw[0]) + __popc(bw[1]) + __popc(bw[2]) + __popc(bw[3]);
                cnt_o[par][chunk] = __popc(bo[0]) + __popc(bo[1]) + __popc(bo[2]) + __popc(bo[3]);
            }
        }
        __syncthreads();
        if (warp == 0) {      // exclusive prefix over the 32 chunks, in element order
            u32 cw = cnt_w[par][lane], co = cnt_o[par][lane];
            u32 iw = cw, io = co;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                u32 x = __shfl_up_sync(0xffffffffu, iw, o);
                u32 y = __shfl_up_sync(0xffffffffu, io, o);
                if (lane >= o) { iw += x; io += y; }
            }
            cnt_w[par][lane] = iw - cw;
            cnt_o[par][lane] = io - co;
            if (lane == 31) { ws.tile_cnt_w[tile] = iw; ws.tile_cnt_o[tile] = io; }
        }
        __syncthreads();
        float* sw = ws.surv[0] + (u64)tile * TILE;
        float* sea = ws.surv[1] + (u64)tile * TILE;
        float* seas = ws.surv[2] + (u64)tile * TILE;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const int chunk = r * (TPB / 32) + warp;
            u32 pw = cnt_w[par][chunk] + prew[r];
            u32 po = cnt_o[par][chunk] + preo[r];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int j = r * 4 + k;
                if ((mw >> j) & 1u) {
                    sw[pw++] = dwv[j];
                    mk0 = max(mk0, __float_as_uint(dwv[j]) & 0x7fffffffu);
                }
                if ((mo >> j) & 1u) {
                    sea[po] = eav[j];
                    seas[po] = easv[j];
                    ++po;
                    mk1 = max(mk1, __float_as_uint(eav[j]) & 0x7fffffffu);
                    mk2 = max(mk2, __float_as_uint(easv[j]) & 0x7fffffffu);
                }
            }
        }
    }
    if (cur >= 0) flush_max(cur);
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
        const u32 grid = min(tiles, (u32)cfg.sms * 4u);
        mask_compact_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, call);
        prof_mark(cfg, ST_MASK_COMPACT, 1);
    }
    tile_scan_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, ws);
    layout_kernel<<<1, MAX_GROUP_TENSORS, 0, cfg.stream>>>(descs, st, nt, p.bits, call, blob_capacity);
    prof_mark(cfg, ST_SCAN_LAYOUT, 2);
}

}  // namespace excp
