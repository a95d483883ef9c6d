// Algorithm 2 on the device: bitmap rank -> code -> centre,
//   W^_t = W^_(t-1) + C_w[I_w]   (pruned entries keep W^_(t-1) bit for bit)
//   ea^ = C_ea[I_ea], eas^ = C_eas[I_eas]   (0 where pruned)
//
// validate   one block per tensor: header fields against the layout; nothing
//            below reads a record that failed (so no read leaves the record)
// popcount   survivors per tile from the bitmaps
// scan       tensor-wide offsets; totals must equal the header's counts
// decode     per tile: word prefix in shared memory, codes staged in shared
//            memory, dense outputs
#include "excp_common.cuh"

namespace excp {

constexpr int BITS = 4;

__global__ void __launch_bounds__(64) dec_validate_kernel(const DecDesc* __restrict__ descs,
                                                          DecState* __restrict__ st, CallState* call) {
    const int t = blockIdx.x, tid = threadIdx.x;
    const DecDesc& d = descs[t];
    DecState& s = st[t];
    __shared__ u32 ok;
    if (tid == 0) {
        ok = 0;
        if (d.rec_avail >= HEADER_FIXED) {
            const u32* h = reinterpret_cast<const u32*>(d.rec);
            const u64 numel = h[2] | ((u64)h[3] << 32);
            const u64 nnz_w = h[4] | ((u64)h[5] << 32);
            const u64 nnz_o = h[6] | ((u64)h[7] << 32);
            const u64 total = h[12] | ((u64)h[13] << 32);
            if (h[0] == MAGIC && h[1] == VERSION && numel == d.numel && h[8] == BITS && h[9] == KMAX &&
                h[10] == header_bytes(KMAX) && nnz_o <= nnz_w && nnz_w <= numel &&
                total == record_bytes(numel, nnz_w, nnz_o, BITS) && total <= d.rec_avail) {
                ok = 1;
                s.bits = BITS;
                s.nnz_w = (u32)nnz_w; s.nnz_o = (u32)nnz_o;
                s.off_bm_w = header_bytes(KMAX);
                s.off_bm_o = s.off_bm_w + bitmap_bytes(numel);
                s.off_codes[0] = s.off_bm_o + bitmap_bytes(numel);
                s.off_codes[1] = s.off_codes[0] + code_bytes(nnz_w, BITS);
                s.off_codes[2] = s.off_codes[1] + code_bytes(nnz_o, BITS);
            }
        }
        s.valid = ok;
        if (!ok) atomicOr(&call->flags, FLAG_CORRUPT);
    }
    __syncthreads();
    if (ok && tid < 3 * KPAD) {
        const int k = tid / KPAD, j = tid % KPAD;
        s.cent[k][j] = j < KMAX ? reinterpret_cast<const float*>(d.rec + HEADER_FIXED)[k * KMAX + j] : 0.f;
    }
}

// Word w of tensor-local bitmap; words past the stored bitmap read as zero.
__device__ inline u32 bm_word(const unsigned char* rec, u64 off, u64 nwords, u64 w) {
    return w < nwords ? reinterpret_cast<const u32*>(rec + off)[w] : 0u;
}

__global__ void __launch_bounds__(TPB) dec_popcount_kernel(const DecDesc* __restrict__ descs,
                                                           const DecState* __restrict__ st, int nt,
                                                           u32 tiles, Workspace ws) {
    // one warp per tile
    const int lane = threadIdx.x & 31;
    const u32 tile = blockIdx.x * (TPB / 32) + (threadIdx.x >> 5);
    if (tile >= tiles) return;
    const int t = find_tensor(descs, nt, tile);
    u32 cw = 0, co = 0;
    if (st[t].valid) {
        const DecDesc& d = descs[t];
        const u64 nwords = bitmap_bytes(d.numel) / 4;
        const u64 w0 = (u64)(tile - d.tile_begin) * TILE_WORDS;
#pragma unroll
        for (int k = 0; k < TILE_WORDS / 32; ++k) {
            cw += __popc(bm_word(d.rec, st[t].off_bm_w, nwords, w0 + k * 32 + lane));
            co += __popc(bm_word(d.rec, st[t].off_bm_o, nwords, w0 + k * 32 + lane));
        }
    }
    cw = __reduce_add_sync(0xffffffffu, cw);
    co = __reduce_add_sync(0xffffffffu, co);
    if (lane == 0) { ws.tile_cnt_w[tile] = cw; ws.tile_cnt_o[tile] = co; }
}

__global__ void __launch_bounds__(TPB) dec_scan_kernel(const DecDesc* __restrict__ descs,
                                                       DecState* __restrict__ st, Workspace ws,
                                                       CallState* call) {
    const int t = blockIdx.x;
    u32 tw, to;
    scan_tile_counts(descs[t].tile_begin, descs[t].num_tiles, ws, tw, to);
    if (threadIdx.x == 0 && st[t].valid && (tw != st[t].nnz_w || to != st[t].nnz_o)) {
        st[t].valid = 0;
        atomicOr(&call->flags, FLAG_CORRUPT);
    }
}

__global__ void __launch_bounds__(TPB) decode_kernel(const DecDesc* __restrict__ descs,
                                                     const DecState* __restrict__ st, int nt, u32 tiles,
                                                     Workspace ws, CallState* call) {
    __shared__ u32 bw[TILE_WORDS], bo[TILE_WORDS];
    __shared__ u32 pw[TILE_WORDS], po[TILE_WORDS];        // survivors before each word, within the tile
    __shared__ u32 wsum[2][TILE_WORDS / 32];
    __shared__ unsigned char codes[3][TILE / 2 + 16];
    __shared__ float cent[3][KPAD];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u32 bad = 0;
    for (u32 tile = lo; tile < hi; ++tile) {
        __syncthreads();                                  // previous tile fully consumed
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            if (tid < 3 * KPAD) cent[tid / KPAD][tid % KPAD] = st[cur].cent[tid / KPAD][tid % KPAD];
        }
        if (!st[cur].valid) continue;
        const DecDesc& d = descs[cur];
        const DecState& s = st[cur];
        const u64 n = d.numel;
        const u64 nwords = bitmap_bytes(n) / 4;
        const u64 w0 = (u64)(tile - tb) * TILE_WORDS;
        const u32 cntw = ws.tile_cnt_w[tile], cnto = ws.tile_cnt_o[tile];
        const u32 offw = ws.tile_off_w[tile], offo = ws.tile_off_o[tile];
        if (tid < TILE_WORDS) {
            const u32 a = bm_word(d.rec, s.off_bm_w, nwords, w0 + tid);
            const u32 b = bm_word(d.rec, s.off_bm_o, nwords, w0 + tid);
            bw[tid] = a; bo[tid] = b;
            bad |= b & ~a;                                // a moment kept where the weight is pruned
            u32 ia = __popc(a), ib = __popc(b);
            const u32 ca = ia, cb = ib;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                u32 x = __shfl_up_sync(0xffffffffu, ia, o);
                u32 y = __shfl_up_sync(0xffffffffu, ib, o);
                if (lane >= o) { ia += x; ib += y; }
            }
            pw[tid] = ia - ca; po[tid] = ib - cb;
            if (lane == 31) { wsum[0][warp] = ia; wsum[1][warp] = ib; }
        }
        // stage the code bytes of this tile's survivors (ranks [off, off + cnt))
        {
            const unsigned char* src = d.rec + s.off_codes[0] + offw / 2;
            const u32 nb = cntw ? (offw + cntw + 1) / 2 - offw / 2 : 0;
            for (u32 i = tid; i < nb; i += TPB) codes[0][i] = src[i];
            const unsigned char* s1 = d.rec + s.off_codes[1] + offo / 2;
            const unsigned char* s2 = d.rec + s.off_codes[2] + offo / 2;
            const u32 no = cnto ? (offo + cnto + 1) / 2 - offo / 2 : 0;
            for (u32 i = tid; i < no; i += TPB) { codes[1][i] = s1[i]; codes[2][i] = s2[i]; }
        }
        __syncthreads();
        if (tid < TILE_WORDS) {
            u32 aw = 0, ao = 0;
            for (int w = 0; w < warp; ++w) { aw += wsum[0][w]; ao += wsum[1][w]; }
            pw[tid] += aw; po[tid] += ao;
        }
        __syncthreads();
        const u64 base = (u64)(tile - tb) * TILE;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const u32 e0 = r * (TPB * 4) + tid * 4;       // element within the tile
            const u64 i0 = base + e0;
            if (i0 >= n) continue;
            float wp[4];
            load4(d.w_prev, i0, n, wp);
            const u32 word = e0 >> 5, bit = e0 & 31;
            const u32 mw4 = (bw[word] >> bit) & 15u, mo4 = (bo[word] >> bit) & 15u;
            u32 rw = pw[word] + __popc(bw[word] & ((1u << bit) - 1u));
            u32 ro = po[word] + __popc(bo[word] & ((1u << bit) - 1u));
            float ow[4], oa[4], os[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                ow[k] = wp[k]; oa[k] = 0.f; os[k] = 0.f;
                if ((mw4 >> k) & 1u) {
                    const u32 g = offw + rw++;
                    const u32 c = (codes[0][(g >> 1) - (offw >> 1)] >> (4 * (g & 1u))) & 15u;
                    if (c == 0) bad = 1; else ow[k] = __fadd_rn(wp[k], cent[0][c - 1]);
                }
                if ((mo4 >> k) & 1u) {
                    const u32 g = offo + ro++;
                    const u32 ix = (g >> 1) - (offo >> 1), sh = 4 * (g & 1u);
                    const u32 c1 = (codes[1][ix] >> sh) & 15u, c2 = (codes[2][ix] >> sh) & 15u;
                    if (c1 == 0 || c2 == 0) bad = 1;
                    else { oa[k] = cent[1][c1 - 1]; os[k] = cent[2][c2 - 1]; }
                }
            }
            if (i0 + 4 <= n) {
                reinterpret_cast<float4*>(d.w_out + i0)[0] = make_float4(ow[0], ow[1], ow[2], ow[3]);
                reinterpret_cast<float4*>(d.ea_out + i0)[0] = make_float4(oa[0], oa[1], oa[2], oa[3]);
                reinterpret_cast<float4*>(d.eas_out + i0)[0] = make_float4(os[0], os[1], os[2], os[3]);
            } else {
                for (int k = 0; k < 4 && i0 + k < n; ++k) {
                    d.w_out[i0 + k] = ow[k]; d.ea_out[i0 + k] = oa[k]; d.eas_out[i0 + k] = os[k];
                }
            }
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(&call->flags, FLAG_CORRUPT);
}

void launch_decode(const LaunchCfg& cfg, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                   const Workspace& ws, CallState* call) {
    dec_validate_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, call);
    if (!tiles) { prof_mark(cfg, ST_DEC_PREP, 1); return; }
    dec_popcount_kernel<<<(tiles + TPB / 32 - 1) / (TPB / 32), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws);
    dec_scan_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, ws, call);
    prof_mark(cfg, ST_DEC_PREP, 3);
    const u32 grid = min(tiles, (u32)cfg.sms * 4u);
    decode_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, call);
    prof_mark(cfg, ST_DECODE, 1);
}

}  // namespace excp
