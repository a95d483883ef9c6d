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
            const u32 rf = h[11];                         // REC_*: what the record says about itself
            const int bits = (int)h[8];
            const bool width_ok = (rf & REC_RAW) ? bits == 32 : (bits == 2 || bits == 4 || bits == 8);
            const int kc = width_ok ? centres_of(bits) : 0;
            if (width_ok && h[0] == MAGIC && h[1] == VERSION && numel == d.numel && !(rf & ~REC_ALL) && h[8] == (u32)bits &&
                h[9] == (u32)kc && h[10] == header_bytes(kc) && (nnz_o <= nnz_w || (rf & REC_MOMENTS_FREE)) &&
                nnz_w <= numel && nnz_o <= numel &&
                total == record_bytes(numel, nnz_w, nnz_o, bits) && total <= d.rec_avail) {
                ok = 1;
                s.bits = bits;
                s.rflags = rf;
                s.nnz_w = (u32)nnz_w; s.nnz_o = (u32)nnz_o;
                s.off_bm_w = header_bytes(kc);
                s.off_bm_o = s.off_bm_w + bitmap_bytes(numel);
                s.off_codes[0] = s.off_bm_o + bitmap_bytes(numel);
                s.off_codes[1] = s.off_codes[0] + code_bytes(nnz_w, bits);
                s.off_codes[2] = s.off_codes[1] + code_bytes(nnz_o, bits);
            }
        }
        s.valid = ok;
        if (!ok) atomicOr(&call->flags, FLAG_CORRUPT);
    }
    __syncthreads();
    if (ok) {
        const int kc = centres_of((int)s.bits);           // 0: a raw record carries no centres
        for (int i = tid; i < 3 * KCAP; i += 64) {
            const int k = i / KCAP, j = i % KCAP;
            s.cent[k][j] = j < kc ? reinterpret_cast<const float*>(d.rec + HEADER_FIXED)[k * kc + j] : 0.f;
        }
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

// DENSE = false: Algorithm 2.  DENSE = true: the same walk writes each element's code (0 where
// pruned) into the three sections of the dense layout instead.
//
// Warps are autonomous: a warp owns a contiguous run of tiles and nothing synchronises the block.
// Per tile the warp loads the 2 x 128 bitmap words, turns their populations into the rank of
// every word's first survivor (registers and shuffles), parks words and ranks in its own corner
// of shared memory, and then walks the tile in 32 rounds of 128 elements, lane l taking four
// consecutive elements: their survivors have consecutive ranks, so their codes are consecutive
// bits of the section and one 32-bit window per stream (two aligned words read through the
// cache) holds all four.
constexpr int DEC_WARPS = TPB / 32;

struct DecodeSmem {
    u32 bw[DEC_WARPS][TILE_WORDS], bo[DEC_WARPS][TILE_WORDS];   // the tile's bitmap words
    u32 pw[DEC_WARPS][TILE_WORDS], po[DEC_WARPS][TILE_WORDS];   // survivors of the tile before each word
    float cent[DEC_WARPS][3][KCAP];
};

// The `nb`-bit codes of up to four consecutive survivors starting at rank g of a section:
// bits [g * nb, g * nb + 32) of it.  Words are read only where codes of these `have` survivors lie.
__device__ __forceinline__ u32 code_window(const u32* __restrict__ sec, u64 g, u32 nb, u32 have) {
    if (!have) return 0u;
    const u64 bit = g * nb;
    const u32 sh = (u32)bit & 31u;
    const u32 lo = __ldg(sec + (bit >> 5));
    const u32 hi = sh + have * nb > 32u ? __ldg(sec + (bit >> 5) + 1) : 0u;
    return __funnelshift_r(lo, hi, sh);
}

template <bool DENSE, typename WT>
__global__ void __launch_bounds__(TPB) decode_kernel(const DecDesc* __restrict__ descs,
                                                     const DecState* __restrict__ st, int nt, u32 tiles,
                                                     Workspace ws, CallState* call) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecodeSmem& sm = *reinterpret_cast<DecodeSmem*>(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u32 gw = blockIdx.x * DEC_WARPS + warp, nw = gridDim.x * DEC_WARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    u32* bw = sm.bw[warp]; u32* bo = sm.bo[warp]; u32* pw = sm.pw[warp]; u32* po = sm.po[warp];
    float (*cent)[KCAP] = sm.cent[warp];
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u32 bad = 0;
    for (u32 tile = wlo; tile < whi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            __syncwarp();
            if (st[cur].valid) {
                const int kc = centres_of((int)st[cur].bits);
                for (int i = lane; i < 3 * kc; i += 32) cent[i / kc][i % kc] = st[cur].cent[i / kc][i % kc];
            }
            __syncwarp();
        }
        if (!st[cur].valid) continue;
        const DecDesc& d = descs[cur];
        const DecState& s = st[cur];
        const WT* w_prev = static_cast<const WT*>(d.w_prev);
        WT* w_out = static_cast<WT*>(d.w_out);
        const u64 n = d.numel;
        const u64 nwords = bitmap_bytes(n) / 4;
        const u64 w0 = (u64)(tile - tb) * TILE_WORDS;
        const u32 offw = ws.tile_off_w[tile], offo = ws.tile_off_o[tile];
        {   // lane l holds words 4l .. 4l+3 of both bitmaps; ranks by a scan over the lanes
            u32 a[4], b[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                a[k] = bm_word(d.rec, s.off_bm_w, nwords, w0 + 4 * lane + k);
                b[k] = bm_word(d.rec, s.off_bm_o, nwords, w0 + 4 * lane + k);
                if (!(s.rflags & REC_MOMENTS_FREE)) bad |= b[k] & ~a[k];   // a moment kept where the weight is pruned
            }
            if ((u64)(tile - tb + 1) * TILE > n) {        // the tensor ends in this tile: no bit at or past its last element
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const u64 e = (w0 + 4 * lane + k) * 32;                 // first element of the word
                    const u32 stray = e >= n ? 0xffffffffu : (n - e >= 32 ? 0u : 0xffffffffu << (u32)(n - e));
                    bad |= (a[k] | b[k]) & stray;
                }
            }
            const u32 ta = __popc(a[0]) + __popc(a[1]) + __popc(a[2]) + __popc(a[3]);
            const u32 tbm = __popc(b[0]) + __popc(b[1]) + __popc(b[2]) + __popc(b[3]);
            u32 ia = ta, ib = tbm;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const u32 x = __shfl_up_sync(0xffffffffu, ia, o), y = __shfl_up_sync(0xffffffffu, ib, o);
                if (lane >= o) { ia += x; ib += y; }
            }
            u32 ra = ia - ta, rb = ib - tbm;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                bw[4 * lane + k] = a[k]; bo[4 * lane + k] = b[k];
                pw[4 * lane + k] = ra; po[4 * lane + k] = rb;
                ra += __popc(a[k]); rb += __popc(b[k]);
            }
        }
        __syncwarp();
        const bool raw = s.rflags & REC_RAW;              // sections hold fp32 survivors
        const bool absolute = s.rflags & REC_ABSOLUTE;    // the weight stream is W itself
        const u32 nb = raw ? 32u : s.bits;
        const u32 cmask = raw ? 0xffffffffu : (1u << nb) - 1u;
        const u32* sec0 = reinterpret_cast<const u32*>(d.rec + s.off_codes[0]);
        const u32* sec1 = reinterpret_cast<const u32*>(d.rec + s.off_codes[1]);
        const u32* sec2 = reinterpret_cast<const u32*>(d.rec + s.off_codes[2]);
        const u64 base = (u64)(tile - tb) * TILE;
#pragma unroll 2
        for (int r = 0; r < TILE / 128; ++r) {
            const u32 e0 = r * 128 + lane * 4;            // element within the tile
            const u64 i0 = base + e0;
            const bool live = i0 < n;
            if (!DENSE && !__any_sync(0xffffffffu, live)) break;
            float wp[4] = {0.f, 0.f, 0.f, 0.f};
            if (!DENSE && !absolute && live) load4(w_prev, i0, n, wp);
            const u32 word = e0 >> 5, bit = e0 & 31;
            const u32 mw4 = (bw[word] >> bit) & 15u, mo4 = (bo[word] >> bit) & 15u;
            const u64 gw0 = (u64)offw + pw[word] + __popc(bw[word] & ((1u << bit) - 1u));
            const u64 go0 = (u64)offo + po[word] + __popc(bo[word] & ((1u << bit) - 1u));
            float ow[4], oa[4], os[4];
            u32 nib0 = 0, nib1 = 0, nib2 = 0;             // DENSE: the four codes per stream
            if (!raw) {
                u32 win0 = code_window(sec0, gw0, nb, __popc(mw4));
                u32 win1 = code_window(sec1, go0, nb, __popc(mo4));
                u32 win2 = code_window(sec2, go0, nb, __popc(mo4));
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    ow[k] = wp[k]; oa[k] = 0.f; os[k] = 0.f;
                    if ((mw4 >> k) & 1u) {
                        const u32 c = win0 & cmask;
                        win0 >>= nb;
                        if (c == 0) bad = 1; else ow[k] = __fadd_rn(wp[k], cent[0][c - 1]);
                        nib0 |= c << (4 * k);
                    }
                    if ((mo4 >> k) & 1u) {
                        const u32 c1 = win1 & cmask, c2 = win2 & cmask;
                        win1 >>= nb; win2 >>= nb;
                        if (c1 == 0 || c2 == 0) bad = 1;
                        else { oa[k] = cent[1][c1 - 1]; os[k] = cent[2][c2 - 1]; }
                        nib1 |= c1 << (4 * k);
                        nib2 |= c2 << (4 * k);
                    }
                }
            } else {
                u64 gw = gw0, go = go0;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    ow[k] = wp[k]; oa[k] = 0.f; os[k] = 0.f;
                    if ((mw4 >> k) & 1u) ow[k] = __fadd_rn(wp[k], __uint_as_float(__ldg(sec0 + gw++)));
                    if ((mo4 >> k) & 1u) { oa[k] = __uint_as_float(__ldg(sec1 + go)); os[k] = __uint_as_float(__ldg(sec2 + go)); ++go; }
                }
            }
            if (DENSE) {
                // eight lanes hold 32 consecutive elements = 16 bytes of each section: gather them in
                // the first of the eight and write them with one store
                u32 v[3] = {nib0, nib1, nib2};
                const u64 sb = dense_section_bytes(n, BITS);
                unsigned char* sec = d.dense + header_bytes(KMAX) + i0 / 2;
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    const u32 pair = v[j] | (__shfl_down_sync(0xffffffffu, v[j], 1) << 16);
                    const u32 y = __shfl_down_sync(0xffffffffu, pair, 2);
                    const u32 z = __shfl_down_sync(0xffffffffu, pair, 4);
                    const u32 w = __shfl_down_sync(0xffffffffu, pair, 6);
                    if ((lane & 7) == 0 && live) *reinterpret_cast<uint4*>(sec + j * sb) = make_uint4(pair, y, z, w);
                }
            } else if (live) {
                store4(w_out, i0, n, ow);
                store4(d.ea_out, i0, n, oa);
                store4(d.eas_out, i0, n, os);
            }
        }
        __syncwarp();                                     // the warp's shared-memory corner is free again
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(&call->flags, FLAG_CORRUPT);
}

void launch_decode(const LaunchCfg& cfg, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                   const Workspace& ws, CallState* call, int wfmt) {
    dec_validate_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, call);
    if (!tiles) { prof_mark(cfg, ST_DEC_PREP, 1); return; }
    dec_popcount_kernel<<<(tiles + TPB / 32 - 1) / (TPB / 32), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws);
    dec_scan_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, ws, call);
    prof_mark(cfg, ST_DEC_PREP, 3);
    const u32 grid = min((tiles + DEC_WARPS - 1) / DEC_WARPS, (u32)cfg.sms * 4u);
    const size_t smem = sizeof(DecodeSmem);
    auto run = [&](auto tag) {
        using WT = decltype(tag);
        cudaFuncSetAttribute(decode_kernel<false, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        decode_kernel<false, WT><<<grid, TPB, smem, cfg.stream>>>(descs, st, nt, tiles, ws, call);
    };
    if (wfmt == WF_F16) run(__half{});
    else if (wfmt == WF_BF16) run(__nv_bfloat16{});
    else run(float{});
    prof_mark(cfg, ST_DECODE, 1);
}

// ---------------------------------------------------------------------------
// The dense layout (Sections 3.3 and 4.2 as printed): header + centres as in the record (magic
// "EXCD", the container's size at offset 48), then one code per element for dW, ea and eas.

// Header, centres and the zero padding at the end of every section.  One block per tensor.
__global__ void __launch_bounds__(64) dense_header_kernel(const DecDesc* __restrict__ descs,
                                                          DecState* __restrict__ st, CallState* call) {
    const int t = blockIdx.x, tid = threadIdx.x;
    const DecDesc& d = descs[t];
    DecState& s = st[t];
    if (!s.valid) return;
    if (s.rflags || s.bits != BITS) {                     // only 4-bit records of the method proper have a dense layout
        __syncthreads();
        if (tid == 0) { s.valid = 0; atomicOr(&call->flags, FLAG_UNSUPPORTED); }
        return;
    }
    const u64 total = dense_bytes(d.numel, BITS);
    if (total > d.dense_avail) {                          // uniform over the block
        if (tid == 0) { s.valid = 0; atomicOr(&call->flags, FLAG_BLOB_FULL); }
        return;
    }
    const u32 hb = (u32)header_bytes(KMAX);
    u32* out = reinterpret_cast<u32*>(d.dense);
    const u32* in = reinterpret_cast<const u32*>(d.rec);
    for (u32 w = tid; w < hb / 4; w += 64) {
        u32 v = in[w];                                    // counts, bits, K, header size, centres, padding
        if (w == 0) v = DENSE_MAGIC;
        if (w == 12) v = (u32)total;
        if (w == 13) v = (u32)(total >> 32);
        out[w] = v;
    }
    const u64 sb = dense_section_bytes(d.numel, BITS);
    if (sb && tid < 12) {                                 // last 16 bytes of each section
        const int j = tid / 4;
        reinterpret_cast<u32*>(d.dense + hb + (j + 1) * sb - 16)[tid % 4] = 0;
    }
}

void launch_record_to_dense(const LaunchCfg& cfg, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                            const Workspace& ws, CallState* call) {
    dec_validate_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, call);
    if (tiles) {
        dec_popcount_kernel<<<(tiles + TPB / 32 - 1) / (TPB / 32), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws);
        dec_scan_kernel<<<nt, TPB, 0, cfg.stream>>>(descs, st, ws, call);
    }
    dense_header_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, call);
    prof_mark(cfg, ST_DEC_PREP, tiles ? 4 : 2);
    if (!tiles) return;
    const u32 grid = min((tiles + DEC_WARPS - 1) / DEC_WARPS, (u32)cfg.sms * 4u);
    cudaFuncSetAttribute(decode_kernel<true, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecodeSmem));
    decode_kernel<true, float><<<grid, TPB, sizeof(DecodeSmem), cfg.stream>>>(descs, st, nt, tiles, ws, call);
    prof_mark(cfg, ST_DENSE, 1);
}

// Algorithm 2 on the dense layout.  validate: header against the layout; decode: every element
// looks its code up (no ranks needed), counting the non-zero codes; check: the counts must be the
// header's.
__global__ void __launch_bounds__(64) dense_validate_kernel(const DecDesc* __restrict__ descs,
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
            if (h[0] == DENSE_MAGIC && h[1] == VERSION && numel == d.numel && h[8] == BITS && h[9] == KMAX &&
                h[10] == header_bytes(KMAX) && nnz_o <= nnz_w && nnz_w <= numel &&
                total == dense_bytes(numel, BITS) && total <= d.rec_avail) {
                ok = 1;
                s.bits = BITS;
                s.nnz_w = (u32)nnz_w; s.nnz_o = (u32)nnz_o;
            }
        }
        s.valid = ok;
        s.cnt_w = 0; s.cnt_o = 0;
        if (!ok) atomicOr(&call->flags, FLAG_CORRUPT);
    }
    __syncthreads();
    if (ok && tid < 3 * KPAD) {
        const int k = tid / KPAD, j = tid % KPAD;
        s.cent[k][j] = j < KMAX ? reinterpret_cast<const float*>(d.rec + HEADER_FIXED)[k * KMAX + j] : 0.f;
    }
}

// One bit per non-zero 4-bit code of a word of eight.
__device__ __forceinline__ u32 nonzero_nibbles(u32 w) { return (w | (w >> 1) | (w >> 2) | (w >> 3)) & 0x11111111u; }

__global__ void __launch_bounds__(TPB) dense_decode_kernel(const DecDesc* __restrict__ descs,
                                                           DecState* __restrict__ st, int nt, u32 tiles,
                                                           CallState* call) {
    __shared__ float cent[3][KPAD + 1];                   // [0] = the zero centre of code 0
    const int tid = threadIdx.x, lane = tid & 31;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u32 bad = 0, cw = 0, co = 0;
    auto flush = [&](int t) {
        cw = __reduce_add_sync(0xffffffffu, cw);
        co = __reduce_add_sync(0xffffffffu, co);
        if (lane == 0) {
            if (cw) atomicAdd(&st[t].cnt_w, cw);
            if (co) atomicAdd(&st[t].cnt_o, co);
        }
        cw = co = 0;
    };
    for (u32 tile = lo; tile < hi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            if (cur >= 0) flush(cur);
            __syncthreads();
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            if (tid < 3 * (KPAD + 1)) {
                const int k = tid / (KPAD + 1), j = tid % (KPAD + 1);
                cent[k][j] = j ? st[cur].cent[k][j - 1] : 0.f;
            }
            __syncthreads();
        }
        if (!st[cur].valid) continue;
        const DecDesc& d = descs[cur];
        const float* w_prev = static_cast<const float*>(d.w_prev);
        float* w_out = static_cast<float*>(d.w_out);
        const u64 n = d.numel;
        const u64 sb = dense_section_bytes(n, BITS);
        const unsigned char* sec = d.rec + header_bytes(KMAX);
        const u64 base = (u64)(tile - tb) * TILE;
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
            const u64 i0 = base + r * (TPB * 4) + tid * 4;     // four elements = 16 bits per stream
            if (i0 >= n) continue;
            const u32 ww = *reinterpret_cast<const unsigned short*>(sec + i0 / 2);
            const u32 wa = *reinterpret_cast<const unsigned short*>(sec + sb + i0 / 2);
            const u32 we = *reinterpret_cast<const unsigned short*>(sec + 2 * sb + i0 / 2);
            const u32 zw = nonzero_nibbles(ww), za = nonzero_nibbles(wa), ze = nonzero_nibbles(we);
            cw += __popc(zw); co += __popc(za);
            bad |= (za ^ ze) | (za & ~zw);                // moments disagree; a moment kept where the weight is pruned
            const u32 left = n - i0 >= 4 ? 4u : (u32)(n - i0);
            if (left < 4 && ((ww | wa | we) >> (4 * left))) bad = 1;   // codes past the last element
            float wp[4];
            load4(w_prev, i0, n, wp);
            float ow[4], oa[4], os[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const u32 c0 = (ww >> (4 * k)) & 15u, c1 = (wa >> (4 * k)) & 15u, c2 = (we >> (4 * k)) & 15u;
                ow[k] = c0 ? __fadd_rn(wp[k], cent[0][c0]) : wp[k];    // pruned: W^_(t-1) bit for bit
                oa[k] = cent[1][c1];
                os[k] = cent[2][c2];
            }
            store4(w_out, i0, n, ow);
            store4(d.ea_out, i0, n, oa);
            store4(d.eas_out, i0, n, os);
        }
    }
    if (cur >= 0) flush(cur);
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(&call->flags, FLAG_CORRUPT);
}

__global__ void dense_check_kernel(const DecState* __restrict__ st, int nt, CallState* call) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < nt && st[t].valid && (st[t].cnt_w != st[t].nnz_w || st[t].cnt_o != st[t].nnz_o))
        atomicOr(&call->flags, FLAG_CORRUPT);
}

void launch_dense_decode(const LaunchCfg& cfg, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                         CallState* call) {
    dense_validate_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, call);
    prof_mark(cfg, ST_DEC_PREP, 1);
    if (!tiles) return;
    const u32 grid = min(tiles, (u32)cfg.sms * 8u);
    dense_decode_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, call);
    dense_check_kernel<<<(nt + 127) / 128, 128, 0, cfg.stream>>>(st, nt, call);
    prof_mark(cfg, ST_DENSE, 2);
}

}  // namespace excp
