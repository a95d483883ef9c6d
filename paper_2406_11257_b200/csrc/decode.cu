// Algorithm 2 on the device: bitmap rank -> code -> centre,
//   W^_t = W^_(t-1) + C_w[I_w]   (pruned entries keep W^_(t-1) bit for bit)
//   ea^ = C_ea[I_ea], eas^ = C_eas[I_eas]   (0 where pruned)
//
// validate   one block per tensor: header fields against the layout; nothing
//            below reads a record that failed (so no read leaves the record)
// popcount   survivors per tile from the bitmaps
// scan       tensor-wide offsets; totals must equal the header's counts
// decode     per block of 1024 elements: ranks by a warp scan of the bitmap words, codes dealt
//            out to the set positions, then the dense outputs
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
// A tile is walked in four blocks of 1024 elements, each in two phases.
//   A  lane l owns bitmap word l of the block (32 consecutive elements).  A warp scan of the
//      words' populations gives the rank of every word's first survivor; the word's codes are then
//      consecutive bits of the section, fetched as one window and dealt out to the word's set
//      positions four elements at a time (a byte permute with a selector looked up by the 4 mask
//      bits).  The result, one byte per element, goes to the warp's rows in shared memory (or, for
//      the dense layout, straight to the container as 16 bytes per lane).
//   B  eight rounds of 128 elements, lane l taking four consecutive ones: codes from the rows,
//      centres from the table, 16-byte loads of W^_(t-1) and 16-byte stores of the three outputs,
//      all rounds independent of one another.
#ifndef EXCP_DEC_MIN_BLOCKS
#define EXCP_DEC_MIN_BLOCKS 3                // resident blocks per SM the decoder's registers are held to
#endif
#ifndef EXCP_DEC_RB
#define EXCP_DEC_RB 4                        // rounds of phase B whose loads are issued together
#endif
constexpr int DEC_WARPS = TPB / 32;
constexpr int ROW_BYTES = 48;                // 32 codes + padding: 16-byte aligned, rows spread over the banks
constexpr int CENT_SMEM = 16;                // centres kept in shared memory per stream (codes of at most 4 bits)

struct DecodeSmem {
    unsigned char rows[DEC_WARPS][3][32 * ROW_BYTES];   // codes of the block in flight, one byte per element
    float cent[DEC_WARPS][3][CENT_SMEM];
    u32 sel[16];                             // 4 mask bits -> byte-permute selector (see expand_word)
    u32 spread[16];                          // 4 mask bits -> 0x01 in every byte whose bit is set
};

// Code windows: the NB-bit codes of `cnt` consecutive survivors starting at rank g of a section, as
// NB 32-bit words with the first code at bit 0.  Only words that hold such codes are read.
template <int NB>
__device__ __forceinline__ void load_window(const u32* __restrict__ sec, u64 g, u32 cnt, u32 (&c)[NB],
                                            const CallState* call, u64 nnz) {
    if (!EXCP_IN_BOUNDS(call, g + cnt <= nnz)) cnt = 0;      // the codes asked for lie inside the section
    const u64 bit = g * NB;
    const u32 sh = (u32)bit & 31u;
    const u32* p = sec + (bit >> 5);
    const u32 nw = cnt ? (sh + cnt * NB + 31u) >> 5 : 0u;   // words that hold the codes
    u32 w[NB + 1];
#pragma unroll
    for (int k = 0; k <= NB; ++k) w[k] = (u32)k < nw ? __ldg(p + k) : 0u;
#pragma unroll
    for (int k = 0; k < NB; ++k) c[k] = __funnelshift_r(w[k], w[k + 1], sh);
}

// The next four codes of a window as four bytes (code k in byte k).
template <int NB>
__device__ __forceinline__ u32 four_codes(u32 low) {
    if (NB == 8) return low;
    if (NB == 4) {
        const u32 x = (low & 0x00ffu) | ((low & 0xff00u) << 8);
        return (x | (x << 4)) & 0x0f0f0f0fu;
    }
    low &= 0xffu;                                        // NB == 2: two codes per half
    const u32 x = (low | (low << 12)) & 0x000f000fu;
    return (x | (x << 6)) & 0x03030303u;
}

// Deals the codes of window c to the set positions of bitmap word `m`: out[j] holds elements
// 4j .. 4j+3 of the word, one byte each, 0 where the bit is clear.  Returns non-zero if a
// survivor's code is 0 (no record written by the compressor has one).
template <int NB>
__device__ __forceinline__ u32 expand_word(u32 m, u32 (&c)[NB], const u32* __restrict__ sel,
                                           const u32* __restrict__ spread, u32 (&out)[8]) {
    u32 bad = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const u32 m4 = (m >> (4 * j)) & 15u;
        const u32 o = __byte_perm(four_codes<NB>(c[0]), 0u, sel[m4]);
        u32 any = o | (o >> 1);                          // bit 0 of every byte: the byte's code is not 0
        if (NB >= 4) any |= (o >> 2) | (o >> 3);
        if (NB == 8) any |= (o >> 4) | (o >> 5) | (o >> 6) | (o >> 7);
        const u32 nz = any & 0x01010101u;
        bad |= nz ^ spread[m4];
        out[j] = o;
        const u32 s = (u32)__popc(m4) * NB;              // bits used: at most 32
        if (NB == 8 && s == 32u) {
#pragma unroll
            for (int k = 0; k + 1 < NB; ++k) c[k] = c[k + 1];
            c[NB - 1] = 0u;
        } else {
#pragma unroll
            for (int k = 0; k + 1 < NB; ++k) c[k] = __funnelshift_r(c[k], c[k + 1], s);
            c[NB - 1] >>= s;
        }
    }
    return bad;
}

// The sparse form of expand_word for the two moment streams, which share their bitmap word `m` and keep
// few elements: one step per set bit (the caller makes sure that no lane of the warp has more than
// SPARSE_MAX of them, so that a stream's codes fit the first two words of its window).  TO_ROWS: the codes
// go to the lane's (zeroed) rows in shared memory, a byte each; otherwise they are returned as the dense
// layout's 16 bytes, a nibble each (NB = 4).
constexpr u32 SPARSE_MAX = 8;

template <int NB, bool TO_ROWS>
__device__ __forceinline__ u32 expand_sparse2(u32 m, const u32 (&c1)[NB], const u32 (&c2)[NB], unsigned char* row1,
                                              unsigned char* row2, uint4& d1, uint4& d2) {
    u64 w1 = c1[0], w2 = c2[0];
    if (NB > 1) { w1 |= (u64)c1[NB > 1 ? 1 : 0] << 32; w2 |= (u64)c2[NB > 1 ? 1 : 0] << 32; }
    u64 lo1 = 0, hi1 = 0, lo2 = 0, hi2 = 0;
    u32 bad = 0;
    constexpr u32 CMASK = (1u << NB) - 1u;
    if (TO_ROWS) {
        reinterpret_cast<uint4*>(row1)[0] = make_uint4(0, 0, 0, 0); reinterpret_cast<uint4*>(row1)[1] = make_uint4(0, 0, 0, 0);
        reinterpret_cast<uint4*>(row2)[0] = make_uint4(0, 0, 0, 0); reinterpret_cast<uint4*>(row2)[1] = make_uint4(0, 0, 0, 0);
    }
    while (m) {
        const u32 pos = (u32)__ffs((int)m) - 1u;
        m &= m - 1u;
        const u32 k1 = (u32)w1 & CMASK, k2 = (u32)w2 & CMASK;
        w1 >>= NB; w2 >>= NB;
        bad |= (k1 == 0u) | (k2 == 0u);
        if (TO_ROWS) {
            row1[pos] = (unsigned char)k1;
            row2[pos] = (unsigned char)k2;
        } else {
            const u32 sh = 4u * (pos & 15u);
            const u64 v1 = (u64)k1 << sh, v2 = (u64)k2 << sh;
            if (pos < 16u) { lo1 |= v1; lo2 |= v2; } else { hi1 |= v1; hi2 |= v2; }
        }
    }
    if (!TO_ROWS) {
        d1 = make_uint4((u32)lo1, (u32)(lo1 >> 32), (u32)hi1, (u32)(hi1 >> 32));
        d2 = make_uint4((u32)lo2, (u32)(lo2 >> 32), (u32)hi2, (u32)(hi2 >> 32));
    }
    return bad;
}

// Eight bytes-per-element words -> four nibbles-per-element words (the dense layout's 16 bytes).
__device__ __forceinline__ uint4 pack_nibbles(const u32 (&o)[8]) {
    u32 d[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        u32 lo = o[2 * q], hi = o[2 * q + 1];
        lo = (lo | (lo >> 4)) & 0x00ff00ffu; lo = (lo | (lo >> 8)) & 0xffffu;
        hi = (hi | (hi >> 4)) & 0x00ff00ffu; hi = (hi | (hi >> 8)) & 0xffffu;
        d[q] = lo | (hi << 16);
    }
    return make_uint4(d[0], d[1], d[2], d[3]);
}

struct DecTile {                 // what the phases need to know about the tile in hand
    const unsigned char* rec;
    const u32 *sec0, *sec1, *sec2;
    u64 n, base;                 // elements of the tensor; first element of the tile
    u32 rflags;
    int tensor;
};

// One block of 1024 elements whose codes are NB bits wide.  a, b: this lane's words of the two
// bitmaps; gw, go: ranks of their first survivors.
template <bool DENSE, int NB, typename WT>
__device__ __forceinline__ u32 decode_block(const DecTile& t, const DecDesc& d, const DecState& s, DecodeSmem& sm, int warp,
                                            int lane, u32 blk, u32 a, u32 b, u64 gw, u64 go, const CallState* call) {
    u32 bad = 0;
    unsigned char* rw = sm.rows[warp][0] + lane * ROW_BYTES;
    unsigned char* ra = sm.rows[warp][1] + lane * ROW_BYTES;
    unsigned char* rs = sm.rows[warp][2] + lane * ROW_BYTES;
    const u64 e0 = t.base + (u64)blk * 1024u;            // first element of the block
    const u64 sb = DENSE ? dense_section_bytes(t.n, BITS) : 0;
    unsigned char* dout = DENSE ? d.dense + header_bytes(KMAX) + (e0 + 32u * lane) / 2 : nullptr;
    const bool dlive = e0 + 32u * lane < t.n;            // DENSE: 32 codes = 16 bytes per lane and section (NB == 4)
    {
        u32 c[NB], ow8[8];
        load_window<NB>(t.sec0, gw, (u32)__popc(a), c, call, s.nnz_w);
        bad |= expand_word<NB>(a, c, sm.sel, sm.spread, ow8);
        if (DENSE) {
            if (dlive) *reinterpret_cast<uint4*>(dout) = pack_nibbles(ow8);
        } else {
            reinterpret_cast<uint4*>(rw)[0] = make_uint4(ow8[0], ow8[1], ow8[2], ow8[3]);
            reinterpret_cast<uint4*>(rw)[1] = make_uint4(ow8[4], ow8[5], ow8[6], ow8[7]);
        }
    }
    {
        u32 c1[NB], c2[NB];
        const u32 pb = (u32)__popc(b);
        load_window<NB>(t.sec1, go, pb, c1, call, s.nnz_o);
        load_window<NB>(t.sec2, go, pb, c2, call, s.nnz_o);
        if (__reduce_max_sync(0xffffffffu, pb) <= SPARSE_MAX) {      // the usual case: few moments survive
            uint4 d1, d2;
            bad |= expand_sparse2<NB, !DENSE>(b, c1, c2, ra, rs, d1, d2);
            if (DENSE && dlive) {
                *reinterpret_cast<uint4*>(dout + sb) = d1;
                *reinterpret_cast<uint4*>(dout + 2 * sb) = d2;
            }
        } else {
            u32 oa8[8], os8[8];
            bad |= expand_word<NB>(b, c1, sm.sel, sm.spread, oa8);
            bad |= expand_word<NB>(b, c2, sm.sel, sm.spread, os8);
            if (DENSE) {
                if (dlive) {
                    *reinterpret_cast<uint4*>(dout + sb) = pack_nibbles(oa8);
                    *reinterpret_cast<uint4*>(dout + 2 * sb) = pack_nibbles(os8);
                }
            } else {
                reinterpret_cast<uint4*>(ra)[0] = make_uint4(oa8[0], oa8[1], oa8[2], oa8[3]);
                reinterpret_cast<uint4*>(ra)[1] = make_uint4(oa8[4], oa8[5], oa8[6], oa8[7]);
                reinterpret_cast<uint4*>(rs)[0] = make_uint4(os8[0], os8[1], os8[2], os8[3]);
                reinterpret_cast<uint4*>(rs)[1] = make_uint4(os8[4], os8[5], os8[6], os8[7]);
            }
        }
    }
    if (DENSE) return bad;
    __syncwarp();
    const WT* w_prev = static_cast<const WT*>(d.w_prev);
    WT* w_out = static_cast<WT*>(d.w_out);
    const bool absolute = t.rflags & REC_ABSOLUTE;       // the weight stream is W itself
    // Codes of at most 4 bits: the tables in shared memory are indexed by the code itself, and code 0 (pruned)
    // finds 0 for the moments and -0 for the weights: x + (-0) = x for every x, so a pruned weight keeps
    // W^_(t-1) bit for bit (and an absolute one becomes 0 + (-0) = +0) with no test of the code.
    // Wide codes: the tables stay in global memory (cached), entry code - 1.
    const float* cw = NB <= 4 ? sm.cent[warp][0] : s.cent[0];
    const float* ca = NB <= 4 ? sm.cent[warp][1] : s.cent[1];
    const float* cs = NB <= 4 ? sm.cent[warp][2] : s.cent[2];
    constexpr int RB = EXCP_DEC_RB;
#pragma unroll
    for (int r0 = 0; r0 < 8; r0 += RB) {
        float wp[RB][4];
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const u64 i0 = e0 + (u32)(r0 + r) * 128u + 4u * lane;
            wp[r][0] = wp[r][1] = wp[r][2] = wp[r][3] = 0.f;
            if (!absolute && i0 < t.n) load4(w_prev, i0, t.n, wp[r]);
        }
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const u32 e = (u32)(r0 + r) * 128u + 4u * lane;             // element within the block
            const u64 i0 = e0 + e;
            if (i0 >= t.n) continue;
            const u32 ro = (e >> 5) * ROW_BYTES + (e & 31u);
            const u32 kw = *reinterpret_cast<const u32*>(sm.rows[warp][0] + ro);
            const u32 ka = *reinterpret_cast<const u32*>(sm.rows[warp][1] + ro);
            const u32 ks = *reinterpret_cast<const u32*>(sm.rows[warp][2] + ro);
            float ow[4], oa[4], os[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const u32 c0 = (kw >> (8 * k)) & 255u, c1 = (ka >> (8 * k)) & 255u, c2 = (ks >> (8 * k)) & 255u;
                if (NB <= 4) {
                    ow[k] = __fadd_rn(wp[r][k], cw[c0]);
                    oa[k] = ca[c1];
                    os[k] = cs[c2];
                } else {
                    ow[k] = c0 ? __fadd_rn(wp[r][k], cw[c0 - 1]) : wp[r][k];   // pruned: W^_(t-1) bit for bit
                    oa[k] = c1 ? ca[c1 - 1] : 0.f;
                    os[k] = c2 ? cs[c2 - 1] : 0.f;
                }
            }
            store4(w_out, i0, t.n, ow);
            store4(d.ea_out, i0, t.n, oa);
            store4(d.eas_out, i0, t.n, os);
        }
    }
    __syncwarp();                                        // the rows are free again
    return bad;
}

// A block of a record whose sections hold the survivors themselves (fp32, no codes): every element
// first gets its pruned value, then every lane puts the survivors of its word in place.
template <typename WT>
__device__ __forceinline__ void decode_block_raw(const DecTile& t, const DecDesc& d, int lane, u32 blk, u32 a, u32 b,
                                                 u64 gw, u64 go) {
    const WT* w_prev = static_cast<const WT*>(d.w_prev);
    WT* w_out = static_cast<WT*>(d.w_out);
    const bool absolute = t.rflags & REC_ABSOLUTE;
    const u64 e0 = t.base + (u64)blk * 1024u;
    const float zero[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
    for (int r = 0; r < 8; ++r) {
        const u64 i0 = e0 + (u32)r * 128u + 4u * lane;
        if (i0 >= t.n) continue;
        float wp[4] = {0.f, 0.f, 0.f, 0.f};
        if (!absolute) load4(w_prev, i0, t.n, wp);
        store4(w_out, i0, t.n, wp);
        store4(d.ea_out, i0, t.n, zero);
        store4(d.eas_out, i0, t.n, zero);
    }
    __syncwarp();                                        // the warp's stores above are ordered before the ones below
    const u64 i = e0 + 32u * lane;
    for (u32 m = a; m; m &= m - 1u) {
        const u64 el = i + (u32)__ffs((int)m) - 1u;
        const float v = __uint_as_float(__ldg(t.sec0 + gw++));
        wput(w_out, el, absolute ? v : __fadd_rn(wget(w_out, el), v));
    }
    for (u32 m = b; m; m &= m - 1u) {
        const u64 el = i + (u32)__ffs((int)m) - 1u;
        d.ea_out[el] = __uint_as_float(__ldg(t.sec1 + go));
        d.eas_out[el] = __uint_as_float(__ldg(t.sec2 + go));
        ++go;
    }
    __syncwarp();
}

#ifndef EXCP_DENSE_MIN_BLOCKS
#define EXCP_DENSE_MIN_BLOCKS 3
#endif
template <bool DENSE, typename WT>
__global__ void __launch_bounds__(TPB, DENSE ? EXCP_DENSE_MIN_BLOCKS : EXCP_DEC_MIN_BLOCKS) decode_kernel(const DecDesc* __restrict__ descs,
                                                     const DecState* __restrict__ st, int nt, u32 tiles,
                                                     Workspace ws, CallState* call) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecodeSmem& sm = *reinterpret_cast<DecodeSmem*>(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < 16) {
        // selector: byte p of the output takes the next unused code if bit p of the mask is set, else
        // byte 4 of the permute's operand pair (a zero)
        u32 sel = 0, spread = 0, next = 0;
        for (u32 p = 0; p < 4; ++p) {
            const bool on = (threadIdx.x >> p) & 1u;
            sel |= (on ? next : 4u) << (4 * p);
            spread |= (on ? 1u : 0u) << (8 * p);
            next += on;
        }
        sm.sel[threadIdx.x] = sel;
        sm.spread[threadIdx.x] = spread;
    }
    __syncthreads();
    const u32 gw = blockIdx.x * DEC_WARPS + warp, nw = gridDim.x * DEC_WARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u32 bad = 0;
    for (u32 tile = wlo; tile < whi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            __syncwarp();
            if (!DENSE && st[cur].valid && st[cur].bits <= 4) {
                const int kc = centres_of((int)st[cur].bits);
                for (int i = lane; i < 3 * CENT_SMEM; i += 32) {       // entry c = centre of code c; entry 0: see decode_block
                    const int k = i / CENT_SMEM, c = i % CENT_SMEM;
                    sm.cent[warp][k][c] = c == 0 ? (k == 0 ? -0.f : 0.f) : c <= kc ? st[cur].cent[k][c - 1] : 0.f;
                }
            }
            __syncwarp();
        }
        if (!st[cur].valid) continue;
        const DecDesc& d = descs[cur];
        const DecState& s = st[cur];
        DecTile t;
        t.rec = d.rec; t.n = d.numel; t.rflags = s.rflags; t.tensor = cur;
        t.base = (u64)(tile - tb) * TILE;
        t.sec0 = reinterpret_cast<const u32*>(d.rec + s.off_codes[0]);
        t.sec1 = reinterpret_cast<const u32*>(d.rec + s.off_codes[1]);
        t.sec2 = reinterpret_cast<const u32*>(d.rec + s.off_codes[2]);
        const u64 nwords = bitmap_bytes(t.n) / 4;
        const u64 w0 = (u64)(tile - tb) * TILE_WORDS;
        const bool last_tile = t.base + TILE > t.n;      // the tensor ends in this tile
        u64 rank_w = ws.tile_off_w[tile], rank_o = ws.tile_off_o[tile];
        const bool raw = s.rflags & REC_RAW;
        const u32 bits = s.bits;
#pragma unroll 1
        for (u32 blk = 0; blk < TILE / 1024; ++blk) {
            if (w0 + blk * 32u >= nwords) break;          // past the stored bitmap: nothing left in this tile
            const u64 wi = w0 + blk * 32u + lane;
            const u32 a = bm_word(d.rec, s.off_bm_w, nwords, wi);
            const u32 b = bm_word(d.rec, s.off_bm_o, nwords, wi);
            if (!(s.rflags & REC_MOMENTS_FREE)) bad |= b & ~a;       // a moment kept where the weight is pruned
            if (last_tile) {                             // no bit at or past the last element
                const u64 e = wi * 32;
                const u32 stray = e >= t.n ? 0xffffffffu : (t.n - e >= 32 ? 0u : 0xffffffffu << (u32)(t.n - e));
                bad |= (a | b) & stray;
            }
            const u32 pa = (u32)__popc(a), pb = (u32)__popc(b);
            u32 ia = pa, ib = pb;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const u32 x = __shfl_up_sync(0xffffffffu, ia, o), y = __shfl_up_sync(0xffffffffu, ib, o);
                if (lane >= o) { ia += x; ib += y; }
            }
            const u64 gwl = rank_w + ia - pa, gol = rank_o + ib - pb;
            rank_w += __shfl_sync(0xffffffffu, ia, 31);
            rank_o += __shfl_sync(0xffffffffu, ib, 31);
            if (__any_sync(0xffffffffu, bad)) break;     // nothing is decoded past an inconsistency
            if (raw) {
                if (!DENSE) decode_block_raw<WT>(t, d, lane, blk, a, b, gwl, gol);
            } else if (DENSE || bits == 4) {
                bad |= decode_block<DENSE, 4, WT>(t, d, s, sm, warp, lane, blk, a, b, gwl, gol, call);
            } else if (bits == 2) {
                bad |= decode_block<false, 2, WT>(t, d, s, sm, warp, lane, blk, a, b, gwl, gol, call);
            } else {
                bad |= decode_block<false, 8, WT>(t, d, s, sm, warp, lane, blk, a, b, gwl, gol, call);
            }
        }
        if (__any_sync(0xffffffffu, bad)) break;
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
    const u32 grid = min((tiles + DEC_WARPS - 1) / DEC_WARPS, (u32)cfg.sms * (u32)EXCP_DEC_MIN_BLOCKS);
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
    const u32 grid = min((tiles + DEC_WARPS - 1) / DEC_WARPS, (u32)cfg.sms * (u32)EXCP_DENSE_MIN_BLOCKS);
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
                cent[k][j] = j ? st[cur].cent[k][j - 1] : k == 0 ? -0.f : 0.f;   // x + (-0) = x: a pruned weight keeps its bits
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
        // All loads of the tile first, then the arithmetic and the stores.  In a round a warp has 256
        // elements: every lane loads one 32-bit word of codes per stream (its eight elements) and, twice, four
        // weights in the order that keeps a warp's 16-byte accesses contiguous (lane l: elements 4l.. of each
        // half); the codes of those four come from lane l/2 of that half by a shuffle.
        constexpr int R8 = TILE / (TPB * 8);
        u32 ww[R8], wa[R8], we[R8];
        float wp[R8][2][4];
#pragma unroll
        for (int r = 0; r < R8; ++r) {
            const u64 w0 = base + (u64)r * (TPB * 8) + (u64)(tid >> 5) * 256u;     // the warp's first element
            const u64 e0 = w0 + 8u * lane;                 // a section is padded to whole 16-byte units: the word exists
            ww[r] = wa[r] = we[r] = 0;
            if (e0 < n) {
                ww[r] = *reinterpret_cast<const u32*>(sec + e0 / 2);
                wa[r] = *reinterpret_cast<const u32*>(sec + sb + e0 / 2);
                we[r] = *reinterpret_cast<const u32*>(sec + 2 * sb + e0 / 2);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const u64 i0 = w0 + 128u * h + 4u * lane;
                wp[r][h][0] = wp[r][h][1] = wp[r][h][2] = wp[r][h][3] = 0.f;
                if (i0 < n) load4(w_prev, i0, n, wp[r][h]);
            }
        }
#pragma unroll
        for (int r = 0; r < R8; ++r) {
            const u64 w0 = base + (u64)r * (TPB * 8) + (u64)(tid >> 5) * 256u;
            const u64 e0 = w0 + 8u * lane;
            if (e0 < n) {                                   // the checks, on the lane's own eight elements
                const u32 zw = nonzero_nibbles(ww[r]), za = nonzero_nibbles(wa[r]), ze = nonzero_nibbles(we[r]);
                cw += __popc(zw); co += __popc(za);
                bad |= (za ^ ze) | (za & ~zw);            // moments disagree; a moment kept where the weight is pruned
                const u32 left = n - e0 >= 8 ? 8u : (u32)(n - e0);
                if (left < 8 && ((ww[r] | wa[r] | we[r]) >> (4 * left))) bad = 1;   // codes past the last element
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int src = 16 * h + (lane >> 1), sh = 16 * (lane & 1);
                const u32 kw = __shfl_sync(0xffffffffu, ww[r], src) >> sh;
                const u32 ka = __shfl_sync(0xffffffffu, wa[r], src) >> sh;
                const u32 ke = __shfl_sync(0xffffffffu, we[r], src) >> sh;
                const u64 i0 = w0 + 128u * h + 4u * lane;
                if (i0 >= n) continue;
                float ow[4], oa[4], os[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const u32 c0 = (kw >> (4 * k)) & 15u, c1 = (ka >> (4 * k)) & 15u, c2 = (ke >> (4 * k)) & 15u;
                    ow[k] = __fadd_rn(wp[r][h][k], cent[0][c0]);      // code 0: + (-0), W^_(t-1) bit for bit
                    oa[k] = cent[1][c1];
                    os[k] = cent[2][c2];
                }
                store4(w_out, i0, n, ow);
                store4(d.ea_out, i0, n, oa);
                store4(d.eas_out, i0, n, os);
            }
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
