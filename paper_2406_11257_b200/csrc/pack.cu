// Writing one record per tensor (the layout in include/excp.h): header with
// the three codebooks, the two bitmaps, and the final K-means assignment packed
// as 4-bit codes 1..15, two per byte, survivors in index order (Section 4.2).
//
// A tile's survivors start at an arbitrary rank of the tensor, so the first and
// last 32-bit code word of a tile may be shared with its neighbours: those words
// are cleared beforehand and OR-ed into; interior words are stored whole.
#include "excp_common.cuh"
#include <type_traits>

namespace excp {

constexpr int BITS = 4;               // the width the method uses (Section 4.2); 2 and 8 are variants

struct Sections {
    u64 bm_w, bm_o, codes[3];
};
__device__ inline Sections sections_of(u64 numel, u64 nnz_w, u64 nnz_o, int bits = BITS) {
    Sections s;
    s.bm_w = header_bytes(centres_of(bits));
    s.bm_o = s.bm_w + bitmap_bytes(numel);
    s.codes[0] = s.bm_o + bitmap_bytes(numel);
    s.codes[1] = s.codes[0] + code_bytes(nnz_w, bits);
    s.codes[2] = s.codes[1] + code_bytes(nnz_o, bits);
    return s;
}

// Header, zeroed section tails, results for the host.  One block per tensor.
__global__ void __launch_bounds__(64) header_kernel(const TensorDesc* __restrict__ descs,
                                                    TensorState* __restrict__ st, unsigned char* blob,
                                                    CallState* call, TensorResult* results, int bits, u32 rflags) {
    const int t = blockIdx.x, tid = threadIdx.x;
    const TensorState& s = st[t];
    if (tid == 0) {
        TensorResult r;
        r.nnz_w = s.nnz_w; r.nnz_o = s.nnz_o; r.blob_off = s.blob_off; r.blob_bytes = s.blob_bytes;
        r.median = __uint_as_float(s.median_bits); r.mean_abs_ea = s.mean_abs_ea;
        r.thr_w = s.thr_w; r.thr_o = s.thr_o;
        r.sse[0] = r.sse[1] = r.sse[2] = 0.0;             // the packing kernels add to these
        results[t] = r;
        if (s.flags) atomicOr(&call->flags, s.flags);
    }
    if (call->flags & (FLAG_BLOB_FULL | FLAG_TIMEOUT)) return;
    unsigned char* rec = blob + s.blob_off;
    const u64 numel = descs[t].numel, nnz_w = s.nnz_w, nnz_o = s.nnz_o;
    const int kc = centres_of(bits);                  // 15, or 0 when the survivors are stored raw
    const u32 hb = (u32)header_bytes(kc);
    u32* h32 = reinterpret_cast<u32*>(rec);
    for (int w = tid; w < (int)(hb / 4); w += 64) {
        u32 v = 0;
        switch (w) {
            case 0: v = MAGIC; break;
            case 1: v = VERSION; break;
            case 2: v = (u32)numel; break;
            case 3: v = (u32)(numel >> 32); break;
            case 4: v = (u32)nnz_w; break;
            case 5: v = (u32)(nnz_w >> 32); break;
            case 6: v = (u32)nnz_o; break;
            case 7: v = (u32)(nnz_o >> 32); break;
            case 8: v = (u32)bits; break;
            case 9: v = (u32)kc; break;
            case 10: v = hb; break;
            case 11: v = rflags; break;
            case 12: v = (u32)s.blob_bytes; break;
            case 13: v = (u32)(s.blob_bytes >> 32); break;
            default:
                if (w >= 16 && w < 16 + 3 * kc) {
                    const int i = w - 16;
                    v = __float_as_uint(s.s[i / kc].cent[i % kc]);
                }
        }
        h32[w] = v;
    }
    // the last 16 bytes of every code section hold the padding: clear them
    const Sections sec = sections_of(numel, nnz_w, nnz_o, bits);
    if (tid < 12) {
        const int k = tid >> 2;
        const u64 len = code_bytes(k == 0 ? nnz_w : nnz_o, bits);
        if (len) reinterpret_cast<u32*>(rec + sec.codes[k] + len - 16)[tid & 3] = 0u;
    }
}

// Clears the first and last code word of every tile's range (they may be shared).
__global__ void __launch_bounds__(TPB) clear_edges_kernel(const TensorDesc* __restrict__ descs,
                                                          const TensorState* __restrict__ st, int nt,
                                                          u32 tiles, Workspace ws, unsigned char* blob,
                                                          const CallState* call, int bits) {
    if (call->flags & (FLAG_BLOB_FULL | FLAG_TIMEOUT)) return;
    const u32 tile = blockIdx.x * TPB + threadIdx.x;
    if (tile >= tiles) return;
    const u32 PER_WORD = 32u / (u32)bits;
    const int t = find_tensor(descs, nt, tile);
    const TensorState& s = st[t];
    const Sections sec = sections_of(descs[t].numel, s.nnz_w, s.nnz_o, bits);
    unsigned char* rec = blob + s.blob_off;
    for (int k = 0; k < 3; ++k) {
        const u32 cnt = (k == 0 ? ws.tile_cnt_w : ws.tile_cnt_o)[tile];
        if (!cnt) continue;
        const u32 off = (k == 0 ? ws.tile_off_w : ws.tile_off_o)[tile];
        u32* words = reinterpret_cast<u32*>(rec + sec.codes[k]);
        words[off / PER_WORD] = 0u;
        words[(off + cnt - 1) / PER_WORD] = 0u;
    }
}

// Final assignment + packing: NS = 1 for dW, NS = 2 for the two moment streams together (they
// share their counts).  A warp owns a run of tiles and reads their survivor segments with plain
// 16-byte loads.  Within a tile the survivors form rows of 32 / NB (one 32-bit word of codes in the
// tile's own alignment), one row per lane; the tile starts at an arbitrary rank of the tensor, so
// every output word is two neighbouring rows funnel-shifted by the rank's offset in its word: the
// neighbour's row comes by a shuffle, the last row of the previous 32 through a register.
constexpr int PWARPS = TPB / 32;

template <int NS, int NB, bool SSE>
struct PackSmem {
    float thr[PWARPS][NS][1 << NB];     // the K - 1 thresholds, +inf after them: sorted (4 bits) or as find_cluster's tree
    float cent[PWARPS][NS][SSE ? (1 << NB) : 1];   // the K centres (only when the quantisation error is wanted)
};

// Cluster of x = number of thresholds strictly below it.  thr_row: 16 fp32 thresholds
// (ascending, +inf from the 15th on, none of them -0) in shared memory; t3, t7, t11 are copies
// in registers.  Returns 4 * cluster.
__device__ __forceinline__ u32 find_cluster4(float x, float t3, float t7, float t11, const char* thr_row) {
    u32 p = x > t7 ? 32u : 0u;
    p += (x > (p ? t11 : t3)) ? 16u : 0u;
    p += (x > *reinterpret_cast<const float*>(thr_row + p + 4)) ? 8u : 0u;
    p += (x > *reinterpret_cast<const float*>(thr_row + p)) ? 4u : 0u;
    return p;
}

// Cluster of x = number of thresholds below it, for the widths other than 4: NB steps down the
// search tree of the 2^NB - 1 sorted entries (the last ones +inf), stored level by level: node i
// (the root is 1) has the children 2i and 2i + 1.  With the sorted array itself the probes of one
// level lie a power of two apart, all in one shared-memory bank; level by level they are neighbours.
template <int NB>
__device__ __forceinline__ u32 find_cluster(float x, const float* tree) {
    u32 i = 1;
#pragma unroll
    for (int step = 0; step < NB; ++step) i = 2u * i + (x > tree[i] ? 1u : 0u);
    return i - (1u << NB);
}
// Place in the sorted array of node i of that tree.
template <int NB>
__device__ __forceinline__ u32 tree_source(u32 i) {
    const u32 level = 31u - (u32)__clz((int)i);
    return ((2u * (i - (1u << level)) + 1u) << (NB - 1 - level)) - 1u;
}

// SSE: also add up the squared distances to the assigned centres (the statistics' sse_* fields).
template <int NS, int NB, bool SSE>
__global__ void __launch_bounds__(TPB) pack_codes_kernel(const TensorDesc* __restrict__ descs,
                                                         const TensorState* __restrict__ st, int nt,
                                                         u32 tiles, Workspace ws, int stream0,
                                                         unsigned char* blob, CallState* call,
                                                         TensorResult* results) {
    constexpr int PER = 32 / NB;                   // codes per 32-bit word = survivors per row
    constexpr int KTHR = 1 << NB;
    constexpr int U = NS == 1 ? 2 : 1;             // rows a lane has in flight per stream
    __shared__ __align__(16) PackSmem<NS, NB, SSE> sm;
    if (call->flags & (FLAG_BLOB_FULL | FLAG_TIMEOUT)) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u32 gw = blockIdx.x * PWARPS + warp, nw = gridDim.x * PWARPS;
    const u32 wlo = (u32)(((u64)tiles * gw) / nw), whi = (u32)(((u64)tiles * (gw + 1)) / nw);
    const u32* tile_cnt = stream0 == 0 ? ws.tile_cnt_w : ws.tile_cnt_o;
    const u32* tile_off = stream0 == 0 ? ws.tile_off_w : ws.tile_off_o;

    int cur = -1;
    u32 tb = 0, ntl = 0;
    u32* words[NS];
    float t3[NS], t7[NS], t11[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) { words[k] = nullptr; t3[k] = t7[k] = t11[k] = 0.f; }
    double sse[NS];                      // this lane's share of sum (x - centre)^2 in the tensor in hand
#pragma unroll
    for (int k = 0; k < NS; ++k) sse[k] = 0.0;
    auto flush_sse = [&](int t) {        // floating-point atomics: the last bits depend on the order of arrival
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            double v = sse[k];
#pragma unroll
            for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0 && v != 0.0) atomicAdd(&results[t].sse[stream0 + k], v);
            sse[k] = 0.0;
        }
    };

    for (u32 w0 = wlo; w0 < whi; w0 += 32) {
        const u32 nt32 = min(32u, whi - w0);
        const u32 mycnt = (u32)lane < nt32 ? min(tile_cnt[w0 + lane], (u32)TILE) : 0u;   // a count never leads out of its segment
        const u32 myoff = (u32)lane < nt32 ? tile_off[w0 + lane] : 0u;
        for (u32 ti = 0; ti < nt32; ++ti) {
            const u32 cnt = __shfl_sync(0xffffffffu, mycnt, ti);
            const u32 t0 = __shfl_sync(0xffffffffu, myoff, ti);    // tensor-wide rank of the tile's first survivor
            if (!cnt) continue;
            const u32 tile = w0 + ti;
            if (cur < 0 || tile >= tb + ntl) {
                if (SSE && cur >= 0) flush_sse(cur);
                cur = find_tensor(descs, nt, tile);
                tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
                const TensorState& s = st[cur];
                const Sections sec = sections_of(descs[cur].numel, s.nnz_w, s.nnz_o, NB);
                __syncwarp();
#pragma unroll
                for (int k = 0; k < NS; ++k) {
                    words[k] = reinterpret_cast<u32*>(blob + s.blob_off + sec.codes[stream0 + k]);
                    for (int j = lane; j < KTHR; j += 32) {
                        if (NB == 4) sm.thr[warp][k][j] = s.s[stream0 + k].thr[j];
                        else if (j) sm.thr[warp][k][j] = s.s[stream0 + k].thr[tree_source<NB>((u32)j)];
                        if (SSE) sm.cent[warp][k][j] = s.s[stream0 + k].cent[j];
                    }
                }
                __syncwarp();
#pragma unroll
                for (int k = 0; k < NS; ++k) {
                    if (NB == 4) { t3[k] = sm.thr[warp][k][3]; t7[k] = sm.thr[warp][k][7]; t11[k] = sm.thr[warp][k][11]; }
                }
            }
            const u32 nrows = (cnt + PER - 1) / PER;
            const u32 sh = (t0 % PER) * NB;                 // a row's shift inside the tensor's words
            const u32 wbase = t0 / PER;                     // output word of the tile's first row
            const u32 nout = nrows + (sh ? 1u : 0u);        // the last row spills into one more word
            u32 carry[NS];
#pragma unroll
            for (int k = 0; k < NS; ++k) carry[k] = 0;
            for (u32 r0 = 0; r0 < nout; r0 += 32 * U) {
                float xs[U][NS][PER];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const u32 r = r0 + 32 * u + lane;
                    if (r < nrows) {
#pragma unroll
                        for (int k = 0; k < NS; ++k) {
                            const float4* src = reinterpret_cast<const float4*>(ws.surv[stream0 + k] + (u64)tile * TILE + PER * r);
#pragma unroll
                            for (int q = 0; q < PER / 4; ++q) {
                                const float4 v = __ldcs(src + q);
                                xs[u][k][4 * q] = v.x; xs[u][k][4 * q + 1] = v.y; xs[u][k][4 * q + 2] = v.z; xs[u][k][4 * q + 3] = v.w;
                            }
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const u32 m = r0 + 32 * u + lane;               // this lane's row = its output word within the tile
                    if (r0 + 32 * u >= nout) break;                 // warp uniform
#pragma unroll
                    for (int k = 0; k < NS; ++k) {
                        u32 w = 0;
                        if (m < nrows) {
                            const char* thr_row = reinterpret_cast<const char*>(sm.thr[warp][k]);
#pragma unroll
                            for (int i = 0; i < PER; ++i) {
                                const u32 code = NB == 4 ? find_cluster4(xs[u][k][i], t3[k], t7[k], t11[k], thr_row) / 4 + 1
                                                         : find_cluster<NB>(xs[u][k][i], sm.thr[warp][k]) + 1;
                                w |= code << (NB * i);
                            }
                            const u32 have = cnt - PER * m;         // codes of this row that exist (the segment holds stale values after them)
                            if (have < (u32)PER) w &= (1u << (NB * have)) - 1u;
                            if (SSE) {                            // the row's squared distances in fp32, rows added in fp64
                                float acc = 0.f;
#pragma unroll
                                for (int i = 0; i < PER; ++i) {
                                    const u32 code = (w >> (NB * i)) & ((1u << NB) - 1u);
                                    const float d = __fsub_rn(xs[u][k][i], sm.cent[warp][k][code ? code - 1 : 0]);
                                    acc = code ? __fmaf_rn(d, d, acc) : acc;
                                }
                                sse[k] += (double)acc;
                            }
                        }
                        u32 prev = __shfl_up_sync(0xffffffffu, w, 1);
                        if (lane == 0) prev = carry[k];
                        carry[k] = __shfl_sync(0xffffffffu, w, 31);
                        // output word m of the tile = row m shifted up | row m-1 shifted down
                        const u32 v = (w << sh) | (sh ? prev >> (32 - sh) : 0u);
                        if (m < nout) {
                            const u64 g0 = (u64)(wbase + m) * PER;  // ranks the word covers: [g0, g0 + PER)
                            const bool whole = g0 >= t0 && g0 + PER <= (u64)t0 + cnt;
                            if ((whole || v) && EXCP_IN_BOUNDS(call, (u64)(wbase + m) * 4 < code_bytes(stream0 + k == 0 ? st[cur].nnz_w : st[cur].nnz_o, NB))) {
                                if (whole) words[k][wbase + m] = v;
                                else atomicOr(&words[k][wbase + m], v);
                            }
                        }
                    }
                }
            }
        }
    }
    if (SSE && cur >= 0) flush_sse(cur);
}

// Bitmaps: scratch -> record.  One thread per 16 bytes.
__global__ void __launch_bounds__(TPB) copy_bitmaps_kernel(const TensorDesc* __restrict__ descs,
                                                           const TensorState* __restrict__ st, int nt,
                                                           u32 tiles, Workspace ws, unsigned char* blob,
                                                           const CallState* call, u32 hb) {
    if (call->flags & (FLAG_BLOB_FULL | FLAG_TIMEOUT)) return;
    const u64 g = (u64)blockIdx.x * TPB + threadIdx.x;       // uint4 index over all tiles
    const u32 tile = (u32)(g / (TILE_WORDS / 4));
    if (tile >= tiles) return;
    const u32 q = (u32)(g % (TILE_WORDS / 4));
    const int t = find_tensor(descs, nt, tile);
    const u64 numel = descs[t].numel;
    const u64 quads = bitmap_bytes(numel) / 16;              // 16-byte units in one bitmap
    const u64 local = (u64)(tile - descs[t].tile_begin) * (TILE_WORDS / 4) + q;
    if (local >= quads) return;
    unsigned char* rec = blob + st[t].blob_off;
    const uint4 a = reinterpret_cast<const uint4*>(ws.bm_w)[g];
    const uint4 b = reinterpret_cast<const uint4*>(ws.bm_o)[g];
    reinterpret_cast<uint4*>(rec + hb)[local] = a;
    reinterpret_cast<uint4*>(rec + hb + quads * 16)[local] = b;
}

// Quantisation switched off (ablation table of Section 4.4): the survivors themselves go into the
// sections, fp32, in index order.  One warp per tile: its segment of each stream is copied to the
// tile's rank offset in the section.
__global__ void __launch_bounds__(TPB) pack_raw_kernel(const TensorDesc* __restrict__ descs,
                                                       const TensorState* __restrict__ st, int nt, u32 tiles,
                                                       Workspace ws, unsigned char* blob, const CallState* call) {
    if (call->flags & (FLAG_BLOB_FULL | FLAG_TIMEOUT)) return;
    const int lane = threadIdx.x & 31;
    const u32 tile = blockIdx.x * (TPB / 32) + (threadIdx.x >> 5);
    if (tile >= tiles) return;
    const int t = find_tensor(descs, nt, tile);
    const TensorState& s = st[t];
    const Sections sec = sections_of(descs[t].numel, s.nnz_w, s.nnz_o, 32);
    unsigned char* rec = blob + s.blob_off;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const u32 cnt = (k == 0 ? ws.tile_cnt_w : ws.tile_cnt_o)[tile];
        const u32 off = (k == 0 ? ws.tile_off_w : ws.tile_off_o)[tile];
        const float* src = ws.surv[k] + (u64)tile * TILE;
        float* dst = reinterpret_cast<float*>(rec + sec.codes[k]) + off;
        for (u32 i = lane; i < cnt; i += 32) dst[i] = src[i];
    }
}

void launch_pack(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                 const Workspace& ws, const Params& p, unsigned char* blob, CallState* call,
                 TensorResult* results, bool want_sse) {
    header_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, blob, call, results, stored_bits(p), record_flags(p));
    if (!tiles) { prof_mark(cfg, ST_HEADER_EDGES, 1); return; }
    if (p.flags & OPT_NO_QUANT) {
        prof_mark(cfg, ST_HEADER_EDGES, 1);
        pack_raw_kernel<<<(tiles + TPB / 32 - 1) / (TPB / 32), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, blob, call);
        prof_mark(cfg, ST_PACK_CODES, 1);
        const u64 quads = (u64)tiles * (TILE_WORDS / 4);
        copy_bitmaps_kernel<<<(u32)((quads + TPB - 1) / TPB), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, blob, call,
                                                                                   (u32)header_bytes(0));
        prof_mark(cfg, ST_COPY_BITMAPS, 1);
        return;
    }
    clear_edges_kernel<<<(tiles + TPB - 1) / TPB, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, blob, call, p.bits);
    prof_mark(cfg, ST_HEADER_EDGES, 2);
    const u32 grid = min((tiles + PWARPS - 1) / PWARPS, (u32)cfg.sms * 6u);
    auto run = [&](auto nb_tag, auto sse_tag) {
        constexpr int NB = decltype(nb_tag)::value;
        constexpr bool SSE = decltype(sse_tag)::value;
        pack_codes_kernel<1, NB, SSE><<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, 0, blob, call, results);
        pack_codes_kernel<2, NB, SSE><<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, 1, blob, call, results);
    };
    auto run_width = [&](auto sse_tag) {
        if (p.bits == 4) run(std::integral_constant<int, 4>{}, sse_tag);
        else if (p.bits == 2) run(std::integral_constant<int, 2>{}, sse_tag);
        else run(std::integral_constant<int, 8>{}, sse_tag);
    };
    if (want_sse) run_width(std::true_type{});
    else run_width(std::false_type{});
    prof_mark(cfg, ST_PACK_CODES, 2);
    const u64 quads = (u64)tiles * (TILE_WORDS / 4);
    copy_bitmaps_kernel<<<(u32)((quads + TPB - 1) / TPB), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws,
                                                                               blob, call, (u32)header_bytes(centres_of(p.bits)));
    prof_mark(cfg, ST_COPY_BITMAPS, 1);
}

}  // namespace excp
