// Writing one record per tensor (the layout in include/excp.h): header with
// the three codebooks, the two bitmaps, and the final K-means assignment packed
// as 4-bit codes 1..15, two per byte, survivors in index order (Section 4.1).
//
// A tile's survivors start at an arbitrary rank of the tensor, so the first and
// last 32-bit code word of a tile may be shared with its neighbours: those words
// are cleared beforehand and OR-ed into; interior words are stored whole.
#include "excp_common.cuh"

namespace excp {

constexpr int BITS = 4;
constexpr int PER_WORD = 32 / BITS;   // 8 codes per 32-bit word

struct Sections {
    u64 bm_w, bm_o, codes[3];
};
__device__ inline Sections sections_of(u64 numel, u64 nnz_w, u64 nnz_o) {
    Sections s;
    s.bm_w = header_bytes(KMAX);
    s.bm_o = s.bm_w + bitmap_bytes(numel);
    s.codes[0] = s.bm_o + bitmap_bytes(numel);
    s.codes[1] = s.codes[0] + code_bytes(nnz_w, BITS);
    s.codes[2] = s.codes[1] + code_bytes(nnz_o, BITS);
    return s;
}

// Header, zeroed section tails, results for the host.  One block per tensor.
__global__ void __launch_bounds__(64) header_kernel(const TensorDesc* __restrict__ descs,
                                                    TensorState* __restrict__ st, unsigned char* blob,
                                                    CallState* call, TensorResult* results) {
    const int t = blockIdx.x, tid = threadIdx.x;
    const TensorState& s = st[t];
    if (tid == 0) {
        TensorResult r;
        r.nnz_w = s.nnz_w; r.nnz_o = s.nnz_o; r.blob_off = s.blob_off; r.blob_bytes = s.blob_bytes;
        r.median = __uint_as_float(s.median_bits); r.mean_abs_ea = s.mean_abs_ea;
        r.thr_w = s.thr_w; r.thr_o = s.thr_o;
        results[t] = r;
        if (s.flags) atomicOr(&call->flags, s.flags);
    }
    if (call->flags & FLAG_BLOB_FULL) return;
    unsigned char* rec = blob + s.blob_off;
    const u64 numel = descs[t].numel, nnz_w = s.nnz_w, nnz_o = s.nnz_o;
    const u32 hb = (u32)header_bytes(KMAX);
    u32* h32 = reinterpret_cast<u32*>(rec);
    if (tid < (int)(hb / 4)) {
        u32 v = 0;
        switch (tid) {
            case 0: v = MAGIC; break;
            case 1: v = VERSION; break;
            case 2: v = (u32)numel; break;
            case 3: v = (u32)(numel >> 32); break;
            case 4: v = (u32)nnz_w; break;
            case 5: v = (u32)(nnz_w >> 32); break;
            case 6: v = (u32)nnz_o; break;
            case 7: v = (u32)(nnz_o >> 32); break;
            case 8: v = BITS; break;
            case 9: v = KMAX; break;
            case 10: v = hb; break;
            case 12: v = (u32)s.blob_bytes; break;
            case 13: v = (u32)(s.blob_bytes >> 32); break;
            default:
                if (tid >= 16 && tid < 16 + 3 * KMAX) {
                    const int i = tid - 16;
                    v = __float_as_uint(s.s[i / KMAX].cent[i % KMAX]);
                }
        }
        h32[tid] = v;
    }
    // the last 16 bytes of every code section hold the padding: clear them
    const Sections sec = sections_of(numel, nnz_w, nnz_o);
    if (tid < 12) {
        const int k = tid >> 2;
        const u64 len = code_bytes(k == 0 ? nnz_w : nnz_o, BITS);
        if (len) reinterpret_cast<u32*>(rec + sec.codes[k] + len - 16)[tid & 3] = 0u;
    }
}

// Clears the first and last code word of every tile's range (they may be shared).
__global__ void __launch_bounds__(TPB) clear_edges_kernel(const TensorDesc* __restrict__ descs,
                                                          const TensorState* __restrict__ st, int nt,
                                                          u32 tiles, Workspace ws, unsigned char* blob,
                                                          const CallState* call) {
    if (call->flags & FLAG_BLOB_FULL) return;
    const u32 tile = blockIdx.x * TPB + threadIdx.x;
    if (tile >= tiles) return;
    const int t = find_tensor(descs, nt, tile);
    const TensorState& s = st[t];
    const Sections sec = sections_of(descs[t].numel, s.nnz_w, s.nnz_o);
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

// Final assignment + packing of one stream.
__global__ void __launch_bounds__(TPB) pack_codes_kernel(const TensorDesc* __restrict__ descs,
                                                         const TensorState* __restrict__ st, int nt,
                                                         u32 tiles, const float* __restrict__ surv,
                                                         const u32* __restrict__ tile_cnt,
                                                         const u32* __restrict__ tile_off, int stream,
                                                         unsigned char* blob, const CallState* call) {
    __shared__ float thr[KPAD];
    __shared__ unsigned char code[TILE];
    if (call->flags & FLAG_BLOB_FULL) return;
    const int tid = threadIdx.x;
    u32 lo, hi;
    block_range(tiles, lo, hi);
    int cur = -1;
    u32 tb = 0, ntl = 0;
    u32* words = nullptr;
    for (u32 tile = lo; tile < hi; ++tile) {
        if (cur < 0 || tile >= tb + ntl) {
            cur = find_tensor(descs, nt, tile);
            tb = descs[cur].tile_begin; ntl = descs[cur].num_tiles;
            const TensorState& s = st[cur];
            const Sections sec = sections_of(descs[cur].numel, s.nnz_w, s.nnz_o);
            words = reinterpret_cast<u32*>(blob + s.blob_off + sec.codes[stream]);
            __syncthreads();
            if (tid < KPAD) thr[tid] = s.s[stream].thr[tid];
        }
        __syncthreads();                       // thr ready; previous tile's codes consumed
        const u32 cnt = tile_cnt[tile];
        if (cnt == 0) continue;
        const u32 off = tile_off[tile];
        const float* data = surv + (u64)tile * TILE;
        for (u32 i = tid; i < cnt; i += TPB) {
            const float x = data[i];
            int p = (x > thr[7]) ? 8 : 0;
            p += (x > thr[p + 3]) ? 4 : 0;
            p += (x > thr[p + 1]) ? 2 : 0;
            p += (x > thr[p]) ? 1 : 0;
            code[i] = (unsigned char)(p + 1);
        }
        __syncthreads();
        const u32 w0 = off / PER_WORD, w1 = (off + cnt - 1) / PER_WORD;
        for (u32 w = w0 + tid; w <= w1; w += TPB) {
            u32 v = 0;
            const s64 first = (s64)w * PER_WORD - (s64)off;      // local index of the word's code 0
#pragma unroll
            for (int k = 0; k < PER_WORD; ++k) {
                const s64 i = first + k;
                if (i >= 0 && i < (s64)cnt) v |= (u32)code[i] << (BITS * k);
            }
            if (first >= 0 && first + PER_WORD <= (s64)cnt) words[w] = v;
            else atomicOr(&words[w], v);
        }
    }
}

// Bitmaps: scratch -> record.  One thread per 16 bytes.
__global__ void __launch_bounds__(TPB) copy_bitmaps_kernel(const TensorDesc* __restrict__ descs,
                                                           const TensorState* __restrict__ st, int nt,
                                                           u32 tiles, Workspace ws, unsigned char* blob,
                                                           const CallState* call) {
    if (call->flags & FLAG_BLOB_FULL) return;
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
    const u64 hb = header_bytes(KMAX);
    const uint4 a = reinterpret_cast<const uint4*>(ws.bm_w)[g];
    const uint4 b = reinterpret_cast<const uint4*>(ws.bm_o)[g];
    reinterpret_cast<uint4*>(rec + hb)[local] = a;
    reinterpret_cast<uint4*>(rec + hb + quads * 16)[local] = b;
}

void launch_pack(const LaunchCfg& cfg, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                 const Workspace& ws, const Params& p, unsigned char* blob, CallState* call,
                 TensorResult* results) {
    header_kernel<<<nt, 64, 0, cfg.stream>>>(descs, st, blob, call, results);
    if (!tiles) { prof_mark(cfg, ST_HEADER_EDGES, 1); return; }
    clear_edges_kernel<<<(tiles + TPB - 1) / TPB, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws, blob, call);
    prof_mark(cfg, ST_HEADER_EDGES, 2);
    const u32 grid = min(tiles, (u32)cfg.sms * 8u);
    pack_codes_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws.surv[0], ws.tile_cnt_w,
                                                     ws.tile_off_w, 0, blob, call);
    pack_codes_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws.surv[1], ws.tile_cnt_o,
                                                     ws.tile_off_o, 1, blob, call);
    pack_codes_kernel<<<grid, TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws.surv[2], ws.tile_cnt_o,
                                                     ws.tile_off_o, 2, blob, call);
    prof_mark(cfg, ST_PACK_CODES, 3);
    const u64 quads = (u64)tiles * (TILE_WORDS / 4);
    copy_bitmaps_kernel<<<(u32)((quads + TPB - 1) / TPB), TPB, 0, cfg.stream>>>(descs, st, nt, tiles, ws,
                                                                               blob, call);
    prof_mark(cfg, ST_COPY_BITMAPS, 1);
}

}  // namespace excp
