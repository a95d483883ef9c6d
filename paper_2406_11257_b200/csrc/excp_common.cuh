// Shared declarations of the ExCP kernels: tile geometry, per-tensor device
// records, small device helpers, and the launch wrappers each .cu file exports.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace excp {

typedef unsigned long long u64;
typedef long long s64;
typedef unsigned int u32;

// A tile is the unit of work of every sweep: 4096 consecutive elements of one
// tensor = 256 threads x 4 rounds x one float4.  Tiles never span tensors, so a
// tile's 128 bitmap words and its survivor segment belong to exactly one tensor.
constexpr int TILE = 4096;
constexpr int TPB = 256;
constexpr int TILE_WORDS = TILE / 32;
constexpr int ROUNDS = TILE / (TPB * 4);         // 4
constexpr int CHUNKS = ROUNDS * (TPB / 32);      // 32 warp-chunks of 128 elements per tile

constexpr int HIST1_BITS = 13;                   // first radix-select level: top 13 of 31 key bits
constexpr int HIST1_BINS = 1 << HIST1_BITS;
constexpr int HIST1_SHIFT = 31 - HIST1_BITS;     // 18 bits left for the in-bin select
constexpr int KMAX = 15;                         // centres at 4 bits
constexpr int KPAD = 16;
constexpr int KCAP = 256;                        // room for the centres of the widest code (8 bits: 255)
constexpr int SAMPLE_MAX = 1024;                 // K-means start sample
constexpr int MAX_GROUP_TENSORS = 1024;
constexpr int KM_MAX_GRID = 1024;                // blocks of a K-means sweep (two per SM)

constexpr u32 FLAG_NONFINITE = 1u;               // NaN/Inf input or negative second moment
constexpr u32 FLAG_BLOB_FULL = 2u;               // records do not fit blob_capacity
constexpr u32 FLAG_CORRUPT = 4u;                 // decompress: inconsistent record
constexpr u32 FLAG_INTERNAL = 8u;                // a self-check failed (candidate count mismatch)
constexpr u32 FLAG_TIMEOUT = 16u;                // a bounded wait on an asynchronous copy ran out
constexpr u32 FLAG_UNSUPPORTED = 32u;            // a record variant the called routine does not handle

// Ablation switches of a compress call (ViT table caption; ablation table of Section 4.4)
constexpr u32 OPT_NO_W2M = 1u;                   // M_o without the conjunction with M_w
constexpr u32 OPT_NO_M2W = 2u;                   // M_w = [ |dW| > alpha ], alpha the set threshold
constexpr u32 OPT_NO_RESIDUAL = 4u;              // the weights themselves, not their residual
constexpr u32 OPT_NO_PRUNE = 8u;                 // every element kept
constexpr u32 OPT_NO_QUANT = 16u;                // survivors stored as fp32
constexpr u32 OPT_ALL = 31u;
// What a record says about itself (header offset 44)
constexpr u32 REC_MOMENTS_FREE = 1u;             // M_o need not lie inside M_w
constexpr u32 REC_ABSOLUTE = 2u;                 // the weight stream is W: Algorithm 2 adds nothing
constexpr u32 REC_RAW = 4u;                      // bits = 32, K = 0: sections hold fp32 survivors
constexpr u32 REC_ALL = 7u;

constexpr u32 MAGIC = 0x50435845u;
constexpr u32 DENSE_MAGIC = 0x44435845u;         // "EXCD": one code per element, 0 = pruned
constexpr u32 VERSION = 1u;
constexpr int HEADER_FIXED = 64;

// Storage format of the weight tensors (W_t, W^_(t-1), W^_t); the moments are always fp32.
enum WeightFormat { WF_F32 = 0, WF_F16 = 1, WF_BF16 = 2 };

struct TensorDesc {              // built on the host, one per tensor of a group
    const void* w_t;             // fp32, fp16 or bf16 (the call's weight format)
    const void* w_prev;
    const float* ea;
    const float* eas;
    u64 numel;
    u64 tensor_index;            // position in the checkpoint (enters the start sample)
    u32 tile_begin;              // first tile of this tensor within the group
    u32 num_tiles;
    u32 pad_[2];                 // 64 bytes: indexing the array is a shift
};

struct StreamState {             // K-means state of one stream (0 = dW, 1 = ea, 2 = eas)
    float cent[KCAP];            // centres, ascending; 0 from K on
    float thr[KCAP];             // thr[j] = largest fp32 <= (c_j + c_j+1)/2; +inf from K-1 on
    u32 maxkey;                  // max |x| bit pattern over the survivors
    int e;                       // fixed-point exponent E
    float scale1, scale2;        // 2^(30-E) split in two exact factors
};

struct TensorState {             // device scratch, zeroed per group
    u32 hist1[HIST1_BINS];
    u64 sum_lo[256];             // exact sum of |ea|: low/high halves of warp partial sums,
    u64 sum_hi[256];             //   indexed by the partial sum's exponent
    u64 sum_low[256];            // mantissa sums of the rare elements far below a warp's maximum
    u32 bin1;
    u32 rank_in_bin;
    u32 bin_count;
    u32 cand_count;
    u32 flags;
    u32 median_bits;
    float mean_abs_ea;
    float thr_w, thr_o;
    u32 nnz_w, nnz_o;
    u32 lo_key, hi_key;          // bracket of magnitude patterns that should hold the median (from a sample)
    u32 count_below;             // elements below the bracket
    u32 med_done;                // the sample was the whole tensor: median already known
    u32 need_hist;               // the bracket missed the median: take the histogram path
    u32 sel_hs;                  // select among the bracket's keys: bits of key - lo_key still open,
    u32 sel_prefix;              //   the bits above them,
    u32 sel_rank;                //   the rank wanted among the keys that share those bits
    u32 sel_done[4];             // blocks that have added their counts, per digit pass
    u32 sel_hist[4][256];        // digit counts per pass
    u32 pad_;
    u64 blob_off;                // start of this tensor's record in the blob
    u64 blob_bytes;
    StreamState s[3];
};

struct TensorResult {            // copied back to the host at the end of a call
    u64 nnz_w, nnz_o, blob_off, blob_bytes;
    float median, mean_abs_ea, thr_w, thr_o;
    double sse[3];               // sum of squared distances to the assigned centre, per stream (when asked for)
};

struct CallState {               // one per handle, device resident
    u64 blob_cursor;             // running end of the records written so far
    u32 flags;                   // OR of every tensor's flags
    u32 pad_;
};

constexpr int NCELL = 4096;       // value cells per tensor and stream for the K-means iterations
constexpr int NCLASS = 512;       // sign x exponent field of an fp32 value = its top nine bits

// K-means working state of one stream of one tensor.  The cells are a monotone map of fp32 values
// to 0..NCELL-1 (see cell_of): every (sign, exponent) class owns a power-of-two number of equal
// steps of the mantissa, more of them where a sample of the survivors is dense.
struct CellStream {
    u32 tab[NCLASS];             // class of the value key (see cell_of) -> (first cell << 8) | mantissa shift
    u32 cnt[NCELL];              // survivors per cell
    u64 mag[NCELL];              // sum of |Q| per cell; once planned: low word = start of the cell in the
                                 //   gathered copy, high word = values gathered so far
    u32 cntpre[NCELL + 1];       // exclusive prefix of cnt
    u32 first_pos;               // first cell of the non-negative values
    s64 sumpre[NCELL + 1];       // exclusive prefix of the signed fixed-point sums
    u32 sel[NCELL / 32];         // cells whose values are in the gathered copy
    u32 it_done;                 // Lloyd iterations completed
    u32 active;                  // iterations remain: the next round plans and gathers for them
};
struct CellState {
    CellStream s[3];
};

struct Workspace {               // device arrays sized for cap_tiles tiles
    float* bkt[3];               // gathered copy: the survivors of the selected cells, cell after cell
    CellState* cst;              // per tensor of the group
    float* surv[3];              // survivors, each tile's compacted at the tile's own start
    u32* bm_w;                   // bitmaps, TILE_WORDS words per tile
    u32* bm_o;
    u32* tile_cnt_w;             // survivors per tile
    u32* tile_cnt_o;
    u32* tile_off_w;             // exclusive prefix of the counts within the tensor
    u32* tile_off_o;
};

struct KmArrays {                // further device arrays of the K-means stage alone
    u32* pending;                // streams whose first round of iterations met a cell that was not gathered
    u32* rows[3];                // per stream: survivors per cell of every (block, tensor) share of the counting
                                 //   sweep, row (block + tensor) of NCELL words
    u32* pos[3];                 // the same shape: where each share's values of a cell start in the gathered copy
};

struct Params {
    float alpha, beta;
    int bits, kmeans_iters;
    u64 seed;
    int median_source;
    u32 flags;                   // OPT_*
    int wfmt;                    // WeightFormat of w_t and w_prev
    int km_margin;               // cells gathered on either side of every predicted threshold (-1: none)
    u64 wait_ns;                 // how long a warp waits for an asynchronous copy before it gives up
};
__host__ __device__ inline int stored_bits(const Params& p) { return (p.flags & OPT_NO_QUANT) ? 32 : p.bits; }
__host__ __device__ inline u32 record_flags(const Params& p) {
    return ((p.flags & OPT_NO_W2M) ? REC_MOMENTS_FREE : 0u) | ((p.flags & OPT_NO_RESIDUAL) ? REC_ABSOLUTE : 0u) |
           ((p.flags & OPT_NO_QUANT) ? REC_RAW : 0u);
}

struct DecDesc {                 // decompress: one per tensor of a group
    const unsigned char* rec;    // start of the record
    u64 rec_avail;               // bytes the caller says belong to it
    const void* w_prev;          // fp32, fp16 or bf16 (the call's weight format), like w_out
    void* w_out;
    float* ea_out;
    float* eas_out;
    u64 numel;
    u32 tile_begin;
    u32 num_tiles;
    unsigned char* dense;        // record -> dense layout: where the container goes
    u64 dense_avail;             // and the room there
};

struct DecState {                // decompress scratch per tensor
    u32 valid;
    u32 bits;
    u32 nnz_w, nnz_o;
    u32 cnt_w, cnt_o;            // dense layout: non-zero codes met while decoding
    u32 rflags, pad_;            // the record's flags (REC_*)
    u64 off_bm_w, off_bm_o, off_codes[3];
    float cent[3][KCAP];
};

// ---- layout arithmetic (host and device) ----------------------------------
__host__ __device__ inline u64 align16(u64 n) { return (n + 15ull) & ~15ull; }
__host__ __device__ inline u64 header_bytes(int k) { return align16(HEADER_FIXED + 12ull * k); }
__host__ __device__ inline int centres_of(int bits) { return bits == 32 ? 0 : (1 << bits) - 1; }
__host__ __device__ inline u64 bitmap_bytes(u64 numel) { return align16(4ull * ((numel + 31) / 32)); }
__host__ __device__ inline u64 code_bytes(u64 nnz, int bits) { return align16((nnz * bits + 7) / 8); }
__host__ __device__ inline u64 dense_section_bytes(u64 numel, int bits) { return align16((numel * bits + 7) / 8); }
__host__ __device__ inline u64 dense_bytes(u64 numel, int bits) {
    return header_bytes((1 << bits) - 1) + 3 * dense_section_bytes(numel, bits);
}
__host__ __device__ inline u64 record_bytes(u64 numel, u64 nnz_w, u64 nnz_o, int bits) {
    return header_bytes(centres_of(bits)) + 2 * bitmap_bytes(numel) + code_bytes(nnz_w, bits) +
           2 * code_bytes(nnz_o, bits);
}

// ---- device helpers ---------------------------------------------------------
#ifdef __CUDACC__
// A warp gave up waiting for a copy somewhere in this call: every later kernel returns at once, so
// nothing is computed from arrays that were only partly written.
__device__ __forceinline__ bool call_aborted(const CallState* call) { return (call->flags & FLAG_TIMEOUT) != 0u; }

// The checked build (-DEXCP_DEBUG_BOUNDS): every index that depends on data is tested before it is
// used; a violation raises FLAG_INTERNAL (the call returns EXCP_ERR_CUDA) and the access is skipped.
// Nothing traps.  In the normal build the test is the constant `true`.
#ifdef EXCP_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(const CallState* call, bool in_bounds) {
    if (!in_bounds) atomicOr(const_cast<u32*>(&call->flags), FLAG_INTERNAL);
    return in_bounds;
}
#define EXCP_IN_BOUNDS(call, cond) bounds_ok((call), (cond))
#else
#define EXCP_IN_BOUNDS(call, cond) (true)
#endif

// Tensor that owns group tile `tile` (descs are in tile order).
__device__ inline int find_tensor(const TensorDesc* __restrict__ descs, int n, u32 tile) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (descs[mid].tile_begin <= tile) lo = mid; else hi = mid - 1;
    }
    return lo;
}
__device__ inline int find_tensor(const DecDesc* __restrict__ descs, int n, u32 tile) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (descs[mid].tile_begin <= tile) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// A stored weight as fp32 (exact: both 16-bit formats are subsets of fp32), and back (round to
// nearest even).
__device__ __forceinline__ float wget(const float* p, u64 i) { return p[i]; }
__device__ __forceinline__ float wget(const __half* p, u64 i) { return __half2float(p[i]); }
__device__ __forceinline__ float wget(const __nv_bfloat16* p, u64 i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void wput(float* p, u64 i, float v) { p[i] = v; }
__device__ __forceinline__ void wput(__half* p, u64 i, float v) { p[i] = __float2half_rn(v); }
__device__ __forceinline__ void wput(__nv_bfloat16* p, u64 i, float v) { p[i] = __float2bfloat16_rn(v); }

// Four consecutive 16-bit weights at i0 (a multiple of 4) as fp32; as load4 below.
template <typename WT>
__device__ inline int load4(const WT* __restrict__ p, u64 i0, u64 n, float v[4]) {
    if (i0 + 4 <= n) {
        const uint2 t = __ldcs(reinterpret_cast<const uint2*>(p + i0));
        const WT* h = reinterpret_cast<const WT*>(&t);
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = wget(h, k);
        return 4;
    }
    int c = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        if (i0 + k < n) { v[k] = wget(p, i0 + k); c = k + 1; } else v[k] = 0.f;
    }
    return c;
}
// Four results to weights i0..i0+3 (those that exist).
__device__ inline void store4(float* p, u64 i0, u64 n, const float v[4]) {
    if (i0 + 4 <= n) { *reinterpret_cast<float4*>(p + i0) = make_float4(v[0], v[1], v[2], v[3]); return; }
    for (int k = 0; k < 4 && i0 + k < n; ++k) p[i0 + k] = v[k];
}
template <typename WT>
__device__ inline void store4(WT* p, u64 i0, u64 n, const float v[4]) {
    if (i0 + 4 <= n) {
        uint2 t;
        WT* h = reinterpret_cast<WT*>(&t);
#pragma unroll
        for (int k = 0; k < 4; ++k) wput(h, k, v[k]);
        *reinterpret_cast<uint2*>(p + i0) = t;
        return;
    }
    for (int k = 0; k < 4 && i0 + k < n; ++k) wput(p, i0 + k, v[k]);
}

// Four consecutive elements starting at i0 (a multiple of 4).  Elements at or
// past n read as 0 and are reported through the return value (count valid).
__device__ inline int load4(const float* __restrict__ p, u64 i0, u64 n, float v[4]) {
    if (i0 + 4 <= n) {
        float4 t = __ldcs(reinterpret_cast<const float4*>(p + i0));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
        return 4;
    }
    int c = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        if (i0 + k < n) { v[k] = __ldcs(p + i0 + k); c = k + 1; } else v[k] = 0.f;
    }
    return c;
}

// Contiguous share of [0, total) for block b of g.
__device__ inline void block_range(u32 total, u32& lo, u32& hi) {
    lo = (u32)(((u64)total * blockIdx.x) / gridDim.x);
    hi = (u32)(((u64)total * (blockIdx.x + 1)) / gridDim.x);
}

__device__ inline u64 warp_sum_u64(u64 v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Exclusive prefix of the per-tile survivor counts of the tiles [tb, tb + ntl)
// (one tensor), written to tile_off_*; totals returned to every thread.
// Called by a whole block of TPB threads.
__device__ inline void scan_tile_counts(u32 tb, u32 ntl, const Workspace& ws, u32& tot_w, u32& tot_o) {
    __shared__ u32 wtot[2][TPB / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u32 carry_w = 0, carry_o = 0;
    for (u32 b0 = 0; b0 < ntl; b0 += TPB) {
        const u32 i = b0 + tid;
        const u32 cw = i < ntl ? ws.tile_cnt_w[tb + i] : 0u;
        const u32 co = i < ntl ? ws.tile_cnt_o[tb + i] : 0u;
        u32 iw = cw, io = co;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            u32 x = __shfl_up_sync(0xffffffffu, iw, o);
            u32 y = __shfl_up_sync(0xffffffffu, io, o);
            if (lane >= o) { iw += x; io += y; }
        }
        if (lane == 31) { wtot[0][warp] = iw; wtot[1][warp] = io; }
        __syncthreads();
        u32 bw = 0, bo = 0, tw = 0, to = 0;
#pragma unroll
        for (int w = 0; w < TPB / 32; ++w) {
            if (w < warp) { bw += wtot[0][w]; bo += wtot[1][w]; }
            tw += wtot[0][w]; to += wtot[1][w];
        }
        if (i < ntl) {
            ws.tile_off_w[tb + i] = carry_w + bw + iw - cw;
            ws.tile_off_o[tb + i] = carry_o + bo + io - co;
        }
        carry_w += tw; carry_o += to;
        __syncthreads();
    }
    tot_w = carry_w; tot_o = carry_o;
}
#endif

// ---- launch wrappers --------------------------------------------------------
enum Stage {                       // for the optional per-stage event timing
    ST_STATS1 = 0, ST_STATS2, ST_MASK_COMPACT, ST_SCAN_LAYOUT, ST_KMEANS_START, ST_CELL_COUNT, ST_CELL_GATHER,
    ST_KMEANS_ITERATE, ST_CELL_PLAN, ST_HEADER_EDGES, ST_PACK_CODES, ST_COPY_BITMAPS, ST_DEC_PREP,
    ST_DECODE, ST_KMEANS_RETRY, ST_DENSE, ST_COUNT
};

struct Profiler;
struct LaunchCfg {
    int sms;
    cudaStream_t stream;
    Profiler* prof;
};
// Counts `launches` kernel launches; with timing enabled also records an event
// that closes stage `stage` (implemented beside the handle).
void prof_mark(const LaunchCfg& cfg, int stage, int launches);

void launch_stats(const LaunchCfg&, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                  const Workspace& ws, const Params& p, CallState* call);
void launch_mask_compact(const LaunchCfg&, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                         const Workspace& ws, const Params& p, CallState* call, u64 blob_capacity);
void launch_kmeans(const LaunchCfg&, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                   const Workspace& ws, const KmArrays& km, const Params& p, CallState* call);
void launch_pack(const LaunchCfg&, const TensorDesc* descs, TensorState* st, int nt, u32 tiles,
                 const Workspace& ws, const Params& p, unsigned char* blob, CallState* call,
                 TensorResult* results, bool want_sse);
void launch_decode(const LaunchCfg&, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                   const Workspace& ws, CallState* call, int wfmt = WF_F32);
void launch_record_to_dense(const LaunchCfg&, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                            const Workspace& ws, CallState* call);
void launch_dense_decode(const LaunchCfg&, const DecDesc* descs, DecState* st, int nt, u32 tiles,
                         CallState* call);
void launch_wait_selftest(const LaunchCfg&, CallState* call, u64 limit_ns);

}  // namespace excp
