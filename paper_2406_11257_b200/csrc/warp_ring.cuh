// A warp's private ring of shared-memory stages fed by bulk asynchronous copies,
// and the cursor with which a warp walks the dense chunks of its run of tiles.
//
// The dense sweeps (statistics, mask + compaction, decode) are all built the same
// way: every warp owns a contiguous run of tiles, lane 0 keeps NS x CH values per
// stage in flight for the chunks ahead, the warp consumes chunk after chunk, and no
// warp ever waits for another one.
#pragma once
#include "excp_common.cuh"
#include "tma.cuh"

namespace excp {

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

template <int NS, int CH, int ST>
struct WarpRing {
    static constexpr int STAGE_FLOATS = NS * CH;
    float* buf;                    // ST stages of NS streams of CH values
    unsigned long long* bar;       // one barrier per stage
    u32 i_stage, c_stage, c_phase, inflight;
    u64 limit_ns;                  // how long a wait may last

    __device__ void init(float* b, unsigned long long* r, int lane, u64 wait_limit_ns) {
        buf = b; bar = r; i_stage = 0; c_stage = 0; c_phase = 0; inflight = 0; limit_ns = wait_limit_ns;
        if (lane == 0) {
            for (int s = 0; s < ST; ++s) mbar_init(&bar[s], 1);
            mbar_fence_init();
        }
        __syncwarp();
    }
    __device__ bool can_issue() const { return inflight < (u32)ST; }

    // Starts the copies of one chunk: bytes[k] bytes (a multiple of 16, possibly 0) from each
    // non-null source into stream k's slot of the stage.  Called by the whole warp; lane 0 talks
    // to the copy engine.
    __device__ void issue_bytes(int lane, const void* const (&src)[NS], const u32 (&bytes)[NS]) {
        if (lane == 0) {
            unsigned long long* b = &bar[i_stage];
            float* dst = buf + i_stage * STAGE_FLOATS;
            u32 total = 0;
#pragma unroll
            for (int k = 0; k < NS; ++k) total += src[k] != nullptr ? bytes[k] : 0u;
            if (total) {
                mbar_arrive_expect_tx(b, total);
#pragma unroll
                for (int k = 0; k < NS; ++k)
                    if (src[k] && bytes[k]) bulk_g2s(dst + k * CH, src[k], bytes[k], b);
            } else {
                mbar_arrive(b);
            }
        }
        i_stage = i_stage + 1 == (u32)ST ? 0u : i_stage + 1;
        ++inflight;
    }
    // The same for fp32 streams: `nbulk` values (a multiple of 4, possibly 0) from each source.
    __device__ void issue(int lane, const float* const (&src)[NS], u32 nbulk) {
        const void* vs[NS];
        u32 bytes[NS];
#pragma unroll
        for (int k = 0; k < NS; ++k) { vs[k] = src[k]; bytes[k] = nbulk * 4u; }
        issue_bytes(lane, vs, bytes);
    }
    // Blocks (bounded) until the oldest chunk in flight has landed.
    __device__ bool wait() { return mbar_wait_warp(&bar[c_stage], c_phase, limit_ns); }
    // After a wait that ran out: lets every copy still in flight land (each wait bounded by DRAIN_NS,
    // far above what a copy needs), so that the warp leaves with nothing writing into its stages.
    static constexpr u64 DRAIN_NS = 2000000000ull;
    __device__ void drain() {
        while (inflight) {
            mbar_wait_warp(&bar[c_stage], c_phase, DRAIN_NS);
            if (++c_stage == (u32)ST) { c_stage = 0; c_phase ^= 1u; }
            --inflight;
        }
    }
    __device__ const float* stage() const { return buf + c_stage * STAGE_FLOATS; }
    // Every lane is done reading the stage: it may be refilled.
    __device__ void release() {
        __syncwarp();
        if (++c_stage == (u32)ST) { c_stage = 0; c_phase ^= 1u; }
        --inflight;
    }
};

// A warp's position inside its run of tiles, in chunks of CH values.  The tensor is looked
// up once per tile (enter_tile); chunk arithmetic stays in 32 bits.
template <int CH>
struct TileWalk {
    static constexpr u32 CHUNKS_PER_TILE = TILE / CH;
    u32 tile, chunk;
    u32 tv;                        // values of this tile that exist (0..TILE)
    int tns;                       // tensor owning `tile` (-1: none yet)
    u32 tb, ntl;                   // that tensor's tile range
    u64 numel, toff;               // its size; offset of this tile's first value in it

    __device__ void start(u32 t) { tile = t; chunk = 0; tv = 0; tns = -1; tb = 0; ntl = 0; numel = 0; toff = 0; }
    // Call at the first chunk of every tile; true if the tensor changed.
    template <typename Desc>
    __device__ bool enter_tile(const Desc* __restrict__ descs, int nt) {
        bool changed = false;
        if (tns < 0 || tile >= tb + ntl) {
            tns = find_tensor(descs, nt, tile);
            tb = descs[tns].tile_begin; ntl = descs[tns].num_tiles; numel = descs[tns].numel;
            changed = true;
        }
        toff = (u64)(tile - tb) * TILE;
        tv = toff >= numel ? 0u : (u32)min((u64)TILE, numel - toff);
        return changed;
    }
    __device__ u32 valid() const {                      // values of this chunk that exist
        const u32 o = chunk * CH;
        return tv > o ? min((u32)CH, tv - o) : 0u;
    }
    __device__ u64 elem0() const { return toff + chunk * CH; }
    __device__ void next() { if (++chunk == CHUNKS_PER_TILE) { chunk = 0; ++tile; } }
};

// Four consecutive values at offset o (a multiple of 4) of a chunk: from the stage where the
// bulk copy brought them, from global memory for the ragged last values of a tensor, 0 past it.
template <typename WT>
__device__ __forceinline__ void fetch4w(const float* __restrict__ slot, const WT* __restrict__ g, u32 o,
                                        u32 nbulk, u32 valid, float out[4]) {
    const WT* st = reinterpret_cast<const WT*>(slot);     // a 16-bit stream fills the first half of its slot
    if (o + 4 <= nbulk) {
        const uint2 t = *reinterpret_cast<const uint2*>(st + o);
        const WT* h = reinterpret_cast<const WT*>(&t);
#pragma unroll
        for (int k = 0; k < 4; ++k) out[k] = wget(h, k);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const u32 i = o + k;
            out[k] = i < nbulk ? wget(st, i) : (i < valid ? wget(g, i) : 0.f);
        }
    }
}
__device__ __forceinline__ void fetch4(const float* __restrict__ st, const float* __restrict__ g, u32 o,
                                       u32 nbulk, u32 valid, float out[4]) {
    if (o + 4 <= nbulk) {
        const float4 t = *reinterpret_cast<const float4*>(st + o);
        out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const u32 i = o + k;
            out[k] = i < nbulk ? st[i] : (i < valid ? __ldg(g + i) : 0.f);
        }
    }
}

}  // namespace excp
