// Walking the survivor segments of a warp's run of tiles.
//
// After the mask sweep the survivors of tile t lie at the start of the tile's own
// 4096-value segment, tile_cnt[t] of them.  A warp owns a contiguous run of tiles; it reads
// the counts of 32 tiles at a time (one per lane), and streams the occupied parts of the
// segments through its ring of stages in chunks of CH values, NS streams side by side
// (the two moment streams share their counts).  Lane 0 keeps ST chunks in flight.
#pragma once
#include "excp_common.cuh"
#include "tma.cuh"

namespace excp {

template <int NS, int CH, int ST>
struct SegRing {
    static constexpr int STAGE_FLOATS = NS * CH;
    float* buf;
    unsigned long long* bar;
    u32 whi;                       // end of the warp's run of tiles
    u32 w0, wn;                    // current window: tiles [w0, w0 + wn), wn <= 32
    u32 mycnt;                     // count of tile w0 + lane (0 past the run)
    u32 nz;                        // lanes whose tile has survivors
    u32 it, i_cnt, ic;             // issue cursor: tile in the window (32 = done), its count, value offset
    u32 ct, c_cnt, cc;             // consume cursor
    u32 i_stage, c_stage, c_phase, inflight;

    __device__ void init(float* b, unsigned long long* r, int lane, u32 wlo, u32 whi_) {
        buf = b; bar = r; whi = whi_; w0 = wlo; wn = 0;
        i_stage = c_stage = c_phase = inflight = 0;
        it = ct = 32; i_cnt = c_cnt = ic = cc = 0; mycnt = 0; nz = 0;
        if (lane == 0) {
            for (int s = 0; s < ST; ++s) mbar_init(&bar[s], 1);
            mbar_fence_init();
        }
        __syncwarp();
    }
    // A new run of tiles for the same ring; nothing may be in flight (every issued chunk has been
    // consumed), so the barriers keep their phases.
    __device__ void restart(u32 wlo, u32 whi_) {
        whi = whi_; w0 = wlo; wn = 0;
        it = ct = 32; i_cnt = c_cnt = ic = cc = 0; mycnt = 0; nz = 0;
    }
    // first non-empty tile of the window after position i (i = -1: from the start); 32 if none
    __device__ u32 next_tile(int i) const {
        const u32 m = i >= 31 ? 0u : nz & (0xffffffffu << (i + 1));
        return m ? (u32)__ffs((int)m) - 1u : 32u;
    }
    __device__ u32 next_start() const { return w0 + wn; }
    __device__ u32 cnt_of(u32 i) const { return __shfl_sync(0xffffffffu, mycnt, i); }   // tile i of the window
    // Loads the next window, which ends before `limit` (and before the end of the run, and after
    // at most 32 tiles); false when the run is finished.
    __device__ bool next_window(const u32* __restrict__ tile_cnt, int lane, u32 limit) {
        w0 += wn;
        if (w0 >= whi) { wn = 0; return false; }
        wn = min(32u, min(limit, whi) - w0);
        mycnt = (u32)lane < wn ? min(tile_cnt[w0 + lane], (u32)TILE) : 0u;   // a count never leads out of its segment
        nz = __ballot_sync(0xffffffffu, mycnt != 0);
        it = ct = next_tile(-1);
        i_cnt = c_cnt = it < 32 ? __shfl_sync(0xffffffffu, mycnt, it) : 0u;
        ic = cc = 0;
        return true;
    }
    __device__ bool have() const { return ct < 32; }
    __device__ void issue_ahead(int lane, const float* const (&surv)[NS]) {
        while (it < 32 && inflight < (u32)ST) {
            if (lane == 0) {
                const u32 nel = min((u32)CH, i_cnt - ic);
                const u32 bytes = ((nel + 3u) & ~3u) * 4u;       // stays inside the tile's segment
                unsigned long long* b = &bar[i_stage];
                float* dst = buf + i_stage * STAGE_FLOATS;
                const u64 off = (u64)(w0 + it) * TILE + ic;
                mbar_arrive_expect_tx(b, NS * bytes);
#pragma unroll
                for (int k = 0; k < NS; ++k) bulk_g2s(dst + k * CH, surv[k] + off, bytes, b);
            }
            i_stage = i_stage + 1 == (u32)ST ? 0u : i_stage + 1;
            ++inflight;
            ic += CH;
            if (ic >= i_cnt) {
                ic = 0;
                it = next_tile((int)it);
                i_cnt = it < 32 ? __shfl_sync(0xffffffffu, mycnt, it) : 0u;
            }
        }
    }
    __device__ u32 tile() const { return w0 + ct; }
    __device__ u32 tile_cnt_cur() const { return c_cnt; }
    __device__ u32 off() const { return cc; }                                   // first value of the chunk in its segment
    __device__ u32 nel() const { return min((u32)CH, c_cnt - cc); }              // values in the chunk
    __device__ bool wait() { return mbar_wait_warp(&bar[c_stage], c_phase); }
    __device__ const float* stage() const { return buf + c_stage * STAGE_FLOATS; }
    __device__ void advance() {
        __syncwarp();                                   // every lane is done with the stage
        if (++c_stage == (u32)ST) { c_stage = 0; c_phase ^= 1u; }
        --inflight;
        cc += CH;
        if (cc >= c_cnt) {
            cc = 0;
            ct = next_tile((int)ct);
            c_cnt = ct < 32 ? __shfl_sync(0xffffffffu, mycnt, ct) : 0u;
        }
    }
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

}  // namespace excp
