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
    u32 w0, wn;                    // current window of up to 32 tiles
    u32 mycnt;                     // count of tile w0 + lane
    u32 it, ic;                    // issue cursor: tile within the window, value offset in its segment
    u32 ct, cc;                    // consume cursor
    u32 i_stage, c_stage, c_phase, inflight;

    __device__ void init(float* b, unsigned long long* r, int lane, u32 wlo, u32 whi_) {
        buf = b; bar = r; whi = whi_; w0 = wlo; wn = 0;
        i_stage = c_stage = c_phase = inflight = 0;
        if (lane == 0) {
            for (int s = 0; s < ST; ++s) mbar_init(&bar[s], 1);
            mbar_fence_init();
        }
        __syncwarp();
    }
    __device__ u32 cnt_of(u32 i) const { return __shfl_sync(0xffffffffu, mycnt, i); }
    // Loads the next window; false when the run is finished.  `first` on the first call.
    __device__ bool next_window(const u32* __restrict__ tile_cnt, int lane, bool first) {
        if (!first) w0 += 32;
        if (w0 >= whi) return false;
        wn = min(32u, whi - w0);
        mycnt = (u32)lane < wn ? tile_cnt[w0 + lane] : 0u;
        it = ic = ct = cc = 0;
        while (it < wn && cnt_of(it) == 0) ++it;
        ct = it;
        return true;
    }
    __device__ bool have() const { return ct < wn; }
    __device__ void issue_ahead(int lane, const float* const (&surv)[NS]) {
        while (it < wn && inflight < (u32)ST) {
            const u32 c = cnt_of(it);
            const u32 nel = min((u32)CH, c - ic);
            if (lane == 0) {
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
            if (ic >= c) {
                ic = 0; ++it;
                while (it < wn && cnt_of(it) == 0) ++it;
            }
        }
    }
    __device__ u32 tile() const { return w0 + ct; }
    __device__ u32 tile_cnt_cur() const { return cnt_of(ct); }
    __device__ u32 off() const { return cc; }                                   // first value of the chunk in its segment
    __device__ u32 nel() const { return min((u32)CH, cnt_of(ct) - cc); }         // values in the chunk
    __device__ bool wait() { return mbar_wait_warp(&bar[c_stage], c_phase); }
    __device__ const float* stage() const { return buf + c_stage * STAGE_FLOATS; }
    __device__ void advance() {
        __syncwarp();                                   // every lane is done with the stage
        if (++c_stage == (u32)ST) { c_stage = 0; c_phase ^= 1u; }
        --inflight;
        const u32 c = cnt_of(ct);
        cc += CH;
        if (cc >= c) {
            cc = 0; ++ct;
            while (ct < wn && cnt_of(ct) == 0) ++ct;
        }
    }
};

// Cluster of x = number of thresholds strictly below it.  thr_row: 16 fp32 thresholds
// (ascending, +inf from the 15th on) in shared memory; t3, t7, t11 are copies in registers.
// Returns 4 * cluster.
__device__ __forceinline__ u32 find_cluster4(float x, float t3, float t7, float t11, const char* thr_row) {
    u32 p = x > t7 ? 32u : 0u;
    p += (x > (p ? t11 : t3)) ? 16u : 0u;
    p += (x > *reinterpret_cast<const float*>(thr_row + p + 4)) ? 8u : 0u;
    p += (x > *reinterpret_cast<const float*>(thr_row + p)) ? 4u : 0u;
    return p;
}

}  // namespace excp
