// Bulk asynchronous copies global -> shared memory (the TMA engine's 1-D form,
// cp.async.bulk) completing on an mbarrier.  No multicast, no cluster: every
// copy lands in the issuing CTA's own shared memory.
//
// Rules the callers keep: source and destination 16-byte aligned, size a
// multiple of 16 bytes; a waiting warp polls until a deadline and gives up as a whole
// (so that no thread is left behind at a later barrier), reporting through a flag.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace excp {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the asynchronous proxy.
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// One arrival that also announces `bytes` of copies to come.
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok;
}

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Whole-warp wait for phase `parity`; false once `limit_ns` nanoseconds have passed without it
// (the caller sets an error flag, lets its other copies land and leaves as a warp).  A healthy
// copy completes within microseconds.
__device__ __forceinline__ bool mbar_wait_warp(unsigned long long* bar, uint32_t parity, unsigned long long limit_ns) {
    if (limit_ns == 0) return false;                             // no time at all: every wait fails (exercises the error path)
    for (uint32_t i = 0; i < 16; ++i)
        if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        const bool late = global_ns() - t0 > limit_ns;
        if (__any_sync(0xffffffffu, late)) return false;         // one clock reading decides for the warp
        __nanosleep(200);
    }
}

}  // namespace excp
