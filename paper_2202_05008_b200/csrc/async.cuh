// mbarrier and bulk-copy (TMA, cp.async.bulk) primitives shared by the rollout kernels.
// Every wait is bounded: it gives up after a cycle budget so that a kernel can flag
// EVO_ERR_TIMEOUT and leave instead of hanging the device.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace evo {

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// One bulk copy global -> shared of `bytes` (multiple of 16, both addresses 16-byte aligned),
// completion counted on `bar` (which gets one arrival with the expected byte count).
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Bounded wait.  try_wait is given a suspend-time hint, so a waiting warp sleeps in hardware
// instead of taking issue slots from the warps that work; the loop re-arms it until the phase
// completes or ~2^(*max_cycles_log2) SM clocks have passed (the limit lives in the device status
// block, so a test can make it short).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, const uint32_t* max_cycles_log2)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    const long long t0 = clock64();
    const long long limit = 1ll << *max_cycles_log2;      // read only once the wait has to sleep
    for (;;) {
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity), "r"(20000u) : "memory");     // hint: 20 us
        if (done) return true;
        if (clock64() - t0 > limit) return false;
    }
}

}  // namespace evo
