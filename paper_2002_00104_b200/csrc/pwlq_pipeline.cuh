// Bulk asynchronous copies (the TMA engine's untiled cp.async.bulk, global -> shared, completion
// counted in bytes on an mbarrier) and mbarrier helpers for the HBM-bound streaming kernels: a CTA
// keeps the copies of its next spans in flight while it works on the current one, without
// spending registers on them.
//
// Rules kept here: source and destination 16-byte aligned, size a multiple of 16 bytes (spans
// that do not qualify are staged with ordinary loads instead); no multicast, no cluster; every
// wait is bounded and reports expiry instead of spinning forever.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace pwlq {

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// One poll may park the thread for up to kSuspendNs (a hint to the hardware), so that waiting
// threads do not compete for issue slots with the warps that already have their data.
constexpr unsigned kSuspendNs = 2000;
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity), "r"(kSuspendNs) : "memory");
    return ok != 0;
}
// Bounded wait: false after kMaxSpins unsuccessful polls, i.e. after about half a second, far
// longer than any copy can take.
constexpr int kMaxSpins = 1 << 18;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, int max_spins = kMaxSpins) {
    for (int i = 0; i < max_spins; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// The same with a pause between polls, for waits that are expected to last: the waiting warps
// then leave the issue slots to the warps that have work.
__device__ __forceinline__ bool mbar_wait_relaxed(uint64_t* bar, unsigned parity) {
    for (int i = 0; i < kMaxSpins; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(100);
    }
    return false;
}
// Makes the barrier initialisation visible to the asynchronous proxy.
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// Orders earlier generic-proxy accesses to shared memory before later asynchronous-proxy ones.
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, unsigned bytes,
                                              uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

}  // namespace pwlq
