// Thin wrappers over the mbarrier / asynchronous-store PTX used for data-driven synchronisation
// between the CTAs of a cluster (sm_90+ instructions, compiled for sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ unsigned cta_smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ unsigned cluster_addr(unsigned local_addr, unsigned rank) {
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void mbarrier_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// one arrival plus the number of bytes this phase is going to receive
__device__ __forceinline__ void mbarrier_arrive_expect(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbarrier_test(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Waits for the phase with the given parity, at most `limit` clocks.  Returns false on expiry.
__device__ __forceinline__ bool mbarrier_wait_bounded(unsigned bar, unsigned parity, long long limit) {
    if (mbarrier_test(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbarrier_test(bar, parity))
        if (clock64() - t0 > limit) return false;
    return true;
}

// 16-byte store into another CTA's shared memory that reports its bytes to an mbarrier of that CTA
__device__ __forceinline__ void st_async_16(unsigned remote_addr, uint4 v, unsigned remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(
                     remote_addr),
                 "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(remote_bar)
                 : "memory");
}

}  // namespace
