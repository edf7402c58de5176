// Thin wrappers over the sm_100a asynchronous-copy and mbarrier PTX used by both kernels.
// Every wait is bounded: it returns false instead of spinning forever.
#pragma once

#include <stdint.h>

namespace speckv {

constexpr uint32_t kWaitLimit = 1u << 24;            // polls of an mbarrier before a wait gives up
constexpr unsigned long long kWaitNs = 2000000000ull;   // ... or two seconds, whichever comes first

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for the phase with the given parity: gives up after limit_ns nanoseconds (or
// kWaitLimit polls), or as soon as `abort` (shared memory) becomes non-zero.  Each lane decides for
// itself: use it where a subset of lanes waits on barriers of their own.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int *abort = nullptr,
                                          unsigned long long limit_ns = kWaitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (abort && *abort) return false;
        if ((i & 63u) == 63u && global_ns() - t0 > limit_ns) return false;
    }
    return false;
}
// The same wait made by all 32 lanes of a warp, with one answer for the whole warp: lanes that gave up
// in the same instant in which others saw the phase complete look once more (a completed phase stays
// complete until this warp moves on), so the warp never splits into lanes that leave and lanes that stay.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const volatile int *abort = nullptr,
                                               unsigned long long limit_ns = kWaitNs)
{
    bool ok = mbar_try_wait(bar, parity);
    if (__all_sync(0xFFFFFFFFu, ok)) return true;
    if (!ok) ok = mbar_wait(bar, parity, abort, limit_ns);
    if (__all_sync(0xFFFFFFFFu, ok)) return true;
    if (!ok) ok = mbar_try_wait(bar, parity);
    return __all_sync(0xFFFFFFFFu, ok);
}
// bulk asynchronous copy global -> shared (bytes multiple of 16; both addresses 16-byte aligned);
// completion is signalled on the mbarrier as transaction bytes
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// asks for `bytes` (multiple of 16) at a 16-byte aligned global address to be brought into L2; a hint
__device__ __forceinline__ void prefetch_l2(const void *src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
// bulk asynchronous copy shared -> global, tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void bulk_s2g(void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// makes this thread's shared-memory writes visible to later asynchronous-proxy reads
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

}  // namespace speckv
