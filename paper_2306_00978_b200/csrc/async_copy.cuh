// mbarrier, bulk-copy and bounded-wait helpers shared by the kernels that stage data
// through shared memory with the asynchronous copy engine.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace awq {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a wait gives up after ~2 s by default
constexpr unsigned int kTimeoutCode = 0x57A17u;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// non-blocking poll (try_wait may suspend the thread until the phase completes or a time limit)
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

struct WaitCtl {
    unsigned int* status;            // device status words (global memory): [0] code, [1] wait limit in us (0: default)
    volatile unsigned int* abort;    // block-wide "giving up" flag (shared memory)
};
// How long a wait may last: the default, or what awq_set_wait_limit_us stored (read on the slow
// path only, i.e. by a wait that is already waiting).
__device__ __forceinline__ unsigned long long wait_limit_ns(const WaitCtl& ctl) {
    const unsigned int us = *reinterpret_cast<volatile unsigned int*>(ctl.status + 1);
    return us ? (unsigned long long)us * 1000ull : kWaitLimitNs;
}
// Limit of the end-of-block drain (copies already issued must land before the block exits).
__device__ __forceinline__ unsigned long long drain_limit_ns(const WaitCtl& ctl) {
    const unsigned long long lim = wait_limit_ns(ctl);
    return lim < 200000000ull ? lim : 200000000ull;
}

// Bounded wait on an mbarrier phase.  Returns false once the block is giving up: either this
// wait ran out of time (it then records the time-out) or another thread's did.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtl& ctl) {
    if (*ctl.abort) return false;
    const unsigned long long t0 = global_ns(), limit = wait_limit_ns(ctl);
    for (unsigned int i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 0u) {
            if (*ctl.abort) return false;
            if (global_ns() - t0 > limit) {
                *ctl.abort = 1u;
                atomicExch(ctl.status, kTimeoutCode);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtl& ctl) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl);
}

// The same for warps whose wait may be long and is not latency-critical (copy and flush
// warps): sleep between polls so that the spinning does not take issue slots from the math warps.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, const WaitCtl& ctl) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns(), limit = wait_limit_ns(ctl);
    for (;;) {
        __nanosleep(128);
        if (mbar_try_wait(bar, parity)) return true;
        if (*ctl.abort) return false;
        if (global_ns() - t0 > limit) {
            *ctl.abort = 1u;
            atomicExch(ctl.status, kTimeoutCode);
            return false;
        }
    }
}

// global -> shared bulk copy (sizes and both addresses multiples of 16 bytes), completion
// counted in bytes on an mbarrier of this block
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// The same with an L2 eviction hint: data that is read exactly once (the packed weights of a
// matrix-vector product) should not push the activations and outputs out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
// hint: bring the 128-byte line at p into L2 (harmless if the line is rewritten later: L2 is coherent)
__device__ __forceinline__ void prefetch_l2(const void* p) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

}  // namespace awq
