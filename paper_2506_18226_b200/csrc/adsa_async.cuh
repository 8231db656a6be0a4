// Asynchronous-copy plumbing shared by the staged kernels: mbarrier and bulk-copy PTX wrappers,
// bounded waits, and the merge of two online-softmax states.
#pragma once

#include "adsa_dev.cuh"

namespace adsa {

constexpr int kCopySpinLimit = 1 << 20;          // polls of one mbarrier before a block gives up on it
constexpr int kCopySpinAfterTimeout = 1 << 10;   // once a wait has run out, later waits of that thread are short
constexpr int kInputSpinLimit = 1 << 19;         // polls (a load and a 200 ns sleep each) of an inputs-have-landed word: about a second

// ---- PTX wrappers ---------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int limit)
{
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> this CTA's shared memory; dst, src 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds128(const void *p) { return *reinterpret_cast<const uint4 *>(p); }

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// wait with a pause between polls, for waits that are normally long (a whole ring round)
__device__ __forceinline__ bool mbar_wait_sleepy(uint32_t bar, uint32_t parity, int limit)
{
    for (int i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 4) __nanosleep(64);
    }
    return false;
}

// merge online-softmax state (m2, l2, a2) into (m, l, a); logits are in log2 units
__device__ __forceinline__ void merge2(float &m, float &l, float (&a)[8], float m2, float l2, const float (&a2)[8])
{
    float M = fmaxf(m, m2);
    float w1 = exp2f(m - M), w2 = exp2f(m2 - M);
    l = l * w1 + l2 * w2;
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = a[e] * w1 + a2[e] * w2;
    m = M;
}

}  // namespace adsa
