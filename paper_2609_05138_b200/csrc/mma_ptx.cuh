// tcgen05 / mbarrier / bulk-copy PTX wrappers shared by the tensor-core sweeps.
#pragma once

#include "common.cuh"

namespace bmu {

static const uint32_t MMA_WAIT_LIMIT = 1u << 22;

// power of two that brings the largest head weight just below 2^15 (fp16 range)
__host__ __device__ __forceinline__ float head_scale(uint32_t max_bits)
{
#ifdef __CUDA_ARCH__
    const float mx = __uint_as_float(max_bits);
#else
    union { float f; uint32_t u; } c; c.u = max_bits; const float mx = c.f;
#endif
    if (!(mx > 0.f) || max_bits >= 0x7f800000u) return 1.f;
    int e;
    frexpf(mx, &e);
    int k = 15 - e;
    k = k > 127 ? 127 : (k < -126 ? -126 : k);
    return ldexpf(1.f, k);
}

__device__ __forceinline__ uint32_t mm_smem(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mm_bar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mm_bar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mm_bar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mm_bar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; "
                 "selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  The first wait of a block that runs out records `code` in the status word
// and raises the block's abort flag; every later wait of the block then returns at once.
__device__ __forceinline__ bool mm_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                        uint32_t *status, uint32_t code)
{
    if (*abort_flag) return false;
    for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin) {
        if (mm_bar_try(bar, parity)) return true;
        if ((spin & 255u) == 255u && *abort_flag) return false;
    }
    atomicOr(status, code);
    *abort_flag = 1u;
    return false;
}
__device__ __forceinline__ void mm_bulk_load(uint32_t dst, const void *src, uint32_t bytes,
                                             uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// shared-memory matrix descriptor: K-major, no swizzle; `lbo` = bytes between the two core
// matrices along K, `sbo` = bytes between groups of 8 rows
__device__ __forceinline__ u64 mm_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    return (u64)((addr >> 4) & 0x3fffu) | ((u64)(lbo >> 4) << 16) | ((u64)(sbo >> 4) << 32) |
           (1ull << 46);
}
// D[tmem] (+)= A[smem] * B[smem]^T, fp16 inputs, fp32 accumulate, M = 128, N = MMA_DOCS, K = 16
__device__ __forceinline__ void mm_mma(uint32_t tmem_d, u64 adesc, u64 bdesc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mm_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mm_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void mm_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void mm_tmem_ld8(uint32_t taddr, uint32_t v[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]),
                   "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr) : "memory");
}

__device__ __forceinline__ int mm_doc_of_lane(int lane)
{
    return ((lane & 1) << 2) | (lane & 2) | ((lane & 4) >> 2);
}


__device__ __forceinline__ void mm_tmem_ld16(uint32_t taddr, uint32_t v[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, "
                 "%10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]),
                   "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]),
                   "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr) : "memory");
}

}  // namespace bmu
