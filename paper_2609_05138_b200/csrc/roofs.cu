// Microbenchmarks that measure, on the GPU the library runs on, the on-chip
// ceilings the gather-accumulate sweep is measured against: L2->SM read
// bandwidth (128-bit loads and bulk copies into shared memory), the
// L1 / shared-memory -> register bandwidth, and the fp32 add issue rate.
// The paper reports its kernel against the L2 roof of its own card
// (Section 6, Table 3); these give the same denominators for this one.
#include "common.cuh"

namespace bmu {

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

// Every block sweeps the whole buffer (far larger than L1, resident in L2) with
// 128-bit loads that bypass L1, `rounds` times, each block starting at its own
// offset so that the blocks do not march in step.  Four blocks of 512 threads per
// SM with eight loads in flight per thread keep 256 KB per SM on the wing.
__global__ void __launch_bounds__(512, 4)
roof_l2_ldg_kernel(const uint4 *__restrict__ buf, size_t n_vec, int rounds, uint32_t *sink)
{
    uint4 acc = make_uint4(0, 0, 0, 0);
    const size_t start = ((size_t)blockIdx.x * 7919u * 512u) % n_vec;
    for (int r = 0; r < rounds; ++r) {
        for (size_t i = threadIdx.x; i < n_vec; i += 8 * 512) {
            const size_t a = start + i;
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                size_t idx = a + (size_t)u * 512;
                if (idx >= n_vec) idx -= n_vec;
                if (idx >= n_vec) idx -= n_vec;
                v[u] = __ldcg(buf + idx);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { acc.x ^= v[u].x; acc.y ^= v[u].y; acc.z ^= v[u].z; acc.w ^= v[u].w; }
        }
    }
    if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x12345677u) sink[0] = acc.x;
}

// Same sweep through bulk asynchronous copies (global -> shared, completion on
// an mbarrier): one thread per block keeps `DEPTH` copies of `piece` bytes in
// flight.  Waits are bounded; on timeout the block sets sink[1] and leaves.
template <int DEPTH>
__global__ void __launch_bounds__(32)
roof_l2_bulk_kernel(const char *__restrict__ buf, size_t bytes, int piece, int rounds,
                    uint32_t *sink)
{
    extern __shared__ __align__(128) char smem[];
    __shared__ __align__(8) unsigned long long bar[DEPTH];
    if (threadIdx.x != 0) return;
    for (int d = 0; d < DEPTH; ++d)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar[d])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const size_t n_piece = bytes / piece;
    const size_t start = ((size_t)blockIdx.x * 7919u) % n_piece;
    const size_t total = n_piece * (size_t)rounds;
    uint32_t phase = 0;      // bit d = parity of barrier d
    bool dead = false;
    for (size_t it = 0; it < total + DEPTH && !dead; ++it) {
        const int d = (int)(it % DEPTH);
        if (it >= DEPTH) {   // wait for the copy issued DEPTH iterations ago
            uint32_t ok = 0;
            for (int spin = 0; spin < (1 << 22) && !ok; ++spin)
                asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                             : "=r"(ok) : "r"(smem_u32(&bar[d])), "r"((phase >> d) & 1u) : "memory");
            if (!ok) { sink[1] = 1; dead = true; break; }
            phase ^= 1u << d;
        }
        if (it < total) {
            size_t p = start + it % n_piece;
            if (p >= n_piece) p -= n_piece;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(smem_u32(&bar[d])), "r"(piece) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(smem + (size_t)d * piece)), "l"(buf + p * piece), "r"(piece),
                           "r"(smem_u32(&bar[d])) : "memory");
        }
    }
}

// Loads and bulk copies at once, the way the tensor-core sweep pulls bytes into an SM: fifteen
// warps of a block sweep the buffer with 128-bit loads (as above) while up to sixteen threads
// of the sixteenth warp each keep MIX_DEPTH bulk copies of `piece` bytes in flight (as many
// threads as 64 KB of shared memory give buffers to), until the loading warps are done.  Bytes delivered by loads are known beforehand; the bytes the bulk
// copies delivered are counted in *bulk_bytes.  Waits are bounded (sink[1] on timeout).
static const int MIX_DEPTH = 4;
static const int MIX_SMEM = 65536;
__global__ void __launch_bounds__(512, 2)
roof_l2_mixed_kernel(const char *__restrict__ buf, size_t bytes, int piece, int issuers, int rounds,
                     unsigned long long *bulk_bytes, uint32_t *sink)
{
    extern __shared__ __align__(128) char smem[];
    __shared__ __align__(8) unsigned long long bar[16 * MIX_DEPTH];
    __shared__ uint32_t loaders_done;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int d = 0; d < 16 * MIX_DEPTH; ++d)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar[d])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        loaders_done = 0u;
    }
    __syncthreads();
    if (warp < 15) {
        const uint4 *vbuf = reinterpret_cast<const uint4 *>(buf);
        const size_t n_vec = bytes / 16;
        uint4 acc = make_uint4(0, 0, 0, 0);
        const size_t start = ((size_t)blockIdx.x * 7919u * 480u) % n_vec;
        for (int r = 0; r < rounds; ++r) {
            for (size_t i = threadIdx.x; i < n_vec; i += 8 * 480) {
                const size_t a = start + i;
                uint4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    size_t idx = a + (size_t)u * 480;
                    if (idx >= n_vec) idx -= n_vec;
                    if (idx >= n_vec) idx -= n_vec;
                    v[u] = __ldcg(vbuf + idx);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) { acc.x ^= v[u].x; acc.y ^= v[u].y; acc.z ^= v[u].z; acc.w ^= v[u].w; }
            }
        }
        if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x12345677u) sink[0] = acc.x;
        __syncwarp();
        if (lane == 0) atomicAdd(&loaders_done, 1u);
    } else if (lane < issuers) {
        volatile uint32_t *done = &loaders_done;
        char *mine = smem + (size_t)lane * MIX_DEPTH * piece;
        unsigned long long *mybar = bar + lane * MIX_DEPTH;
        const size_t n_piece = bytes / piece;
        size_t p = ((size_t)blockIdx.x * 7919u + (size_t)lane * 104729u) % n_piece;
        unsigned long long moved = 0;
        uint32_t phase = 0, inflight = 0;          // bit d: parity of barrier d / a copy is in flight
        bool dead = false;
        for (size_t it = 0; !dead; ++it) {
            const int d = (int)(it % MIX_DEPTH);
            if (inflight & (1u << d)) {
                uint32_t ok = 0;
                for (int spin = 0; spin < (1 << 22) && !ok; ++spin)
                    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                                 : "=r"(ok) : "r"(smem_u32(&mybar[d])), "r"((phase >> d) & 1u) : "memory");
                if (!ok) { sink[1] = 1; dead = true; break; }
                phase ^= 1u << d;
                inflight &= ~(1u << d);
                moved += (unsigned long long)piece;
            }
            if (*done >= 15u) {
                if (!inflight) break;
                continue;                              // drain what is still in flight
            }
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(smem_u32(&mybar[d])), "r"(piece) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_u32(mine + (size_t)d * piece)), "l"(buf + p * piece), "r"(piece),
                           "r"(smem_u32(&mybar[d])) : "memory");
            inflight |= 1u << d;
            if (++p >= n_piece) p = 0;
        }
        atomicAdd(bulk_bytes, moved);
    }
}

// Shared memory -> registers: conflict-free 128-bit loads from a block-local
// buffer, summed so that they cannot be dropped.
__global__ void __launch_bounds__(1024)
roof_smem_kernel(int iters, uint32_t *sink)
{
    __shared__ uint4 buf[2048];          // 32 KB
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) buf[i] = make_uint4(i, i * 3, i * 5, i * 7);
    __syncthreads();
    uint4 acc = make_uint4(0, 0, 0, 0);
    int idx = threadIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            uint4 v = buf[(idx + u * 160) & 2047];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        idx = (idx + 32) & 2047;
    }
    if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x12345677u) sink[0] = acc.x;
}

// L1-resident global loads -> registers (each block re-reads its own 64 KB).
__global__ void __launch_bounds__(1024)
roof_l1_kernel(const uint4 *__restrict__ buf, int iters, uint32_t *sink)
{
    const uint4 *mine = buf + (size_t)blockIdx.x * 4096;
    uint4 acc = make_uint4(0, 0, 0, 0);
    int idx = threadIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            uint4 v = __ldg(mine + ((idx + u * 416) & 4095));
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        idx = (idx + 32) & 4095;
    }
    if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x12345677u) sink[0] = acc.x;
}

// fp32 adds per second: independent chains of packed (PACKED) or scalar adds.
template <bool PACKED>
__global__ void __launch_bounds__(1024)
roof_fadd_kernel(int iters, float seed, uint32_t *sink)
{
    if constexpr (PACKED) {
        u64 a[8];
        const u64 w = ((u64)__float_as_uint(seed) << 32) | __float_as_uint(seed * 0.5f);
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = ((u64)(threadIdx.x + i) << 32) | (uint32_t)i;
        for (int it = 0; it < iters; ++it)
#pragma unroll
            for (int i = 0; i < 8; ++i) add2(a[i], w);
        u64 x = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) x ^= a[i];
        if (x == 0x123456789abcdefull) sink[0] = (uint32_t)x;
    } else {
        float a[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = (float)(threadIdx.x + i);
        for (int it = 0; it < iters; ++it)
#pragma unroll
            for (int i = 0; i < 16; ++i) a[i] += seed;
        float x = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) x += a[i];
        if (x == 0.12345f) sink[0] = __float_as_uint(x);
    }
}

static int timed(cudaStream_t s, float *ms, void (*launch)(void *), void *ctx)
{
    cudaEvent_t e0, e1;
    BMU_CUDA(cudaEventCreate(&e0));
    BMU_CUDA(cudaEventCreate(&e1));
    launch(ctx);                                  // warm-up
    BMU_CUDA(cudaEventRecord(e0, s));
    launch(ctx);
    BMU_CUDA(cudaEventRecord(e1, s));
    BMU_CUDA(cudaEventSynchronize(e1));
    BMU_CUDA(cudaGetLastError());
    BMU_CUDA(cudaEventElapsedTime(ms, e0, e1));
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return BMU_OK;
}

struct Ctx {
    int kind; cudaStream_t s; int sms; const char *buf; size_t bytes; int piece; int rounds;
    int iters; uint32_t *sink; int issuers; unsigned long long *bulk_bytes;
};

static void do_launch(void *p)
{
    Ctx &c = *static_cast<Ctx *>(p);
    switch (c.kind) {
    case 0: roof_l2_ldg_kernel<<<c.sms * 4, 512, 0, c.s>>>(reinterpret_cast<const uint4 *>(c.buf), c.bytes / 16, c.rounds, c.sink); break;
    case 1: roof_l2_bulk_kernel<8><<<c.sms * 4, 32, 8 * c.piece, c.s>>>(c.buf, c.bytes, c.piece, c.rounds, c.sink); break;
    case 2: roof_smem_kernel<<<c.sms, 1024, 0, c.s>>>(c.iters, c.sink); break;
    case 3: roof_l1_kernel<<<c.sms, 1024, 0, c.s>>>(reinterpret_cast<const uint4 *>(c.buf), c.iters, c.sink); break;
    case 4: roof_fadd_kernel<false><<<c.sms * 2, 1024, 0, c.s>>>(c.iters, 1.0f, c.sink); break;
    case 5: roof_fadd_kernel<true><<<c.sms * 2, 1024, 0, c.s>>>(c.iters, 1.0f, c.sink); break;
    case 6:
        cudaMemsetAsync(c.bulk_bytes, 0, sizeof(unsigned long long), c.s);
        roof_l2_mixed_kernel<<<c.sms * 2, 512, MIX_SMEM, c.s>>>(c.buf, c.bytes, c.piece, c.issuers, c.rounds,
                                                               c.bulk_bytes, c.sink);
        break;
    }
}

}  // namespace bmu

using namespace bmu;

extern "C" BMU_API int bmu_measure_roof(int which, void *buffer, size_t buffer_bytes, int piece,
                                        double *out_value, void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!out_value || which < 0 || which > 6) { set_error("bad argument"); return BMU_ERR_INVALID_ARG; }
    int dev = 0, sms = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    BMU_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (!buffer || buffer_bytes < ((size_t)1 << 20) || (reinterpret_cast<uintptr_t>(buffer) & 255)) {
        set_error("buffer must be 256-byte aligned device memory of at least 1 MiB");
        return BMU_ERR_WORKSPACE;
    }
    Ctx c;
    c.kind = which; c.s = s; c.sms = sms; c.sink = static_cast<uint32_t *>(buffer);
    c.buf = static_cast<const char *>(buffer) + 256;
    c.bytes = 0; c.piece = 0; c.rounds = 0; c.iters = 0; c.issuers = 0;
    c.bulk_bytes = reinterpret_cast<unsigned long long *>(static_cast<char *>(buffer) + 64);
    double work = 0;
    if (which == 6) {
        if (piece < 256 || piece % 16 || piece > MIX_SMEM / MIX_DEPTH) {
            set_error("piece must be a multiple of 16 in [256, %d]", MIX_SMEM / MIX_DEPTH);
            return BMU_ERR_INVALID_ARG;
        }
        size_t usable = (buffer_bytes - 256) / 65536 * 65536 / piece * piece / 16 * 16;
        c.bytes = usable; c.piece = piece;
        c.issuers = MIX_SMEM / (MIX_DEPTH * piece) < 16 ? MIX_SMEM / (MIX_DEPTH * piece) : 16;
        c.rounds = (int)(((size_t)2 << 30) / usable) / 2 + 1;   // about 1 GiB of loads per block
        work = (double)(usable / 16 * 16) * c.rounds * sms * 2;
        BMU_CUDA(cudaFuncSetAttribute(roof_l2_mixed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MIX_SMEM));
    } else if (which == 0 || which == 1) {
        size_t usable = (buffer_bytes - 256) / 65536 * 65536;
        if (which == 1) {
            if (piece < 16 || piece % 16 || piece > 24576) { set_error("piece must be a multiple of 16 in [16, 24576]"); return BMU_ERR_INVALID_ARG; }
            usable = usable / piece * piece;
            BMU_CUDA(cudaFuncSetAttribute(roof_l2_bulk_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * piece));
        }
        c.bytes = usable; c.piece = piece;
        c.rounds = (int)(((size_t)2 << 30) / usable) / 4 + 1;   // about 0.5 GiB per block
        work = (double)usable * c.rounds * sms * 4;
    } else if (which == 2 || which == 3) {
        if (which == 3 && buffer_bytes < 256 + (size_t)sms * 65536) { set_error("buffer too small"); return BMU_ERR_WORKSPACE; }
        c.iters = 20000;
        work = (double)c.iters * 8 * 16 * 1024 * sms;
    } else {
        c.iters = 40000;
        work = (double)c.iters * 16 * 1024 * sms * 2;
    }
    BMU_CUDA(cudaMemsetAsync(buffer, 0, 256, s));
    float ms = 0;
    int rc = timed(s, &ms, do_launch, &c);
    if (rc) return rc;
    uint32_t flags[2] = {0, 0};
    unsigned long long bulk = 0;
    BMU_CUDA(cudaMemcpyAsync(flags, buffer, sizeof(flags), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaMemcpyAsync(&bulk, c.bulk_bytes, sizeof(bulk), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    if (flags[1]) { set_error("bulk-copy wait timed out"); return BMU_ERR_TIMEOUT; }
    if (which == 6) work += (double)bulk;       // the bulk copies' share, counted by the kernel
    *out_value = work / (ms * 1e-3);
    return BMU_OK;
}
