// Tensor-core head + gathered tail: the sweep split by feature frequency.
//
// On a frequency-ordered vocabulary (the paper keeps that relabelling as
// substrate, Table 8) the few hundred most frequent features carry more than
// half of all neuron-feature updates, and the block of documents x frequent
// features is dense enough (about one entry in six) to be a real contraction.
// So the sum over a document's features is cut in two:
//
//   s_ij = sum_{f in x_i, f <  H} W[f][j]        head: binary X_head x W_head on
//                                                tcgen05 tensor cores, fp32
//                                                accumulators in tensor memory
//        + sum_{f in x_i, f >= H} W[f][j]        tail: gathered rows, as in the
//                                                tiled sweep
//
// A block carries 128 length-ordered documents through slabs of 512 neurons.
// Head: W_head is split beforehand (head_split_kernel) into fp16 hi + lo parts
// of W * 2^k -- hi + lo reproduces an fp32 weight to 2^-22 relative, X is exact,
// products are exact, the accumulator is fp32 -- and laid out in global memory as
// the very shared-memory images the MMA wants (K-major, no swizzle, 8 x 16-byte
// core matrices), so a pipeline stage is one plain 16 KB bulk copy.  The MMA is
// D[neuron][document] = W_head-tile[128 x K] * X_head[128 docs x K]^T with the
// neurons of a slab dealt to four accumulator tiles so that tensor-memory lane
// 32q + t of tile c holds neuron 128q + 4t + c: the thread that reads "its" lane
// from the four tiles gets four consecutive neurons (one 128-bit piece of a
// codebook row) for eight documents -- exactly the register layout of the tail.
// Tail: a warp takes 8 documents x 128 neurons, starts from the head sums read
// out of tensor memory and adds the remaining rows with 128-bit loads.
// One warp streams the stages, one thread issues the MMAs, sixteen warps sweep;
// the MMAs of the next slab run while the tail of this one is swept.  Every wait
// is bounded and reports through the status word.
#include "common.cuh"
#include "mma_ptx.cuh"

#include <cuda_fp16.h>
#include <math_constants.h>

namespace bmu {

#ifndef BMU_MMA_STAGES
#define BMU_MMA_STAGES 4
#endif
static const int MMA_NS = BMU_MMA_STAGES;            // ring stages
static const int MMA_TAIL_WARPS = MMA_DOCS / 8;      // 16
static const int MMA_THREADS = (MMA_TAIL_WARPS + 2) * 32;
static const int MMA_TMEM_COLS = 4 * MMA_DOCS;       // 512: four accumulator tiles
static inline size_t mma_smem_bytes(int head)
{
    return (size_t)MMA_DOCS * head * 2 + MMA_NS * MMA_STAGE_BYTES + (2 * MMA_NS + 3) * 8 +
           MMA_DOCS * 8 + 16;
}

__global__ void head_absmax_kernel(const float *__restrict__ W, int64_t M, int64_t m_full,
                                   int head, const uint16_t *__restrict__ feat,
                                   uint32_t *__restrict__ out)
{
    const int64_t n4 = m_full / 4, total = n4 * head;
    uint32_t mx = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t f = i / n4, c = i - f * n4;
        const int64_t row = feat ? (int64_t)feat[f] : f;
        const float4 v = __ldg(reinterpret_cast<const float4 *>(W + row * M) + c);
        mx = max(mx, __float_as_uint(fabsf(v.x)));
        mx = max(mx, __float_as_uint(fabsf(v.y)));
        mx = max(mx, __float_as_uint(fabsf(v.z)));
        mx = max(mx, __float_as_uint(fabsf(v.w)));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if ((threadIdx.x & 31) == 0 && mx) atomicMax(out, mx);
}

// One thread per (slab, group of 8 features, neuron): both fp16 parts of 8 weights, as one
// 16-byte row of a core matrix each.  Stage order inside a slab: tile c (neuron % 4), part
// (hi, lo), block of 64 features; inside a stage the core matrix of (8 rows, 8 features)
// lies at (row / 8) * 1024 + (feature / 8) * 128.
__global__ void __launch_bounds__(MMA_SLAB)
head_split_kernel(const float *__restrict__ W, int64_t M, int head, const uint16_t *__restrict__ feat,
                  const uint32_t *__restrict__ head_max, unsigned char *__restrict__ img)
{
    const int KB = head / 64, SPS = 8 * KB;
    const int sl = blockIdx.x, kcg = blockIdx.y, jin = threadIdx.x;
    const float S = head_scale(*head_max);
    const float *col = W + (int64_t)sl * MMA_SLAB + jin;
    __align__(16) __half hi[8];
    __align__(16) __half lo[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int64_t row = feat ? (int64_t)feat[kcg * 8 + e] : (int64_t)(kcg * 8 + e);
        const float w = __ldg(col + row * M) * S;
        hi[e] = __float2half_rn(w);
        lo[e] = __float2half_rn(w - __half2float(hi[e]));
    }
    const int c = jin & 3, r = ((jin >> 7) << 5) | ((jin >> 2) & 31);
    const int kb = kcg >> 3, kc = kcg & 7;
    const size_t off = (size_t)(r >> 3) * 1024 + (size_t)kc * 128 + (size_t)(r & 7) * 16;
    const size_t st_hi = (size_t)sl * SPS + (size_t)(c * 2 + 0) * KB + kb;
    const size_t st_lo = (size_t)sl * SPS + (size_t)(c * 2 + 1) * KB + kb;
    *reinterpret_cast<uint4 *>(img + st_hi * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(hi);
    *reinterpret_cast<uint4 *>(img + st_lo * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(lo);
}

size_t head_image_bytes(int64_t M, int head)
{
    return (size_t)(M / MMA_SLAB) * mma_stages_per_slab(head) * MMA_STAGE_BYTES;
}

// bit pattern of the largest |weight| among the head rows (both tensor-core sweeps)
int launch_head_absmax(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                       uint32_t *head_max, cudaStream_t s)
{
    BMU_CUDA(cudaMemsetAsync(head_max, 0, sizeof(uint32_t), s));
    head_absmax_kernel<<<592, 256, 0, s>>>(W, M, m_full, head, feat, head_max);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

int launch_head_split(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                      uint32_t *head_max, unsigned char *head_img, cudaStream_t s)
{
    if (m_full <= 0) return BMU_OK;
    int rc = launch_head_absmax(W, M, m_full, head, feat, head_max, s);
    if (rc) return rc;
    const dim3 grid((unsigned)(m_full / MMA_SLAB), head / 8);
    head_split_kernel<<<grid, MMA_SLAB, 0, s>>>(W, M, head, feat, head_max, head_img);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

__global__ void __launch_bounds__(MMA_THREADS, 1)
sweep_mma_kernel(const MmaArgs a)
{
    constexpr int T = 8;
    constexpr int NS = MMA_NS;
    constexpr int NTW = MMA_TAIL_WARPS;
    const int H = a.head, KB = H / 64, SPS = 8 * KB;           // stages per slab
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *xs = smem;                                   // X_head image, 128 docs x H
    unsigned char *ring = smem + (size_t)MMA_DOCS * H * 2;      // NS stages of W_head
    u64 *bars = reinterpret_cast<u64 *>(ring + NS * MMA_STAGE_BYTES);
    u64 *keys = bars + 2 * NS + 3;                              // running minimum per document
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(keys + MMA_DOCS);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    uint32_t *skip_flag = tmem_slot + 2;
    const uint32_t full0 = mm_smem(bars), empty0 = mm_smem(bars + NS);
    const uint32_t tmem_full = mm_smem(bars + 2 * NS), tmem_empty = mm_smem(bars + 2 * NS + 1);
    const uint32_t drain = mm_smem(bars + 2 * NS + 2);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t group = blockIdx.x;
    const int n_slabs = (a.j_hi - a.j_lo) / MMA_SLAB;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) {
            mm_bar_init(full0 + 8 * i, 1);
            mm_bar_init(empty0 + 8 * i, 1);
        }
        mm_bar_init(tmem_full, 1);
        mm_bar_init(tmem_empty, NTW);
        mm_bar_init(drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        *abort_flag = 0u;
        *skip_flag = *reinterpret_cast<volatile uint32_t *>(a.status);
    }
    __syncthreads();
    if (*skip_flag) return;          // a block before this one gave up: let the grid drain

    if (warp == NTW) {               // tensor memory for the four accumulator tiles
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(mm_smem(tmem_slot)), "r"((uint32_t)MMA_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // X_head of this block's documents as fp16 zeros and ones: document n, features 8*kc .. +7
    // at (n / 8) * (H * 16) + kc * 128 + (n % 8) * 16
    for (int idx = threadIdx.x; idx < MMA_DOCS * (H / 8); idx += MMA_THREADS) {
        const int n = idx & (MMA_DOCS - 1), kc = idx / MMA_DOCS;
        const int64_t tile = group * (MMA_DOCS / T) + (n >> 3);
        uint32_t bits = 0;
        if (tile < a.n_tiles)
            bits = (__ldcs(a.tile_head + (group * MMA_DOCS + n) * (H / 32) + (kc >> 2)) >>
                    ((kc & 3) * 8)) & 0xffu;
        uint4 v;
        v.x = ((bits & 1u) ? 0x3c00u : 0u) | ((bits & 2u) ? 0x3c000000u : 0u);
        v.y = ((bits & 4u) ? 0x3c00u : 0u) | ((bits & 8u) ? 0x3c000000u : 0u);
        v.z = ((bits & 16u) ? 0x3c00u : 0u) | ((bits & 32u) ? 0x3c000000u : 0u);
        v.w = ((bits & 64u) ? 0x3c00u : 0u) | ((bits & 128u) ? 0x3c000000u : 0u);
        *reinterpret_cast<uint4 *>(xs + (size_t)(n >> 3) * (H * 16) + (size_t)kc * 128 + (n & 7) * 16) = v;
    }
    if (threadIdx.x < MMA_DOCS) keys[threadIdx.x] = KEY_WORST;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == NTW) {
        // ---------------- producer: streams the stages of every slab through the ring
        if (lane == 0) {
            const unsigned char *src = a.head_img;
            const int total = n_slabs * SPS;
            int issued = 0;
            for (int c = 0; c < total; ++c) {
                const int slot = c % NS;
                if (c >= NS && !mm_wait(empty0 + 8 * slot, ((c / NS) - 1) & 1, abort_flag, a.status, 1u))
                    break;
                mm_bar_expect_tx(full0 + 8 * slot, (uint32_t)MMA_STAGE_BYTES);
                mm_bulk_load(mm_smem(ring + (size_t)slot * MMA_STAGE_BYTES),
                             src + (size_t)c * MMA_STAGE_BYTES, (uint32_t)MMA_STAGE_BYTES,
                             full0 + 8 * slot);
                issued = c + 1;
            }
            if (*abort_flag)         // gave up: let the copies in flight land before leaving
                for (int c = issued > NS ? issued - NS : 0; c < issued; ++c)
                    for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin)
                        if (mm_bar_try(full0 + 8 * (c % NS), (c / NS) & 1)) break;
        }
        __syncwarp();
    } else if (warp == NTW + 1) {
        // ---------------- one thread issues every MMA
        if (lane == 0) {
            // fp32 accumulate, fp16 A and B, both K-major, N = 128, M = 128
            const uint32_t idesc = (1u << 4) | ((uint32_t)(MMA_DOCS >> 3) << 17) | (8u << 24);
            const uint32_t ring_u32 = mm_smem(ring), xs_u32 = mm_smem(xs);
            bool ok = true;
            for (int sl = 0; sl < n_slabs && ok; ++sl) {
                if (sl > 0) ok = mm_wait(tmem_empty, (sl - 1) & 1, abort_flag, a.status, 2u);
                if (!ok) break;
                mm_fence_after();
                for (int i = 0; i < SPS; ++i) {
                    const int c = sl * SPS + i, slot = c % NS;
                    if (!mm_wait(full0 + 8 * slot, (c / NS) & 1, abort_flag, a.status, 4u)) {
                        ok = false;
                        break;
                    }
                    mm_fence_after();
                    const int tile_c = i / (2 * KB), kb = i % KB; // i = (tile * 2 + part) * KB + kb
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const u64 ad = mm_desc(ring_u32 + slot * (uint32_t)MMA_STAGE_BYTES + u * 256, 128, 1024);
                        const u64 bd = mm_desc(xs_u32 + (kb * 8 + 2 * u) * 128, 128, (uint32_t)H * 16);
                        mm_mma(tmem + tile_c * MMA_DOCS, ad, bd, idesc, ((i % (2 * KB)) | u) != 0);
                    }
                    mm_commit(empty0 + 8 * slot);                // stage free once these MMAs are done
                }
                if (ok) mm_commit(tmem_full);                    // head sums of the slab are complete
            }
            mm_commit(drain);                                    // nothing in flight past this point
            for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin)
                if (mm_bar_try(drain, 0)) break;
        }
        __syncwarp();
    } else {
        // ---------------- tail: 8 documents x 128 neurons per task
        const int q = warp & 3, g = warp >> 2;
        const float inv_s = 1.f / head_scale(__ldg(a.head_max));
        const uint32_t rowbytes = (uint32_t)(a.M * 4);
        const int mydoc = mm_doc_of_lane(lane);
        for (int sl = 0; sl < n_slabs; ++sl) {
            const int j0 = a.j_lo + sl * MMA_SLAB + q * 128;
            for (int it = 0; it < NTW / 4; ++it) {
                const int o = g + 4 * it;                        // the block's o-th tile of 8
                const int64_t tile = group * (MMA_DOCS / T) + o;
                const bool live = tile < a.n_tiles;
                u64 acc[T][2];
#pragma unroll
                for (int t = 0; t < T; ++t) acc[t][0] = acc[t][1] = 0ull;
                if (live) {
                    const uint32_t tl = __ldg(a.tile_len + tile);
                    const uint32_t rows = tl & 0xffffu, full = tl >> 16;
                    const uint4 *gp = a.tile_ids + __ldg(a.tile_off + tile);
                    const char *base = reinterpret_cast<const char *>(a.W + j0 + lane * 4);
                    uint32_t b = 0;
                    uint4 qn = __ldcs(gp);
                    for (; b < full; ++b) {
                        const uint4 qq = qn;
                        qn = __ldcs(gp + b + 1);
                        const uint32_t f[T] = {qq.x & 0xffffu, qq.x >> 16, qq.y & 0xffffu, qq.y >> 16,
                                               qq.z & 0xffffu, qq.z >> 16, qq.w & 0xffffu, qq.w >> 16};
                        ulonglong2 w[T];
    #pragma unroll
                        for (int t = 0; t < T; ++t)
                            w[t] = __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)f[t] * rowbytes));
    #pragma unroll
                        for (int t = 0; t < T; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
                    }
                    for (; b < rows; ++b) {                          // some documents have run out
                        const uint4 qq = qn;
                        qn = __ldcs(gp + b + 1);
                        const uint32_t f[T] = {qq.x & 0xffffu, qq.x >> 16, qq.y & 0xffffu, qq.y >> 16,
                                               qq.z & 0xffffu, qq.z >> 16, qq.w & 0xffffu, qq.w >> 16};
                        ulonglong2 w[T];
#pragma unroll
                        for (int t = 0; t < T; ++t)
                            w[t] = f[t] != 0xffffu
                                       ? __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)f[t] * rowbytes))
                                       : make_ulonglong2(0ull, 0ull);
#pragma unroll
                        for (int t = 0; t < T; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
                    }
                }
                // the head sums of these documents, from tensor memory: the MMAs of this slab ran
                // while the tail was being gathered
                if (it == 0) mm_wait(tmem_full, sl & 1, abort_flag, a.status, 8u);
                mm_fence_after();
                uint32_t hv[4][8];
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    mm_tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * MMA_DOCS + o * T), hv[c]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (it == NTW / 4 - 1) {                         // tensor memory may be overwritten
                    mm_fence_before();
                    __syncwarp();
                    if (lane == 0) mm_bar_arrive(tmem_empty);
                }
                if (!live) continue;
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    const float s0 = __uint_as_float(hv[0][t]) * inv_s, s1 = __uint_as_float(hv[1][t]) * inv_s;
                    const float s2 = __uint_as_float(hv[2][t]) * inv_s, s3 = __uint_as_float(hv[3][t]) * inv_s;
                    add2(acc[t][0], ((u64)__float_as_uint(s1) << 32) | __float_as_uint(s0));
                    add2(acc[t][1], ((u64)__float_as_uint(s3) << 32) | __float_as_uint(s2));
                }
                // distances, then the transposing butterfly of the tiled sweep
                const int col = j0 + lane * 4;
                const float4 n = __ldg(reinterpret_cast<const float4 *>(a.norms + col));
                const float n4[4] = {n.x, n.y, n.z, n.w};
                u64 k[T];
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    const float s4[4] = {lo_f(acc[t][0]), hi_f(acc[t][0]), lo_f(acc[t][1]), hi_f(acc[t][1])};
                    Best<false> bst;
                    bst.init();
#pragma unroll
                    for (int c = 0; c < 4; ++c) bst.push(fmaf(-2.f, s4[c], n4[c]), col + c);
                    k[t] = make_key(bst.d1, bst.j1);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const u64 send = (lane & 1) ? k[i] : k[i + 4];
                    const u64 keep = (lane & 1) ? k[i + 4] : k[i];
                    const u64 got = __shfl_xor_sync(0xffffffffu, send, 1);
                    k[i] = got < keep ? got : keep;
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const u64 send = (lane & 2) ? k[i] : k[i + 2];
                    const u64 keep = (lane & 2) ? k[i + 2] : k[i];
                    const u64 got = __shfl_xor_sync(0xffffffffu, send, 2);
                    k[i] = got < keep ? got : keep;
                }
                {
                    const u64 send = (lane & 4) ? k[0] : k[1];
                    const u64 keep = (lane & 4) ? k[1] : k[0];
                    const u64 got = __shfl_xor_sync(0xffffffffu, send, 4);
                    k[0] = got < keep ? got : keep;
                }
                u64 got = __shfl_xor_sync(0xffffffffu, k[0], 8);
                k[0] = got < k[0] ? got : k[0];
                got = __shfl_xor_sync(0xffffffffu, k[0], 16);
                k[0] = got < k[0] ? got : k[0];
                if (lane < T) atomicMin(reinterpret_cast<unsigned long long *>(keys + o * T + mydoc), k[0]);
            }
        }
        __syncwarp();
    }

    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    if (threadIdx.x < MMA_DOCS) {
        const int64_t p = group * MMA_DOCS + threadIdx.x;
        if (p < a.N) {
            const int32_t orig = __ldg(a.perm + p);
            Best<false>::commit(keys[threadIdx.x], KEY_WORST, a.state, nullptr, orig, a.first);
        }
    }
    if (warp == NTW)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)MMA_TMEM_COLS) : "memory");
}

int launch_sweep_mma(const MmaArgs &a, const bmu_opts &o, cudaStream_t s)
{
    (void)o;
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    if ((a.j_hi - a.j_lo) % MMA_SLAB != 0 || a.j_lo % MMA_SLAB != 0) {
        set_error("tensor-core sweep handles whole %d-neuron slabs only", MMA_SLAB);
        return BMU_ERR_INVALID_ARG;
    }
    if (a.head != 256 && a.head != 512) {
        set_error("tensor-core sweep: head_rows must be 256 or 512");
        return BMU_ERR_INVALID_ARG;
    }
    static bool configured[64];
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        BMU_CUDA(cudaFuncSetAttribute(sweep_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)mma_smem_bytes(MMA_HEAD_MAX)));
        configured[dev] = true;
    }
    const unsigned blocks = (unsigned)((a.N + MMA_DOCS - 1) / MMA_DOCS);
    sweep_mma_kernel<<<blocks, MMA_THREADS, mma_smem_bytes(a.head), s>>>(a);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
