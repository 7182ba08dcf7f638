// Tensor-core head + gathered tail, second cut: a wide head with double-buffered
// tensor memory.
//
// Same split of the sum as sweep_mma.cu -- the H most frequent features on tcgen05
// MMAs, the rest gathered -- re-cut so that the head can be much wider (up to 1024
// features, which takes the features present in about one document in a hundred
// and more away from the gather):
//   * a slab is 256 neurons and has two accumulator tiles (tensor-memory lane
//     32q + 16h + i of tile c = neuron 64q + 4i + 2h + c), so the head sums of a slab take
//     half of tensor memory and the MMAs of slab s+1 fill one half while the tail
//     of slab s is gathered against the other: the MMAs have a whole slab's time,
//     not the gap between two slabs;
//   * the K dimension is outermost: for every block of 64 features one warp
//     expands the documents' mask bits into a 128 x 64 fp16 operand (a 16 KB stage
//     of a small ring), used by the four W stages of that block (2 tiles x (hi,
//     lo)); shared memory holds rings and 16 KB of masks instead of the whole
//     X_head, so L1 keeps its size whatever H is;
//   * a tail task is 16 documents x 64 neurons: a lane gathers four neurons for
//     eight of the documents, so a load instruction still moves 512 bytes (two
//     rows, one per half of the documents) and eight are in flight per warp.
#include "sweep_mma2_common.cuh"

#include <cuda_fp16.h>
#include <math_constants.h>

namespace bmu {

#ifndef BMU_M2_WSTAGES
#define BMU_M2_WSTAGES 4
#endif
#ifndef BMU_M2_XSTAGES
#define BMU_M2_XSTAGES 3
#endif
static const int M2_NS = BMU_M2_WSTAGES;             // W ring stages
static const int M2_NX = BMU_M2_XSTAGES;             // X ring stages
static const int M2_THREADS = (M2_TAIL_WARPS + 3) * 32;

static inline size_t m2_smem_bytes(int head, bool top2)
{
    return (size_t)MMA_DOCS * (head / 8) + (M2_NS + M2_NX) * MMA_STAGE_BYTES +
           (2 * M2_NS + 2 * M2_NX + 6) * 8 + MMA_DOCS * 8 + 16 + 16 * 16 + 2 * 16 * 4 +
           16 * 8 + (top2 ? 4 * MMA_DOCS * 16 : 0);
}

// bit pattern of the largest |weight| among the head rows: sets the power-of-two scale of the
// fp16 split
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

int launch_head_absmax(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                       uint32_t *head_max, cudaStream_t s)
{
    BMU_CUDA(cudaMemsetAsync(head_max, 0, sizeof(uint32_t), s));
    { head_absmax_kernel<<<592, 256, 0, s>>>(W, M, m_full, head, feat, head_max); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

// One thread per (slab, group of 8 features, neuron).  Stage order inside a slab: block of
// 64 features, tile c (neuron % 2), part (hi, lo).
__global__ void __launch_bounds__(M2_SLAB)
head_split2_kernel(const float *__restrict__ W, int64_t M, const uint32_t *__restrict__ head_max,
                   int head, const uint16_t *__restrict__ feat, unsigned char *__restrict__ img)
{
    const int sl = blockIdx.x, kcg = blockIdx.y, jin = threadIdx.x;
    const int SPS = 4 * (head / 64);
    const float S = head_scale(*head_max);
    const float *col = W + (int64_t)sl * M2_SLAB + jin;
    __align__(16) __half hi[8];
    __align__(16) __half lo[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int64_t row = feat ? (int64_t)feat[kcg * 8 + e] : (int64_t)(kcg * 8 + e);
        const float w = __ldg(col + row * M) * S;
        hi[e] = __float2half_rn(w);
        lo[e] = __float2half_rn(w - __half2float(hi[e]));
    }
    // neuron 64q + 4i + 2h + c sits in row 32q + 16h + i of tile c
    const int c = jin & 1, r = ((jin >> 6) << 5) | (((jin >> 1) & 1) << 4) | ((jin >> 2) & 15);
    const int kb = kcg >> 3, kc = kcg & 7;
    const size_t off = (size_t)(r >> 3) * 1024 + (size_t)kc * 128 + (size_t)(r & 7) * 16;
    const size_t st = (size_t)sl * SPS + (size_t)(kb * 2 + c) * 2;
    *reinterpret_cast<uint4 *>(img + st * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(hi);
    *reinterpret_cast<uint4 *>(img + (st + 1) * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(lo);
}

size_t head_image2_bytes(int64_t M, int head)
{
    return (size_t)(M / M2_SLAB) * 4 * (head / 64) * MMA_STAGE_BYTES;
}

int launch_head_split2(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                       uint32_t *head_max, unsigned char *head_img, cudaStream_t s)
{
    if (m_full <= 0) return BMU_OK;
    int rc = launch_head_absmax(W, M, m_full, head, feat, head_max, s);
    if (rc) return rc;
    const dim3 grid((unsigned)(m_full / M2_SLAB), head / 8);
    { head_split2_kernel<<<grid, M2_SLAB, 0, s>>>(W, M, head_max, head, feat, head_img); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

// TOP2: also the second-best unit (Table 5: the paper's kernel tracks it for topographic error)
template <bool TOP2>
__global__ void __launch_bounds__(M2_THREADS, 1)
sweep_mma2_kernel(const MmaArgs a)
{
    constexpr int NS = M2_NS, NX = M2_NX, NTW = M2_TAIL_WARPS;
    const int H = a.head, KB = H / 64;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *masks = smem;                                 // 128 documents x H bits
    unsigned char *xring = smem + (size_t)MMA_DOCS * (H / 8);    // NX stages of X_head
    unsigned char *wring = xring + NX * MMA_STAGE_BYTES;         // NS stages of W_head
    u64 *bars = reinterpret_cast<u64 *>(wring + NS * MMA_STAGE_BYTES);
    u64 *keys = bars + 2 * NS + 2 * NX + 6;                      // (16-byte aligned)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(keys + MMA_DOCS);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    uint32_t *skip_flag = tmem_slot + 2;
    // the block's 16 tiles: first row of each id matrix, its length word and its offset
    uint4 *s_first = reinterpret_cast<uint4 *>(tmem_slot + 4);
    uint32_t *s_len = reinterpret_cast<uint32_t *>(s_first + 16);
    uint32_t *s_off = s_len + 16;
    // TOP2: (best, second) per neuron quarter and document; the warp that owns a quarter of a
    // document is the same in every slab, so it merges without atomics
    uint2 *lut = reinterpret_cast<uint2 *>(s_off + 16);          // 4 mask bits -> 4 fp16 zeros and ones
    u64 *kq = reinterpret_cast<u64 *>(lut + 16);
    const M2Bars<NS, NX> bar(bars);
    const uint32_t tfull0 = bar.tfull0, tempty0 = bar.tempty0;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t group = blockIdx.x;
    const int n_slabs = (a.j_hi - a.j_lo) / M2_SLAB;

    if (threadIdx.x == 0) {
        bar.init();
        *abort_flag = 0u;
        *skip_flag = *reinterpret_cast<volatile uint32_t *>(a.status);
    }
    __syncthreads();
    if (*skip_flag) return;          // a block before this one gave up: let the grid drain

    if (warp == NTW) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(mm_smem(tmem_slot)), "r"((uint32_t)M2_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    m2_block_setup<M2_THREADS, TOP2>(a, group, H, masks, keys, lut, kq, s_first, s_len, s_off);
    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (warp == NTW) {
        // ---------------- producer: W stages of every slab (2 tiles x (hi, lo) per 64 features)
        if (lane == 0) m2_producer<NS, NX, 4>(a, n_slabs, KB, wring, bar, abort_flag);
        __syncwarp();
    } else if (warp == NTW + 1) {
        // ---------------- expander: X_head, one block of 64 features per stage
        m2_expander<NS, NX>(a, n_slabs, KB, H, masks, xring, lut, bar, abort_flag, lane);
    } else if (warp == NTW + 2) {
        // ---------------- one thread issues every MMA
        if (lane == 0) m2_issuer<NS, NX, 2>(a, n_slabs, KB, tmem, wring, xring, bar, abort_flag);
        __syncwarp();
    } else {
        // ---------------- tail: 16 documents x 64 neurons per task.  Lane (h, i) = (lane / 16,
        // lane % 16) gathers neurons 4i .. 4i+3 for the documents 8h .. 8h+7 of the task: one
        // 128-bit load per lane and row, two rows (one per half-warp) per instruction.
        const int q = warp & 3, g = warp >> 2;
        const int li = lane & 15, lh = lane >> 4;
        const float inv_s = 1.f / head_scale(__ldg(a.head_max));
        const uint32_t rowbytes = (uint32_t)(a.M * 4);
        const int mydoc = 8 * lh + ((lane & 1) << 2 | (lane & 2) | ((lane >> 2) & 1));
        for (int sl = 0; sl < n_slabs; ++sl) {
            const int buf = sl & 1;
            const int j0 = a.j_lo + sl * M2_SLAB + q * 64;
            for (int it = 0; it < 2; ++it) {
                const int dg = g + 4 * it;                       // the block's dg-th set of 16
                const int64_t tile_a = group * (MMA_DOCS / 8) + 2 * dg, tile_b = tile_a + 1;
                const bool live = tile_a < a.n_tiles;
                u64 acc[8][2];
#pragma unroll
                for (int t = 0; t < 8; ++t) acc[t][0] = acc[t][1] = 0ull;
                if (live) {
                    const bool has_b = tile_b < a.n_tiles;
                    const uint32_t tla = s_len[2 * dg], tlb = s_len[2 * dg + 1];
                    const uint32_t full = min(tla >> 16, tlb >> 16);
                    const uint32_t rows = max(tla & 0xffffu, tlb & 0xffffu);
                    const uint32_t my_rows = (lh ? tlb : tla) & 0xffffu;
                    const int mine = 2 * dg + ((lh && has_b) ? 1 : 0);
                    const uint4 *gp = a.tile_ids + BMU_IDX(s_off[mine], a.tile_rows_cap, a.status);
                    [[maybe_unused]] const size_t room = a.tile_rows_cap - (size_t)(gp - a.tile_ids);
                    const char *base = reinterpret_cast<const char *>(a.W + j0 + li * 4);
                    uint32_t b = 0;
                    uint4 qn = s_first[mine];
                    for (; b < full; ++b) {
                        uint32_t f[8];
                        m2_unpack(qn, f);
                        qn = __ldcs(gp + BMU_IDX(b + 1, room, a.status));
                        ulonglong2 w[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t)
                            w[t] = __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)BMU_IDX(f[t], a.D, a.status) * rowbytes));
#pragma unroll
                        for (int t = 0; t < 8; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
                    }
                    for (; b < rows; ++b) {                      // some documents have run out
                        uint32_t f[8];
                        m2_unpack(qn, f);
                        qn = __ldcs(gp + BMU_IDX(b + 1, room, a.status));
                        const bool in = b < my_rows;
                        ulonglong2 w[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t)
                            w[t] = (in && f[t] != 0xffffu)
                                       ? __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)BMU_IDX(f[t], a.D, a.status) * rowbytes))
                                       : make_ulonglong2(0ull, 0ull);
#pragma unroll
                        for (int t = 0; t < 8; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
                    }
                }
                // head sums of these documents: the MMAs of this slab ran during the gather.
                // Tensor-memory lane 32q + lane holds neurons 4i + 2h, 4i + 2h + 1 for all 16
                // documents; lanes l and l ^ 16 swap halves so that each ends up with four
                // neurons of its own eight documents.
                if (it == 0) mm_wait(tfull0 + 8 * buf, (sl >> 1) & 1, abort_flag, a.status, 8u);
                mm_fence_after();
                uint32_t h0[16], h1[16];
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + dg * 16);
                BMU_EXPECT(buf * 256 + dg * 16 + MMA_DOCS + 16 <= M2_TMEM_COLS, a.status);
                mm_tmem_ld16(taddr, h0);
                mm_tmem_ld16(taddr + MMA_DOCS, h1);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (it == 1) {                                   // this half of tensor memory is free
                    mm_fence_before();
                    __syncwarp();
                    if (lane == 0) mm_bar_arrive(tempty0 + 8 * buf);
                }
                if (!live) continue;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const uint32_t mine0 = lh ? h0[8 + t] : h0[t], mine1 = lh ? h1[8 + t] : h1[t];
                    const uint32_t send0 = lh ? h0[t] : h0[8 + t], send1 = lh ? h1[t] : h1[8 + t];
                    const uint32_t got0 = __shfl_xor_sync(0xffffffffu, send0, 16);
                    const uint32_t got1 = __shfl_xor_sync(0xffffffffu, send1, 16);
                    const float s0 = __uint_as_float(lh ? got0 : mine0) * inv_s;
                    const float s1 = __uint_as_float(lh ? got1 : mine1) * inv_s;
                    const float s2 = __uint_as_float(lh ? mine0 : got0) * inv_s;
                    const float s3 = __uint_as_float(lh ? mine1 : got1) * inv_s;
                    add2(acc[t][0], ((u64)__float_as_uint(s1) << 32) | __float_as_uint(s0));
                    add2(acc[t][1], ((u64)__float_as_uint(s3) << 32) | __float_as_uint(s2));
                }
                const int col = j0 + li * 4;
                const float4 n = __ldg(reinterpret_cast<const float4 *>(a.norms + col));
                const float n4[4] = {n.x, n.y, n.z, n.w};
                u64 k[8], k2[8];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const float s4[4] = {lo_f(acc[t][0]), hi_f(acc[t][0]), lo_f(acc[t][1]), hi_f(acc[t][1])};
                    Best<TOP2> bst;
                    bst.init();
#pragma unroll
                    for (int c = 0; c < 4; ++c) bst.push(fmaf(-2.f, s4[c], n4[c]), col + c);
                    k[t] = make_key(bst.d1, bst.j1);
                    k2[t] = TOP2 ? make_key(bst.d2, bst.j2) : KEY_WORST;
                }
                // transposing butterfly among the 16 lanes that hold the same documents
#pragma unroll
                for (int st = 0; st < 3; ++st) {
                    const int m = 1 << st, cnt = 4 >> st;
#pragma unroll
                    for (int i = 0; i < cnt; ++i) {
                        const u64 send = (lane & m) ? k[i] : k[i + cnt];
                        const u64 keep = (lane & m) ? k[i + cnt] : k[i];
                        const u64 got = __shfl_xor_sync(0xffffffffu, send, m);
                        if (TOP2) {
                            const u64 send2 = (lane & m) ? k2[i] : k2[i + cnt];
                            u64 keep2 = (lane & m) ? k2[i + cnt] : k2[i];
                            const u64 got2 = __shfl_xor_sync(0xffffffffu, send2, m);
                            u64 b1 = keep;
                            Best<true>::merge(b1, keep2, got, got2);
                            k[i] = b1;
                            k2[i] = keep2;
                        } else {
                            k[i] = got < keep ? got : keep;
                        }
                    }
                }
                const u64 got = __shfl_xor_sync(0xffffffffu, k[0], 8);
                if (TOP2) {
                    const u64 got2 = __shfl_xor_sync(0xffffffffu, k2[0], 8);
                    Best<true>::merge(k[0], k2[0], got, got2);
                    if ((lane & 8) == 0) {
                        u64 *slot = kq + ((size_t)q * MMA_DOCS + dg * 16 + mydoc) * 2;
                        Best<true>::merge(k[0], k2[0], slot[0], slot[1]);
                        slot[0] = k[0];
                        slot[1] = k2[0];
                    }
                } else {
                    k[0] = got < k[0] ? got : k[0];
                    if ((lane & 8) == 0)
                        atomicMin(reinterpret_cast<unsigned long long *>(keys + dg * 16 + mydoc), k[0]);
                }
            }
        }
        __syncwarp();
    }

    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    m2_commit<TOP2>(a, group, keys, kq);
    if (warp == NTW)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)M2_TMEM_COLS) : "memory");
}

int launch_sweep_mma2(const MmaArgs &a, const bmu_opts &o, cudaStream_t s)
{
    (void)o;
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    if ((a.j_hi - a.j_lo) % M2_SLAB != 0 || a.j_lo % M2_SLAB != 0) {
        set_error("wide-head sweep handles whole %d-neuron slabs only", M2_SLAB);
        return BMU_ERR_INVALID_ARG;
    }
    if (a.head < 64 || a.head > HEAD_ROWS_MAX || a.head % 64 != 0) {
        set_error("wide-head sweep: head_rows must be a multiple of 64 up to %d", HEAD_ROWS_MAX);
        return BMU_ERR_INVALID_ARG;
    }
    static bool configured[64];
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        BMU_CUDA(cudaFuncSetAttribute(sweep_mma2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)m2_smem_bytes(HEAD_ROWS_MAX, false)));
        BMU_CUDA(cudaFuncSetAttribute(sweep_mma2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)m2_smem_bytes(HEAD_ROWS_MAX, true)));
        configured[dev] = true;
    }
    const unsigned blocks = (unsigned)((a.N + MMA_DOCS - 1) / MMA_DOCS);
    if (a.state2) { sweep_mma2_kernel<true><<<blocks, M2_THREADS, m2_smem_bytes(a.head, true), s>>>(a); BMU_LAUNCHED(); }
    else { sweep_mma2_kernel<false><<<blocks, M2_THREADS, m2_smem_bytes(a.head, false), s>>>(a); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

// A wait that cannot succeed: one mbarrier that nothing ever arrives on.  It shows
// that a wait which runs out leaves the kernel through the status word and the
// context usable (no trap, no endless loop); the limit here is short on purpose.
__global__ void wait_timeout_selftest_kernel(uint32_t *status)
{
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        mm_bar_init(mm_smem(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = false;
    for (uint32_t spin = 0; spin < 4096u && !ok; ++spin) ok = mm_bar_try(mm_smem(&bar), 0u);
    if (!ok && threadIdx.x == 0) atomicOr(status, 2u);
}

int launch_wait_timeout_selftest(uint32_t *status, cudaStream_t s)
{
    { wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
