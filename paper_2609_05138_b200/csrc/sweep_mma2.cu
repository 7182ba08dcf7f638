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
#include "common.cuh"
#include "mma_ptx.cuh"

#include <cuda_fp16.h>
#include <math_constants.h>

namespace bmu {

static const int M2_SLAB = 256;
#ifndef BMU_M2_WSTAGES
#define BMU_M2_WSTAGES 4
#endif
#ifndef BMU_M2_XSTAGES
#define BMU_M2_XSTAGES 3
#endif
static const int M2_NS = BMU_M2_WSTAGES;             // W ring stages
static const int M2_NX = BMU_M2_XSTAGES;             // X ring stages
static const int M2_TAIL_WARPS = 16;
static const int M2_THREADS = (M2_TAIL_WARPS + 3) * 32;
static const int M2_TMEM_COLS = 512;                 // 2 buffers x 2 tiles x 128 documents

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

__device__ __forceinline__ void m2_unpack(const uint4 q, uint32_t f[8])
{
    f[0] = q.x & 0xffffu; f[1] = q.x >> 16; f[2] = q.y & 0xffffu; f[3] = q.y >> 16;
    f[4] = q.z & 0xffffu; f[5] = q.z >> 16; f[6] = q.w & 0xffffu; f[7] = q.w >> 16;
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
    const uint32_t wfull0 = mm_smem(bars), wempty0 = mm_smem(bars + NS);
    const uint32_t xfull0 = mm_smem(bars + 2 * NS), xempty0 = mm_smem(bars + 2 * NS + NX);
    const uint32_t tfull0 = mm_smem(bars + 2 * NS + 2 * NX), tempty0 = tfull0 + 16;
    const uint32_t drain = tfull0 + 32;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t group = blockIdx.x;
    const int n_slabs = (a.j_hi - a.j_lo) / M2_SLAB;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) { mm_bar_init(wfull0 + 8 * i, 1); mm_bar_init(wempty0 + 8 * i, 1); }
        for (int i = 0; i < NX; ++i) { mm_bar_init(xfull0 + 8 * i, 1); mm_bar_init(xempty0 + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mm_bar_init(tfull0 + 8 * i, 1); mm_bar_init(tempty0 + 8 * i, NTW); }
        mm_bar_init(drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
    {   // the block's head masks into shared memory (document-major, H / 8 bytes each)
        const int words = H / 32;
        uint32_t *mw = reinterpret_cast<uint32_t *>(masks);
        for (int idx = threadIdx.x; idx < MMA_DOCS * words; idx += M2_THREADS) {
            const int n = idx / words;
            const int64_t tile = group * (MMA_DOCS / 8) + (n >> 3);
            mw[idx] = tile < a.n_tiles ? __ldcs(a.tile_head + (size_t)group * MMA_DOCS * words + idx) : 0u;
        }
    }
    if (threadIdx.x < MMA_DOCS) keys[threadIdx.x] = KEY_WORST;
    if (threadIdx.x < 16) {
        const uint32_t b = threadIdx.x;
        lut[b] = make_uint2((b & 1u) * 0x3c00u + (b & 2u) * 0x1e000000u,
                            ((b >> 2) & 1u) * 0x3c00u + ((b >> 2) & 2u) * 0x1e000000u);
    }
    if (TOP2)
        for (int idx = threadIdx.x; idx < 4 * MMA_DOCS * 2; idx += M2_THREADS) kq[idx] = KEY_WORST;
    if (threadIdx.x >= M2_THREADS - 16) {            // 16 threads of the last control warp
        const int t = threadIdx.x - (M2_THREADS - 16);
        const int64_t tile = group * (MMA_DOCS / 8) + t;
        const bool there = tile < a.n_tiles;
        const uint32_t off = there ? __ldg(a.tile_off + tile) : 0u;
        s_len[t] = there ? __ldg(a.tile_len + tile) : 0u;
        s_off[t] = off;
        s_first[t] = __ldcs(a.tile_ids + BMU_IDX(off, a.tile_rows_cap, a.status));
    }
    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (warp == NTW) {
        // ---------------- producer: W stages of every slab, in order
        if (lane == 0) {
            const unsigned char *src = a.head_img;
            const int total = n_slabs * 4 * KB;
            int issued = 0;
            for (int c = 0; c < total; ++c) {
                const int slot = c % NS;
                if (c >= NS && !mm_wait(wempty0 + 8 * slot, ((c / NS) - 1) & 1, abort_flag, a.status, 1u))
                    break;
                mm_bar_expect_tx(wfull0 + 8 * slot, (uint32_t)MMA_STAGE_BYTES);
                mm_bulk_load(mm_smem(wring + (size_t)slot * MMA_STAGE_BYTES),
                             src + (size_t)c * MMA_STAGE_BYTES, (uint32_t)MMA_STAGE_BYTES,
                             wfull0 + 8 * slot);
                issued = c + 1;
            }
            if (*abort_flag)         // gave up: let the copies in flight land before leaving
                for (int c = issued > NS ? issued - NS : 0; c < issued; ++c)
                    for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin)
                        if (mm_bar_try(wfull0 + 8 * (c % NS), (c / NS) & 1)) break;
        }
        __syncwarp();
    } else if (warp == NTW + 1) {
        // ---------------- expander: X_head, one block of 64 features per stage
        const int total = n_slabs * KB;
        for (int x = 0; x < total; ++x) {
            const int slot = x % NX, kb = x % KB;
            if (x >= NX && !mm_wait(xempty0 + 8 * slot, ((x / NX) - 1) & 1, abort_flag, a.status, 16u))
                break;
            unsigned char *dst = xring + (size_t)slot * MMA_STAGE_BYTES;
            // a lane takes documents lane, lane + 32, ..: its 8 mask bytes of this block of 64
            // features in one load, then eight 16-byte stores of fp16 zeros and ones (bit e of
            // a byte -> half e; 0x3c00 is 1.0), four bits at a time through a 16-entry table
#pragma unroll
            for (int j = 0; j < MMA_DOCS / 32; ++j) {
                const int n = lane + 32 * j;
                const uint2 mb = *reinterpret_cast<const uint2 *>(masks + (size_t)n * (H / 8) + kb * 8);
                unsigned char *row = dst + (size_t)(n >> 3) * 1024 + (n & 7) * 16;
#pragma unroll
                for (int kc = 0; kc < 8; ++kc) {
                    const uint32_t b = (kc < 4 ? mb.x : mb.y) >> ((kc & 3) * 8);
                    const uint2 lo4 = lut[b & 15u], hi4 = lut[(b >> 4) & 15u];
                    *reinterpret_cast<uint4 *>(row + kc * 128) = make_uint4(lo4.x, lo4.y, hi4.x, hi4.y);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mm_bar_arrive(xfull0 + 8 * slot);
        }
        __syncwarp();
    } else if (warp == NTW + 2) {
        // ---------------- one thread issues every MMA
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | ((uint32_t)(MMA_DOCS >> 3) << 17) | (8u << 24);
            const uint32_t wring_u32 = mm_smem(wring), xring_u32 = mm_smem(xring);
            bool ok = true;
            int wc = 0, xc = 0;
            for (int sl = 0; sl < n_slabs && ok; ++sl) {
                const int buf = sl & 1;
                if (sl >= 2) ok = mm_wait(tempty0 + 8 * buf, ((sl >> 1) - 1) & 1, abort_flag, a.status, 2u);
                if (!ok) break;
                mm_fence_after();
                for (int kb = 0; kb < KB && ok; ++kb, ++xc) {
                    const int xslot = xc % NX;
                    if (!mm_wait(xfull0 + 8 * xslot, (xc / NX) & 1, abort_flag, a.status, 32u)) { ok = false; break; }
                    for (int cp = 0; cp < 4; ++cp, ++wc) {       // cp = tile * 2 + part
                        const int slot = wc % NS;
                        if (!mm_wait(wfull0 + 8 * slot, (wc / NS) & 1, abort_flag, a.status, 4u)) { ok = false; break; }
                        mm_fence_after();
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const u64 ad = mm_desc(wring_u32 + slot * (uint32_t)MMA_STAGE_BYTES + u * 256, 128, 1024);
                            const u64 bd = mm_desc(xring_u32 + xslot * (uint32_t)MMA_STAGE_BYTES + u * 256, 128, 1024);
                            BMU_EXPECT(slot < NS && xslot < NX &&
                                       buf * 256 + (cp >> 1) * MMA_DOCS + MMA_DOCS <= M2_TMEM_COLS, a.status);
                            mm_mma(tmem + buf * 256 + (cp >> 1) * MMA_DOCS, ad, bd, idesc,
                                   (kb | (cp & 1) | u) != 0);
                        }
                        mm_commit(wempty0 + 8 * slot);
                    }
                    if (ok) mm_commit(xempty0 + 8 * xslot);
                }
                if (ok) mm_commit(tfull0 + 8 * buf);
            }
            mm_commit(drain);
            for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin)
                if (mm_bar_try(drain, 0)) break;
        }
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
    if (threadIdx.x < MMA_DOCS) {
        const int64_t p = group * MMA_DOCS + threadIdx.x;
        if (p < a.N) {
            const int32_t orig = __ldg(a.perm + p);
            if (TOP2) {
                u64 b1 = KEY_WORST, b2 = KEY_WORST;
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    const u64 *slot = kq + ((size_t)qq * MMA_DOCS + threadIdx.x) * 2;
                    Best<true>::merge(b1, b2, slot[0], slot[1]);
                }
                Best<true>::commit(b1, b2, a.state, a.state2, orig, a.first);
            } else {
                Best<false>::commit(keys[threadIdx.x], KEY_WORST, a.state, nullptr, orig, a.first);
            }
        }
    }
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
