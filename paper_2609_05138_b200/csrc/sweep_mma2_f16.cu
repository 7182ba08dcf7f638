// The wide tensor-core sweep (sweep_mma2.cu) for a half-precision codebook, the paper's own
// storage (Section 4.2: 2 bytes per weight; Section 4.3: loads of half pairs).
// Same structure -- 256-neuron slabs, two accumulator tiles, double-buffered tensor memory,
// K-outermost with X expanded per block of 64 features, tail tasks of 16 documents x 64
// neurons -- with these differences: the weights are fp16 already, so the head image is a plain
// re-layout with ONE part (half the MMAs, 2 bytes per weight, no scale); the tail gathers
// 16-byte pieces (eight fp16 neurons per lane, a quarter-warp per 128-byte row piece, four rows
// per load instruction, three id rows = twelve loads in flight per lane) and adds each weight to
// its fp32 sum with the mixed-precision add of sm_100; the head sums leave tensor memory through
// a per-warp transposing buffer in shared memory; and the control warpgroup hands registers to
// the tail warpgroups.  Kept as its own kernel so that the fp32 sweep's code generation is not
// disturbed; the control roles are the shared ones of sweep_mma2_common.cuh.
#include "sweep_mma2_common.cuh"

#include <cuda_fp16.h>
#include <math_constants.h>

namespace bmu {

#ifndef BMU_M2F_WSTAGES
#define BMU_M2F_WSTAGES 4
#endif
#ifndef BMU_M2F_XSTAGES
#define BMU_M2F_XSTAGES 3
#endif
static const int M2_NS = BMU_M2F_WSTAGES;             // W ring stages
static const int M2_NX = BMU_M2F_XSTAGES;             // X ring stages
static const int M2_THREADS = (M2_TAIL_WARPS + 4) * 32;      // 4 tail warpgroups + 1 control warpgroup
#ifndef BMU_M2F_ROWS
#define BMU_M2F_ROWS 3                               // id rows per turn: 4 x ROWS loads in flight per lane
#endif
static const int M2_XCH_BYTES = 16 * 64 * 4;         // a tail warp's 16 documents x 64 head sums

static inline size_t m2_smem_bytes(int head, bool top2)
{
    return (size_t)MMA_DOCS * (head / 8) + (M2_NS + M2_NX) * MMA_STAGE_BYTES +
           (2 * M2_NS + 2 * M2_NX + 6) * 8 + MMA_DOCS * 8 + 16 + 16 * 16 + 2 * 16 * 4 +
           16 * 8 + (top2 ? 4 * MMA_DOCS * 16 : 0) + (size_t)M2_TAIL_WARPS * M2_XCH_BYTES;
}

// Half-precision codebook: the weights are fp16 already, so the image is a re-layout (one part,
// no scale): stage order inside a slab: block of 64 features, tile c.
__global__ void __launch_bounds__(M2_SLAB)
head_split2_f16_kernel(const __half *__restrict__ W16, int64_t M, int head,
                       const uint16_t *__restrict__ feat, unsigned char *__restrict__ img)
{
    const int sl = blockIdx.x, kcg = blockIdx.y, jin = threadIdx.x;
    const int SPS = 2 * (head / 64);
    const __half *col = W16 + (int64_t)sl * M2_SLAB + jin;
    __align__(16) __half h[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int64_t row = feat ? (int64_t)feat[kcg * 8 + e] : (int64_t)(kcg * 8 + e);
        h[e] = col[row * M];
    }
    // accumulator row 32q + 8s + i of tile c holds neuron 64q + 32 (s / 2) + 4i + 2 (s % 2) + c of
    // the slab, so that the 16 lanes of a half-warp hold 32 consecutive neurons
    const int c = jin & 1, r = ((jin >> 6) << 5) | (((jin >> 5) & 1) << 4) | (((jin >> 1) & 1) << 3) | ((jin >> 2) & 7);
    const int kb = kcg >> 3, kc = kcg & 7;
    const size_t off = (size_t)(r >> 3) * 1024 + (size_t)kc * 128 + (size_t)(r & 7) * 16;
    const size_t st = (size_t)sl * SPS + (size_t)(kb * 2 + c);
    *reinterpret_cast<uint4 *>(img + st * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(h);
}

int launch_head_split2_f16(const void *W16, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                           unsigned char *head_img, cudaStream_t s)
{
    if (m_full <= 0) return BMU_OK;
    const dim3 grid((unsigned)(m_full / M2_SLAB), head / 8);
    { head_split2_f16_kernel<<<grid, M2_SLAB, 0, s>>>(static_cast<const __half *>(W16), M, head, feat,
                                                    head_img); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

// fp32 sum + fp16 term in one instruction (mixed-precision add of sm_100: the widening is exact,
// so the result is the one a convert followed by an fp32 add gives)
__device__ __forceinline__ float m2_addh(float c, uint16_t h)
{
    float d;
    asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(c));
    return d;
}

// eight fp16 weights (16 bytes of a half-precision row) added to eight fp32 sums
__device__ __forceinline__ void m2_add_h8(float (&s)[8], const uint4 w)
{
    const uint32_t p[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint16_t h0, h1;
        asm("mov.b32 {%0, %1}, %2;" : "=h"(h0), "=h"(h1) : "r"(p[i]));
        s[2 * i] = m2_addh(s[2 * i], h0);
        s[2 * i + 1] = m2_addh(s[2 * i + 1], h1);
    }
}

// the four ids of a lane's documents: the low or the high half of a row of eight
__device__ __forceinline__ void m2_ids4(const uint4 q, bool upper, uint32_t f[4])
{
    const uint32_t a = upper ? q.z : q.x, b = upper ? q.w : q.y;
    f[0] = a & 0xffffu; f[1] = a >> 16; f[2] = b & 0xffffu; f[3] = b >> 16;
}

// TOP2: also the second-best unit (Table 5: the paper's kernel tracks it for topographic error).
template <bool TOP2>
__global__ void __launch_bounds__(M2_THREADS, 1)
sweep_mma2_f16_kernel(const MmaArgs a)
{
    constexpr int NS = M2_NS, NX = M2_NX, NTW = M2_TAIL_WARPS;
    constexpr int PARTS = 1;                                     // the weights are fp16: no lo part
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
    float *xch0 = reinterpret_cast<float *>(kq + (TOP2 ? 4 * MMA_DOCS * 2 : 0));   // per tail warp
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

    // The control warpgroup (producer, expander, MMA issuer and one idle warp) hands registers
    // to the four tail warpgroups, whose loads in flight are bounded by their registers.  The
    // block is launched with 96 per thread (640 x 96 = 61440); 128 x 56 + 512 x 104 = 60416 fits,
    // so the increase below never waits for registers that nobody releases.
    if (warp >= NTW) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (warp == NTW) {
        // ---------------- producer: W stages of every slab (2 tiles x one part per 64 features)
        if (lane == 0) m2_producer<NS, NX, 2 * PARTS>(a, n_slabs, KB, wring, bar, abort_flag);
        __syncwarp();
    } else if (warp == NTW + 1) {
        // ---------------- expander: X_head, one block of 64 features per stage
        m2_expander<NS, NX>(a, n_slabs, KB, H, masks, xring, lut, bar, abort_flag, lane);
    } else if (warp == NTW + 2) {
        // ---------------- one thread issues every MMA
        if (lane == 0) m2_issuer<NS, NX, PARTS>(a, n_slabs, KB, tmem, wring, xring, bar, abort_flag);
        __syncwarp();
    }   // (the fourth warp only completes the control warpgroup)
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 104;");
        // ---------------- tail: 16 documents x 64 neurons per task.  Lane (s, i) = (lane / 8,
        // lane % 8) gathers neurons 8i .. 8i+7 for the documents 4s .. 4s+3 of the task: one
        // 128-bit load per lane and row, four rows (one per quarter-warp) per instruction.
        const int q = warp & 3, g = warp >> 2;
        const int li = lane & 7, ls = lane >> 3;
        const uint32_t rowbytes = (uint32_t)(a.M * 2);
        const int mydoc = 4 * ls + (((lane & 1) << 1) | ((lane >> 1) & 1));
        float *xch = xch0 + (size_t)warp * (M2_XCH_BYTES / 4);
        for (int sl = 0; sl < n_slabs; ++sl) {
            const int buf = sl & 1;
            const int j0 = a.j_lo + sl * M2_SLAB + q * 64;
            for (int it = 0; it < 2; ++it) {
                const int dg = g + 4 * it;                       // the block's dg-th set of 16
                const int64_t tile_a = group * (MMA_DOCS / 8) + 2 * dg, tile_b = tile_a + 1;
                const bool live = tile_a < a.n_tiles;
                float acc[4][8];
#pragma unroll
                for (int t = 0; t < 4; ++t)
#pragma unroll
                    for (int n = 0; n < 8; ++n) acc[t][n] = 0.f;
                if (live) {
                    const bool has_b = tile_b < a.n_tiles;
                    const uint32_t tla = s_len[2 * dg], tlb = s_len[2 * dg + 1];
                    const uint32_t full = min(tla >> 16, tlb >> 16);
                    const uint32_t rows = max(tla & 0xffffu, tlb & 0xffffu);
                    const uint32_t my_rows = ((ls >> 1) ? tlb : tla) & 0xffffu;
                    const int mine = 2 * dg + (((ls >> 1) && has_b) ? 1 : 0);
                    const bool upper = ls & 1;
                    const uint4 *gp = a.tile_ids + BMU_IDX(s_off[mine], a.tile_rows_cap, a.status);
                    [[maybe_unused]] const size_t room = a.tile_rows_cap - (size_t)(gp - a.tile_ids);
                    const char *base = reinterpret_cast<const char *>(a.W) + (size_t)(j0 + li * 8) * 2;
                    uint32_t b = 0;
                    uint4 qn = s_first[mine];
                    // ROWS rows of ids per turn keep 4 x ROWS 16-byte loads in flight per lane
                    constexpr int ROWS = BMU_M2F_ROWS;
                    for (; b + ROWS - 1 < full; b += ROWS) {
                        uint32_t f[4 * ROWS];
                        m2_ids4(qn, upper, f);
#pragma unroll
                        for (int r = 1; r < ROWS; ++r) m2_ids4(__ldcs(gp + BMU_IDX(b + r, room, a.status)), upper, f + 4 * r);
                        qn = __ldcs(gp + BMU_IDX(b + ROWS, room, a.status));
                        uint4 w[4 * ROWS];
#pragma unroll
                        for (int t = 0; t < 4 * ROWS; ++t)
                            w[t] = __ldg(reinterpret_cast<const uint4 *>(base + (u64)BMU_IDX(f[t], a.D, a.status) * rowbytes));
#pragma unroll
                        for (int t = 0; t < 4 * ROWS; ++t) m2_add_h8(acc[t & 3], w[t]);
                    }
                    for (; b < rows; ++b) {                      // left-over rows, then documents that ran out
                        uint32_t f[4];
                        m2_ids4(qn, upper, f);
                        qn = __ldcs(gp + BMU_IDX(b + 1, room, a.status));
                        const bool in = b < my_rows;
                        uint4 w[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            w[t] = (in && f[t] != 0xffffu)
                                       ? __ldg(reinterpret_cast<const uint4 *>(base + (u64)BMU_IDX(f[t], a.D, a.status) * rowbytes))
                                       : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                        for (int t = 0; t < 4; ++t) m2_add_h8(acc[t], w[t]);
                    }
                }
                // head sums of these documents: the MMAs of this slab ran during the gather.
                // Tensor-memory lane 32q + lane holds neurons 32 (s / 2) + 4i + 2 (s % 2) + {0, 1}
                // for all 16 documents; the warp's buffer turns that into eight neurons of
                // four documents per lane.
                if (it == 0) mm_wait(tfull0 + 8 * buf, (sl >> 1) & 1, abort_flag, a.status, 8u);
                mm_fence_after();
                uint32_t h0[16], h1[16];
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + dg * 16);
                mm_tmem_ld16(taddr, h0);
                mm_tmem_ld16(taddr + MMA_DOCS, h1);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (it == 1) {                                   // this half of tensor memory is free
                    mm_fence_before();
                    __syncwarp();
                    if (lane == 0) mm_bar_arrive(tempty0 + 8 * buf);
                }
                if (!live) continue;
                __syncwarp();                                    // the buffer's last readers are done
#pragma unroll
                for (int d = 0; d < 16; ++d)                     // 128 contiguous bytes per half-warp
                    *reinterpret_cast<uint2 *>(xch + d * 64 + 32 * (ls >> 1) + 4 * li + 2 * (ls & 1)) =
                        make_uint2(h0[d], h1[d]);
                __syncwarp();
                const int sw = li >> 2;                          // lanes 4..7 of a quarter read the
#pragma unroll                                                   // upper half first: no bank conflict
                for (int t = 0; t < 4; ++t) {
                    const float4 *r = reinterpret_cast<const float4 *>(xch + (4 * ls + t) * 64 + 8 * li);
                    const float4 u = r[sw], v = r[sw ^ 1];
                    const float4 lo = sw ? v : u, hi = sw ? u : v;
                    acc[t][0] += lo.x; acc[t][1] += lo.y; acc[t][2] += lo.z; acc[t][3] += lo.w;
                    acc[t][4] += hi.x; acc[t][5] += hi.y; acc[t][6] += hi.z; acc[t][7] += hi.w;
                }
                const int col = j0 + li * 8;
                const float4 na = __ldg(reinterpret_cast<const float4 *>(a.norms + col));
                const float4 nb = __ldg(reinterpret_cast<const float4 *>(a.norms + col + 4));
                const float n8[8] = {na.x, na.y, na.z, na.w, nb.x, nb.y, nb.z, nb.w};
                u64 k[4], k2[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    Best<TOP2> bst;
                    bst.init();
#pragma unroll
                    for (int c = 0; c < 8; ++c) bst.push(fmaf(-2.f, acc[t][c], n8[c]), col + c);
                    k[t] = make_key(bst.d1, bst.j1);
                    k2[t] = TOP2 ? make_key(bst.d2, bst.j2) : KEY_WORST;
                }
                // transposing butterfly among the 8 lanes that hold the same documents
#pragma unroll
                for (int st = 0; st < 2; ++st) {
                    const int m = 1 << st, cnt = 2 >> st;
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
                const u64 got = __shfl_xor_sync(0xffffffffu, k[0], 4);
                if (TOP2) {
                    const u64 got2 = __shfl_xor_sync(0xffffffffu, k2[0], 4);
                    Best<true>::merge(k[0], k2[0], got, got2);
                    if ((lane & 4) == 0) {
                        u64 *slot = kq + ((size_t)q * MMA_DOCS + dg * 16 + mydoc) * 2;
                        Best<true>::merge(k[0], k2[0], slot[0], slot[1]);
                        slot[0] = k[0];
                        slot[1] = k2[0];
                    }
                } else {
                    k[0] = got < k[0] ? got : k[0];
                    if ((lane & 4) == 0)
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

int launch_sweep_mma2_f16(const MmaArgs &a, const bmu_opts &o, cudaStream_t s)
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
        // the register hand-over inside the kernel must fit what a block is launched with, or
        // the increase would wait for ever: refuse to launch a build where it does not
        cudaFuncAttributes fa, fb;
        BMU_CUDA(cudaFuncGetAttributes(&fa, sweep_mma2_f16_kernel<false>));
        BMU_CUDA(cudaFuncGetAttributes(&fb, sweep_mma2_f16_kernel<true>));
        const int regs = fa.numRegs < fb.numRegs ? fa.numRegs : fb.numRegs;
        if (M2_THREADS * regs < 128 * 56 + 512 * 104) {
            set_error("half-precision tensor-core sweep: built with %d registers per thread, the "
                      "register hand-over needs %d", regs, (128 * 56 + 512 * 104 + M2_THREADS - 1) / M2_THREADS);
            return BMU_ERR_UNSUPPORTED;
        }
        BMU_CUDA(cudaFuncSetAttribute(sweep_mma2_f16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)m2_smem_bytes(HEAD_ROWS_MAX, false)));
        BMU_CUDA(cudaFuncSetAttribute(sweep_mma2_f16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)m2_smem_bytes(HEAD_ROWS_MAX, true)));
        configured[dev] = true;
    }
    const unsigned blocks = (unsigned)((a.N + MMA_DOCS - 1) / MMA_DOCS);
    const size_t smem = m2_smem_bytes(a.head, a.state2 != nullptr);
    if (a.state2) { sweep_mma2_f16_kernel<true><<<blocks, M2_THREADS, smem, s>>>(a); BMU_LAUNCHED(); }
    else { sweep_mma2_f16_kernel<false><<<blocks, M2_THREADS, smem, s>>>(a); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
