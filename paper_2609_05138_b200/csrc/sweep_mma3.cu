// Tensor-core head + gathered tail, third cut: 256 documents share every head image.
//
// The head image costs 4 * H bytes per neuron and block; the more documents a block carries,
// the wider a head pays for itself, and the fewer rows are left to the gather.  Here a block
// carries 256 documents (MMA N = 256) through slabs of 128 neurons -- one accumulator tile,
// tensor-memory lane = neuron, column = document, two tiles double-buffered as in
// sweep_mma2.cu -- so the image is shared by twice as many documents and the head can be
// twice as wide for the same bytes.
//
// A tail task is 32 documents x 32 neurons.  Lane (s, i) = (lane / 8, lane % 8) gathers
// neurons 4i .. 4i+3 for the documents 8s .. 8s+7 of the task: a 128-bit load per lane and
// row, four rows of 128 contiguous bytes per instruction, eight instructions in flight.  The
// neurons of a slab are dealt so that tensor-memory lane 8c + i of a quarter holds neuron
// 4i + c: the lane that wants neurons 4i .. 4i+3 finds them in lanes i, 8+i, 16+i, 24+i -- its
// own and the three reached by flipping its s bits -- and the head sums are exchanged with
// 24 shuffles per task.
#include "common.cuh"
#include "mma_ptx.cuh"

#include <cuda_fp16.h>
#include <math_constants.h>

namespace bmu {

static const int M3_SLAB = 128;
static const int M3_DOCS = 256;
static const int M3_NS = 4;                          // W ring stages (16 KB)
static const int M3_NX = 2;                          // X ring stages (32 KB)
static const int M3_TAIL_WARPS = 16;
static const int M3_THREADS = (M3_TAIL_WARPS + 4) * 32;    // + producer, 2 expanders, MMA issuer
static const int M3_TMEM_COLS = 512;                 // 2 buffers x 256 documents
static const size_t M3_XSTAGE = 32768;               // 256 documents x 64 features x fp16
static const int M3_TILES = M3_DOCS / 8;             // 32 tiles of 8 documents per block

static inline size_t m3_smem_bytes()
{
    return M3_NX * M3_XSTAGE + M3_NS * MMA_STAGE_BYTES + (2 * M3_NS + 2 * M3_NX + 6) * 8 +
           M3_DOCS * 8 + 16 + M3_TILES * 16 + 2 * M3_TILES * 4 + 16 * 8;
}

// One thread per (slab, group of 8 features, neuron).  Stage order inside a slab: block of
// 64 features, part (hi, lo).  Neuron 32q + 4i + c of the slab sits in row 32q + 8c + i.
__global__ void __launch_bounds__(M3_SLAB)
head_split3_kernel(const float *__restrict__ W, int64_t M, const uint32_t *__restrict__ head_max,
                   int head, const uint16_t *__restrict__ feat, unsigned char *__restrict__ img)
{
    const int sl = blockIdx.x, kcg = blockIdx.y, jin = threadIdx.x;
    const int SPS = 2 * (head / 64);
    const float S = head_scale(*head_max);
    const float *col = W + (int64_t)sl * M3_SLAB + jin;
    __align__(16) __half hi[8];
    __align__(16) __half lo[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int64_t row = feat ? (int64_t)feat[kcg * 8 + e] : (int64_t)(kcg * 8 + e);
        const float w = __ldg(col + row * M) * S;
        hi[e] = __float2half_rn(w);
        lo[e] = __float2half_rn(w - __half2float(hi[e]));
    }
    const int x = jin & 31, r = (jin & ~31) | ((x & 3) << 3) | (x >> 2);
    const int kb = kcg >> 3, kc = kcg & 7;
    const size_t off = (size_t)(r >> 3) * 1024 + (size_t)kc * 128 + (size_t)(r & 7) * 16;
    const size_t st = (size_t)sl * SPS + (size_t)kb * 2;
    *reinterpret_cast<uint4 *>(img + st * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(hi);
    *reinterpret_cast<uint4 *>(img + (st + 1) * MMA_STAGE_BYTES + off) = *reinterpret_cast<uint4 *>(lo);
}

int launch_head_split3(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                       uint32_t *head_max, unsigned char *head_img, cudaStream_t s)
{
    if (m_full <= 0) return BMU_OK;
    int rc = launch_head_absmax(W, M, m_full, head, feat, head_max, s);
    if (rc) return rc;
    const dim3 grid((unsigned)(m_full / M3_SLAB), head / 8);
    head_split3_kernel<<<grid, M3_SLAB, 0, s>>>(W, M, head_max, head, feat, head_img);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

__device__ __forceinline__ void m3_unpack(const uint4 q, uint32_t f[8])
{
    f[0] = q.x & 0xffffu; f[1] = q.x >> 16; f[2] = q.y & 0xffffu; f[3] = q.y >> 16;
    f[4] = q.z & 0xffffu; f[5] = q.z >> 16; f[6] = q.w & 0xffffu; f[7] = q.w >> 16;
}
// one of four values by a 2-bit selector
__device__ __forceinline__ uint32_t m3_pick(uint32_t sel, uint32_t v0, uint32_t v1, uint32_t v2, uint32_t v3)
{
    const uint32_t a = (sel & 1u) ? v1 : v0, b = (sel & 1u) ? v3 : v2;
    return (sel & 2u) ? b : a;
}

__global__ void __launch_bounds__(M3_THREADS, 1)
sweep_mma3_kernel(const MmaArgs a)
{
    constexpr int NS = M3_NS, NX = M3_NX, NTW = M3_TAIL_WARPS;
    const int H = a.head, KB = H / 64;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *xring = smem;                                 // NX stages of X_head
    unsigned char *wring = xring + NX * M3_XSTAGE;               // NS stages of W_head
    u64 *bars = reinterpret_cast<u64 *>(wring + NS * MMA_STAGE_BYTES);
    u64 *keys = bars + 2 * NS + 2 * NX + 6;                      // (16-byte aligned)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(keys + M3_DOCS);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    uint32_t *skip_flag = tmem_slot + 2;
    uint4 *s_first = reinterpret_cast<uint4 *>(tmem_slot + 4);   // first id row of each tile
    uint32_t *s_len = reinterpret_cast<uint32_t *>(s_first + M3_TILES);
    uint32_t *s_off = s_len + M3_TILES;
    uint2 *lut = reinterpret_cast<uint2 *>(s_off + M3_TILES);    // 4 mask bits -> 4 fp16 zeros and ones
    const uint32_t wfull0 = mm_smem(bars), wempty0 = mm_smem(bars + NS);
    const uint32_t xfull0 = mm_smem(bars + 2 * NS), xempty0 = mm_smem(bars + 2 * NS + NX);
    const uint32_t tfull0 = mm_smem(bars + 2 * NS + 2 * NX), tempty0 = tfull0 + 16;
    const uint32_t drain = tfull0 + 32;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t group = blockIdx.x;
    const int n_slabs = (a.j_hi - a.j_lo) / M3_SLAB;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) { mm_bar_init(wfull0 + 8 * i, 1); mm_bar_init(wempty0 + 8 * i, 1); }
        for (int i = 0; i < NX; ++i) { mm_bar_init(xfull0 + 8 * i, 2); mm_bar_init(xempty0 + 8 * i, 1); }
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
                     ::"r"(mm_smem(tmem_slot)), "r"((uint32_t)M3_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x < M3_DOCS) keys[threadIdx.x] = KEY_WORST;
    if (threadIdx.x < 16) {
        const uint32_t b = threadIdx.x;
        lut[b] = make_uint2((b & 1u) * 0x3c00u + (b & 2u) * 0x1e000000u,
                            ((b >> 2) & 1u) * 0x3c00u + ((b >> 2) & 2u) * 0x1e000000u);
    }
    if (threadIdx.x >= M3_THREADS - M3_TILES) {      // the block's tile offsets, lengths, first rows
        const int t = threadIdx.x - (M3_THREADS - M3_TILES);
        const int64_t tile = group * M3_TILES + t;
        const bool there = tile < a.n_tiles;
        const uint32_t off = there ? __ldg(a.tile_off + tile) : 0u;
        s_len[t] = there ? __ldg(a.tile_len + tile) : 0u;
        s_off[t] = off;
        s_first[t] = __ldcs(a.tile_ids + off);
    }
    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == NTW) {
        // ---------------- producer: W stages of every slab, in order
        if (lane == 0) {
            const unsigned char *src = a.head_img;
            const int total = n_slabs * 2 * KB;
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
    } else if (warp == NTW + 1 || warp == NTW + 3) {
        // ---------------- two expanders: X_head, one block of 64 features per stage, from the
        // documents' mask words in global memory (8 bytes per document and stage); each warp
        // writes half of the stage's 256 documents, four bits at a time through a 16-entry table
        const int half = warp == NTW + 1 ? 0 : 1;
        const int total = n_slabs * KB;
        const int words = H / 32;
        constexpr int PER = M3_DOCS / 64;        // documents per lane
        const uint2 *mrow[PER];
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int n = half * (M3_DOCS / 2) + lane + 32 * j;
            const bool there = group * M3_TILES + (n >> 3) < a.n_tiles;
            mrow[j] = there ? reinterpret_cast<const uint2 *>(
                                  a.tile_head + ((size_t)group * M3_DOCS + n) * words) : nullptr;
        }
        uint2 mb[PER];
#pragma unroll
        for (int j = 0; j < PER; ++j) mb[j] = mrow[j] ? __ldg(mrow[j]) : make_uint2(0u, 0u);
        for (int x = 0; x < total; ++x) {
            const int slot = x % NX;
            uint2 cur[PER];
#pragma unroll
            for (int j = 0; j < PER; ++j) cur[j] = mb[j];
            const int kb_next = (x + 1) % KB;
            if (x + 1 < total) {                 // the next stage's words, fetched during this one
#pragma unroll
                for (int j = 0; j < PER; ++j)
                    mb[j] = mrow[j] ? __ldg(mrow[j] + kb_next) : make_uint2(0u, 0u);
            }
            if (x >= NX && !mm_wait(xempty0 + 8 * slot, ((x / NX) - 1) & 1, abort_flag, a.status, 16u))
                break;
            unsigned char *dst = xring + (size_t)slot * M3_XSTAGE;
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                const int n = half * (M3_DOCS / 2) + lane + 32 * j;
                unsigned char *row = dst + (size_t)(n >> 3) * 1024 + (n & 7) * 16;
#pragma unroll
                for (int kc = 0; kc < 8; ++kc) {
                    const uint32_t b = (kc < 4 ? cur[j].x : cur[j].y) >> ((kc & 3) * 8);
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
        // ---------------- one thread issues every MMA: M = 128 neurons, N = 256 documents
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | ((uint32_t)(M3_DOCS >> 3) << 17) | (8u << 24);
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
                    for (int part = 0; part < 2; ++part, ++wc) {
                        const int slot = wc % NS;
                        if (!mm_wait(wfull0 + 8 * slot, (wc / NS) & 1, abort_flag, a.status, 4u)) { ok = false; break; }
                        mm_fence_after();
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const u64 ad = mm_desc(wring_u32 + slot * (uint32_t)MMA_STAGE_BYTES + u * 256, 128, 1024);
                            const u64 bd = mm_desc(xring_u32 + xslot * (uint32_t)M3_XSTAGE + u * 256, 128, 1024);
                            mm_mma(tmem + buf * 256, ad, bd, idesc, (kb | part | u) != 0);
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
        // ---------------- tail: 32 documents x 32 neurons per task
        const int q = warp & 3, g = warp >> 2;
        const int li = lane & 7, ls = lane >> 3;
        const float inv_s = 1.f / head_scale(__ldg(a.head_max));
        const uint32_t rowbytes = (uint32_t)(a.M * 4);
        const int mydoc = 8 * ls + ((lane & 1) << 2 | (lane & 2) | ((lane >> 2) & 1));
        for (int sl = 0; sl < n_slabs; ++sl) {
            const int buf = sl & 1;
            const int j0 = a.j_lo + sl * M3_SLAB + q * 32;
            for (int it = 0; it < 2; ++it) {
                const int dg = g + 4 * it;                       // the block's dg-th set of 32
                const int mine = 4 * dg + ls;                    // this lane's tile of 8 documents
                const bool live = group * M3_TILES + 4 * dg < a.n_tiles;
                u64 acc[8][2];
#pragma unroll
                for (int t = 0; t < 8; ++t) acc[t][0] = acc[t][1] = 0ull;
                if (live) {
                    const uint32_t l0 = s_len[4 * dg], l1 = s_len[4 * dg + 1];
                    const uint32_t l2 = s_len[4 * dg + 2], l3 = s_len[4 * dg + 3];
                    const uint32_t full = min(min(l0 >> 16, l1 >> 16), min(l2 >> 16, l3 >> 16));
                    const uint32_t rows = max(max(l0 & 0xffffu, l1 & 0xffffu), max(l2 & 0xffffu, l3 & 0xffffu));
                    const uint32_t my_rows = s_len[mine] & 0xffffu;
                    const uint4 *gp = a.tile_ids + s_off[mine];
                    const char *base = reinterpret_cast<const char *>(a.W + j0 + li * 4);
                    uint32_t b = 0;
                    uint4 qn = s_first[mine];
                    for (; b < full; ++b) {
                        uint32_t f[8];
                        m3_unpack(qn, f);
                        qn = __ldcs(gp + b + 1);
                        ulonglong2 w[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t)
                            w[t] = __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)f[t] * rowbytes));
#pragma unroll
                        for (int t = 0; t < 8; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
                    }
                    for (; b < rows; ++b) {                      // some documents have run out
                        uint32_t f[8];
                        m3_unpack(qn, f);
                        qn = __ldcs(gp + b + 1);
                        const bool in = b < my_rows;
                        ulonglong2 w[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t)
                            w[t] = (in && f[t] != 0xffffu)
                                       ? __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)f[t] * rowbytes))
                                       : make_ulonglong2(0ull, 0ull);
#pragma unroll
                        for (int t = 0; t < 8; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
                    }
                }
                // head sums: tensor-memory lane 32q + lane = 8 ls + li holds neuron 4 li + ls of
                // this quarter for the task's 32 documents; lane (ls, li) wants neurons 4 li + c,
                // c = 0 .. 3, for documents 8 ls .. 8 ls + 7: c = ls is its own, c = ls ^ m comes
                // from lane ^ (8 m), which sends its values of the receiver's documents.
                if (it == 0) mm_wait(tfull0 + 8 * buf, (sl >> 1) & 1, abort_flag, a.status, 8u);
                mm_fence_after();
                uint32_t hv[32];
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + dg * 32);
                mm_tmem_ld16(taddr, hv);
                mm_tmem_ld16(taddr + 16, hv + 16);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (it == 1) {                                   // this half of tensor memory is free
                    mm_fence_before();
                    __syncwarp();
                    if (lane == 0) mm_bar_arrive(tempty0 + 8 * buf);
                }
                if (!live) continue;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    // v[m]: the sum of neuron 4 li + (ls ^ m) for document 8 ls + t
                    uint32_t v[4];
                    v[0] = m3_pick((uint32_t)ls, hv[t], hv[8 + t], hv[16 + t], hv[24 + t]);
#pragma unroll
                    for (int m = 1; m < 4; ++m) {
                        // the receiver is lane ^ 8m, its documents are 8 (ls ^ m) + t
                        const uint32_t send = m3_pick((uint32_t)(ls ^ m), hv[t], hv[8 + t], hv[16 + t], hv[24 + t]);
                        v[m] = __shfl_xor_sync(0xffffffffu, send, 8 * m);
                    }
                    // neuron component c holds v[c ^ ls]
                    const float s0 = __uint_as_float(m3_pick((uint32_t)(0 ^ ls), v[0], v[1], v[2], v[3])) * inv_s;
                    const float s1 = __uint_as_float(m3_pick((uint32_t)(1 ^ ls), v[0], v[1], v[2], v[3])) * inv_s;
                    const float s2 = __uint_as_float(m3_pick((uint32_t)(2 ^ ls), v[0], v[1], v[2], v[3])) * inv_s;
                    const float s3 = __uint_as_float(m3_pick((uint32_t)(3 ^ ls), v[0], v[1], v[2], v[3])) * inv_s;
                    add2(acc[t][0], ((u64)__float_as_uint(s1) << 32) | __float_as_uint(s0));
                    add2(acc[t][1], ((u64)__float_as_uint(s3) << 32) | __float_as_uint(s2));
                }
                const int col = j0 + li * 4;
                const float4 n = __ldg(reinterpret_cast<const float4 *>(a.norms + col));
                const float n4[4] = {n.x, n.y, n.z, n.w};
                u64 k[8];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const float s4[4] = {lo_f(acc[t][0]), hi_f(acc[t][0]), lo_f(acc[t][1]), hi_f(acc[t][1])};
                    Best<false> bst;
                    bst.init();
#pragma unroll
                    for (int c = 0; c < 4; ++c) bst.push(fmaf(-2.f, s4[c], n4[c]), col + c);
                    k[t] = make_key(bst.d1, bst.j1);
                }
                // transposing butterfly among the 8 lanes that hold the same documents
#pragma unroll
                for (int st = 0; st < 3; ++st) {
                    const int m = 1 << st, cnt = 4 >> st;
#pragma unroll
                    for (int i = 0; i < cnt; ++i) {
                        const u64 send = (lane & m) ? k[i] : k[i + cnt];
                        const u64 keep = (lane & m) ? k[i + cnt] : k[i];
                        const u64 got = __shfl_xor_sync(0xffffffffu, send, m);
                        k[i] = got < keep ? got : keep;
                    }
                }
                atomicMin(reinterpret_cast<unsigned long long *>(keys + dg * 32 + mydoc), k[0]);
            }
        }
        __syncwarp();
    }

    mm_fence_before();
    __syncthreads();
    mm_fence_after();
    if (threadIdx.x < M3_DOCS) {
        const int64_t p = group * M3_DOCS + threadIdx.x;
        if (p < a.N) {
            const int32_t orig = __ldg(a.perm + p);
            Best<false>::commit(keys[threadIdx.x], KEY_WORST, a.state, nullptr, orig, a.first);
        }
    }
    if (warp == NTW)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)M3_TMEM_COLS) : "memory");
}

int launch_sweep_mma3(const MmaArgs &a, const bmu_opts &o, cudaStream_t s)
{
    (void)o;
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    if ((a.j_hi - a.j_lo) % (2 * M3_SLAB) != 0 || a.j_lo % M3_SLAB != 0) {
        set_error("256-document sweep handles whole pairs of %d-neuron slabs only", M3_SLAB);
        return BMU_ERR_INVALID_ARG;
    }
    if (a.head < 64 || a.head > HEAD_ROWS_MAX || a.head % 64 != 0) {
        set_error("256-document sweep: head_rows must be a multiple of 64 up to %d", HEAD_ROWS_MAX);
        return BMU_ERR_INVALID_ARG;
    }
    static bool configured[64];
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        BMU_CUDA(cudaFuncSetAttribute(sweep_mma3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)m3_smem_bytes()));
        configured[dev] = true;
    }
    const unsigned blocks = (unsigned)((a.N + M3_DOCS - 1) / M3_DOCS);
    sweep_mma3_kernel<<<blocks, M3_THREADS, m3_smem_bytes(), s>>>(a);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
