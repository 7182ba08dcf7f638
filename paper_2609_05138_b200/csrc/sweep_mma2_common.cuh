// The parts the fp32 and the fp16 tensor-core sweeps (sweep_mma2.cu, sweep_mma2_f16.cu) share:
// barrier set, block set-up, and the three control roles -- the warp that streams the W_head
// stages, the warp that expands X_head, the thread that issues the MMAs -- and the final merge
// into the per-document state.  The tail (the gather itself and the way head sums leave
// tensor memory) differs between the two and stays in their own files: folding the two kernels
// into one template cost the fp32 sweep 2 % through register allocation, these inlined pieces
// do not.
#pragma once

#include "common.cuh"
#include "mma_ptx.cuh"

namespace bmu {

static const int M2_SLAB = 256;                      // neurons per slab: two accumulator tiles
static const int M2_TAIL_WARPS = 16;
static const int M2_TMEM_COLS = 512;                 // 2 buffers x 2 tiles x 128 documents

// mbarriers of a block, in shared memory: full / empty per W and X stage, full / empty per
// half of tensor memory, one to drain the MMAs at the end
template <int NS, int NX>
struct M2Bars {
    uint32_t wfull0, wempty0, xfull0, xempty0, tfull0, tempty0, drain;
    static constexpr int COUNT = 2 * NS + 2 * NX + 6;
    __device__ __forceinline__ explicit M2Bars(u64 *bars)
    {
        wfull0 = mm_smem(bars); wempty0 = mm_smem(bars + NS);
        xfull0 = mm_smem(bars + 2 * NS); xempty0 = mm_smem(bars + 2 * NS + NX);
        tfull0 = mm_smem(bars + 2 * NS + 2 * NX); tempty0 = tfull0 + 16;
        drain = tfull0 + 32;
    }
    __device__ __forceinline__ void init() const             // one thread
    {
        for (int i = 0; i < NS; ++i) { mm_bar_init(wfull0 + 8 * i, 1); mm_bar_init(wempty0 + 8 * i, 1); }
        for (int i = 0; i < NX; ++i) { mm_bar_init(xfull0 + 8 * i, 1); mm_bar_init(xempty0 + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mm_bar_init(tfull0 + 8 * i, 1); mm_bar_init(tempty0 + 8 * i, M2_TAIL_WARPS); }
        mm_bar_init(drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
};

__device__ __forceinline__ void m2_unpack(const uint4 q, uint32_t f[8])
{
    f[0] = q.x & 0xffffu; f[1] = q.x >> 16; f[2] = q.y & 0xffffu; f[3] = q.y >> 16;
    f[4] = q.z & 0xffffu; f[5] = q.z >> 16; f[6] = q.w & 0xffffu; f[7] = q.w >> 16;
}

// What every thread of the block does before the roles part ways: the block's head masks into
// shared memory (document-major, H / 8 bytes each), the per-document keys, the table that
// turns four mask bits into four fp16 zeros and ones, and (sixteen threads of the last control
// warp) the block's 16 tiles: first row of each id matrix, its length word and its offset.
template <int THREADS, bool TOP2>
__device__ __forceinline__ void m2_block_setup(const MmaArgs &a, int64_t group, int H,
                                               unsigned char *masks, u64 *keys, uint2 *lut, u64 *kq,
                                               uint4 *s_first, uint32_t *s_len, uint32_t *s_off)
{
    {
        const int words = H / 32;
        uint32_t *mw = reinterpret_cast<uint32_t *>(masks);
        for (int idx = threadIdx.x; idx < MMA_DOCS * words; idx += THREADS) {
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
        for (int idx = threadIdx.x; idx < 4 * MMA_DOCS * 2; idx += THREADS) kq[idx] = KEY_WORST;
    if (threadIdx.x >= THREADS - 16) {
        const int t = threadIdx.x - (THREADS - 16);
        const int64_t tile = group * (MMA_DOCS / 8) + t;
        const bool there = tile < a.n_tiles;
        const uint32_t off = there ? __ldg(a.tile_off + tile) : 0u;
        s_len[t] = there ? __ldg(a.tile_len + tile) : 0u;
        s_off[t] = off;
        s_first[t] = __ldcs(a.tile_ids + BMU_IDX(off, a.tile_rows_cap, a.status));
    }
}

// Producer (one thread): the W_head stages of every slab, in order, through the ring.
// STAGES_PER_KB = accumulator tiles x image parts (4 for fp32 weights: hi and lo; 2 for fp16).
template <int NS, int NX, int STAGES_PER_KB>
__device__ __forceinline__ void m2_producer(const MmaArgs &a, int n_slabs, int KB,
                                            unsigned char *wring, const M2Bars<NS, NX> &b,
                                            volatile uint32_t *abort_flag)
{
    const unsigned char *src = a.head_img;
    const int total = n_slabs * STAGES_PER_KB * KB;
    int issued = 0;
    for (int c = 0; c < total; ++c) {
        const int slot = c % NS;
        if (c >= NS && !mm_wait(b.wempty0 + 8 * slot, ((c / NS) - 1) & 1, abort_flag, a.status, 1u))
            break;
        mm_bar_expect_tx(b.wfull0 + 8 * slot, (uint32_t)MMA_STAGE_BYTES);
        mm_bulk_load(mm_smem(wring + (size_t)slot * MMA_STAGE_BYTES),
                     src + (size_t)c * MMA_STAGE_BYTES, (uint32_t)MMA_STAGE_BYTES,
                     b.wfull0 + 8 * slot);
        issued = c + 1;
    }
    if (*abort_flag)         // gave up: let the copies in flight land before leaving
        for (int c = issued > NS ? issued - NS : 0; c < issued; ++c)
            for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin)
                if (mm_bar_try(b.wfull0 + 8 * (c % NS), (c / NS) & 1)) break;
}

// Expander (one warp): X_head, one block of 64 features per stage.  A lane takes documents
// lane, lane + 32, ..: its 8 mask bytes of this block of 64 features in one load, then eight
// 16-byte stores of fp16 zeros and ones (bit e of a byte -> half e; 0x3c00 is 1.0), four bits
// at a time through the 16-entry table.
template <int NS, int NX>
__device__ __forceinline__ void m2_expander(const MmaArgs &a, int n_slabs, int KB, int H,
                                            const unsigned char *masks, unsigned char *xring,
                                            const uint2 *lut, const M2Bars<NS, NX> &b,
                                            volatile uint32_t *abort_flag, int lane)
{
    const int total = n_slabs * KB;
    for (int x = 0; x < total; ++x) {
        const int slot = x % NX, kb = x % KB;
        if (x >= NX && !mm_wait(b.xempty0 + 8 * slot, ((x / NX) - 1) & 1, abort_flag, a.status, 16u))
            break;
        unsigned char *dst = xring + (size_t)slot * MMA_STAGE_BYTES;
#pragma unroll
        for (int j = 0; j < MMA_DOCS / 32; ++j) {
            const int n = lane + 32 * j;
            const uint2 mb = *reinterpret_cast<const uint2 *>(masks + (size_t)n * (H / 8) + kb * 8);
            unsigned char *row = dst + (size_t)(n >> 3) * 1024 + (n & 7) * 16;
#pragma unroll
            for (int kc = 0; kc < 8; ++kc) {
                const uint32_t bits = (kc < 4 ? mb.x : mb.y) >> ((kc & 3) * 8);
                const uint2 lo4 = lut[bits & 15u], hi4 = lut[(bits >> 4) & 15u];
                *reinterpret_cast<uint4 *>(row + kc * 128) = make_uint4(lo4.x, lo4.y, hi4.x, hi4.y);
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mm_bar_arrive(b.xfull0 + 8 * slot);
    }
    __syncwarp();
}

// MMA issuer (one thread): for every slab and block of 64 features, the MMAs of its W stages
// (tile-major, PARTS image parts per tile) against the X stage, into the half of tensor memory
// that the tail of two slabs ago has released.
template <int NS, int NX, int PARTS>
__device__ __forceinline__ void m2_issuer(const MmaArgs &a, int n_slabs, int KB, uint32_t tmem,
                                          unsigned char *wring, unsigned char *xring,
                                          const M2Bars<NS, NX> &b, volatile uint32_t *abort_flag)
{
    const uint32_t idesc = (1u << 4) | ((uint32_t)(MMA_DOCS >> 3) << 17) | (8u << 24);
    const uint32_t wring_u32 = mm_smem(wring), xring_u32 = mm_smem(xring);
    bool ok = true;
    int wc = 0, xc = 0;
    for (int sl = 0; sl < n_slabs && ok; ++sl) {
        const int buf = sl & 1;
        if (sl >= 2) ok = mm_wait(b.tempty0 + 8 * buf, ((sl >> 1) - 1) & 1, abort_flag, a.status, 2u);
        if (!ok) break;
        mm_fence_after();
        for (int kb = 0; kb < KB && ok; ++kb, ++xc) {
            const int xslot = xc % NX;
            if (!mm_wait(b.xfull0 + 8 * xslot, (xc / NX) & 1, abort_flag, a.status, 32u)) { ok = false; break; }
            for (int cp = 0; cp < 2 * PARTS; ++cp, ++wc) {       // cp = tile * PARTS + part
                const int slot = wc % NS;
                if (!mm_wait(b.wfull0 + 8 * slot, (wc / NS) & 1, abort_flag, a.status, 4u)) { ok = false; break; }
                mm_fence_after();
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const u64 ad = mm_desc(wring_u32 + slot * (uint32_t)MMA_STAGE_BYTES + u * 256, 128, 1024);
                    const u64 bd = mm_desc(xring_u32 + xslot * (uint32_t)MMA_STAGE_BYTES + u * 256, 128, 1024);
                    BMU_EXPECT(slot < NS && xslot < NX &&
                               buf * 256 + (cp / PARTS) * MMA_DOCS + MMA_DOCS <= M2_TMEM_COLS, a.status);
                    mm_mma(tmem + buf * 256 + (cp / PARTS) * MMA_DOCS, ad, bd, idesc,
                           (kb | (cp % PARTS) | u) != 0);
                }
                mm_commit(b.wempty0 + 8 * slot);
            }
            if (ok) mm_commit(b.xempty0 + 8 * xslot);
        }
        if (ok) mm_commit(b.tfull0 + 8 * buf);
    }
    mm_commit(b.drain);
    for (uint32_t spin = 0; spin < MMA_WAIT_LIMIT; ++spin)
        if (mm_bar_try(b.drain, 0)) break;
}

// After the roles have met again: the block's per-document results into the state (one owner
// per document per launch).  TOP2: the four neuron quarters of a document are merged first.
template <bool TOP2>
__device__ __forceinline__ void m2_commit(const MmaArgs &a, int64_t group, const u64 *keys, const u64 *kq)
{
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
}

}  // namespace bmu
