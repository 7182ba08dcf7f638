// Tiled gather-accumulate sweep (the paper's tile lever, Section 4.1, and the
// locality levers of Section 4.2, re-cut for B200).
//
// A warp carries a tile of 8 documents through a slab of 128 neurons: every lane
// owns 4 neurons and keeps 8 x 4 partial sums in registers.  The tiling pass has
// written the tile's ids as a matrix whose row b holds the b-th feature id of
// each of the 8 documents, so one broadcast 128-bit load yields the next feature
// of all eight, the eight row loads that follow are independent (eight in
// flight per warp) and their sums go to statically named accumulators: no
// shuffle, no branch on membership, no dynamic register index.
//
// Why tiles at all when each row load still feeds one document: every document
// lists its ids in ascending order and the documents are length-ordered, so all
// warps of a block -- which start every slab together -- walk the feature axis
// in step, from the frequent ids to the rare ones.  The 8 * NW documents of the
// block therefore ask for the same rows at about the same time, and L1 serves
// the repeats: this is the reuse the paper gets from the co-resident blocks of
// its execution ordering and from chunking, moved one level up, from L2 to L1.
//
// After the last row each lane has 4 distances per document; a transposing
// butterfly (9 exchanges instead of 8 x 5) leaves the reduced (distance, index)
// key of document bitrev3(l & 7) on lane l, where it is merged into that
// document's running minimum for the chunk.
#include "common.cuh"

#include <math_constants.h>

namespace bmu {

static const int TILE_DOCS = 8;

// acc += w where (mask & bit) != 0, as predicated adds (no branch)
__device__ __forceinline__ void add2_if(u64 &a0, u64 &a1, u64 w0, u64 w1, uint32_t mask,
                                        uint32_t bit)
{
    asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %4, %5;\n\tsetp.ne.u32 p, t, 0;\n\t"
        "@p add.rn.f32x2 %0, %0, %2;\n\t@p add.rn.f32x2 %1, %1, %3;\n\t}"
        : "+l"(a0), "+l"(a1) : "l"(w0), "l"(w1), "r"(mask), "r"(bit));
}

template <bool TOP2>
struct Keys {                     // best (and second-best) key of one document
    u64 k1, k2;
    __device__ __forceinline__ void absorb(const Keys &o)
    {
        if (TOP2) Best<true>::merge(k1, k2, o.k1, o.k2);
        else k1 = o.k1 < k1 ? o.k1 : k1;
    }
    __device__ __forceinline__ Keys xchg(int mask) const
    {
        Keys r;
        r.k1 = __shfl_xor_sync(0xffffffffu, k1, mask);
        r.k2 = TOP2 ? __shfl_xor_sync(0xffffffffu, k2, mask) : KEY_WORST;
        return r;
    }
};

// which document's result lane l holds after the butterfly
__device__ __forceinline__ int doc_of_lane(int lane)
{
    return ((lane & 1) << 2) | (lane & 2) | ((lane & 4) >> 2);
}

// 640 resident threads per SM: 96 registers per thread (the 32 sums, eight 128-bit loads in
// flight, no spill) and 20 warps -- the best trade between loads in flight per warp and warps
#ifndef BMU_TILE_THREADS
#define BMU_TILE_THREADS 640
#endif
template <int NW, bool TOP2>
__global__ void __launch_bounds__(NW * 32, BMU_TILE_THREADS / (NW * 32) > 0 ? BMU_TILE_THREADS / (NW * 32) : 1)
sweep_tiles_kernel(const TileArgs a)
{
    constexpr int T = TILE_DOCS;
    if (__ldg(a.status) & PLAN_STATUS_OVERFLOW) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t tile = (int64_t)blockIdx.x * NW + warp;
    const bool active = tile < a.n_tiles;            // idle warps still meet the barriers

    uint32_t rows = 0, full = 0;
    const uint4 *gp = a.tile_ids;
    if (active) {
        const uint32_t tl = __ldg(a.tile_len + tile);
        rows = tl & 0xffffu;
        full = tl >> 16;
        gp = a.tile_ids + BMU_IDX(__ldg(a.tile_off + tile), a.tile_rows_cap, a.status);
    }
    [[maybe_unused]] const size_t room = a.tile_rows_cap - (size_t)(gp - a.tile_ids);
    const int mydoc = doc_of_lane(lane);
    const int64_t myp = tile * T + mydoc;
    const int32_t orig = (active && myp < a.N) ? __ldg(a.perm + myp) : -1;
    Keys<TOP2> run;
    run.k1 = run.k2 = KEY_WORST;
    const uint32_t rowbytes = (uint32_t)(a.M * 4);
    // which of the frequent ids (< head_rows) each document has (kept in shared memory: the
    // registers are needed for loads in flight); `any`: their union
    __shared__ uint32_t s_hm[NW][T];
    uint32_t any = 0;
    if (lane < T) s_hm[warp][lane] = (active && a.head_rows) ? __ldg(a.tile_head + tile * T + lane) : 0u;
    __syncwarp();
#pragma unroll
    for (int t = 0; t < T; ++t) any |= s_hm[warp][t];

    for (int j0 = a.j_lo; j0 < a.j_hi; j0 += 128) {
        __syncthreads();                              // the block's warps start each slab together
        if (!active) continue;
        const char *base = reinterpret_cast<const char *>(a.W + j0 + lane * 4);
        u64 acc[T][2];
#pragma unroll
        for (int t = 0; t < T; ++t) acc[t][0] = acc[t][1] = 0ull;

        // dense head: a frequent row is loaded once for the tile and added to every document
        // that has it -- the reuse of a loaded weight across the tile (Section 4.1)
        if (any) {
#pragma unroll
            for (int f0 = 0; f0 < TILE_HEAD_ROWS; f0 += 8) {
                if (((any >> f0) & 0xffu) == 0) continue;     // nobody has any of these eight
                ulonglong2 w[8];                               // eight rows in flight, as below
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    w[u] = __ldg(reinterpret_cast<const ulonglong2 *>(
                        base + (u64)(f0 + u) * rowbytes));
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    const uint32_t m = s_hm[warp][t];
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        add2_if(acc[t][0], acc[t][1], w[u].x, w[u].y, m, 1u << (f0 + u));
                }
            }
        }
        uint32_t b = 0;
        uint4 qn = __ldg(gp);                         // ids one row ahead of the row loads
        for (; b < full; ++b) {                       // rows where all 8 documents still have an id
            const uint4 q = qn;
            qn = __ldg(gp + BMU_IDX(b + 1, room, a.status));   // (slack rows follow every matrix)
            const uint32_t f[T] = {q.x & 0xffffu, q.x >> 16, q.y & 0xffffu, q.y >> 16,
                                   q.z & 0xffffu, q.z >> 16, q.w & 0xffffu, q.w >> 16};
            ulonglong2 w[T];
#pragma unroll
            for (int t = 0; t < T; ++t)
                w[t] = __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)BMU_IDX(f[t], a.D, a.status) * rowbytes));
#pragma unroll
            for (int t = 0; t < T; ++t) { add2(acc[t][0], w[t].x); add2(acc[t][1], w[t].y); }
        }
        for (; b < rows; ++b) {                       // the ragged end: some documents have run out
            const uint4 q = qn;
            qn = __ldg(gp + BMU_IDX(b + 1, room, a.status));
            const uint32_t f[T] = {q.x & 0xffffu, q.x >> 16, q.y & 0xffffu, q.y >> 16,
                                   q.z & 0xffffu, q.z >> 16, q.w & 0xffffu, q.w >> 16};
#pragma unroll
            for (int t = 0; t < T; ++t)
                if (f[t] != 0xffffu) {
                    const ulonglong2 w =
                        __ldg(reinterpret_cast<const ulonglong2 *>(base + (u64)BMU_IDX(f[t], a.D, a.status) * rowbytes));
                    add2(acc[t][0], w.x);
                    add2(acc[t][1], w.y);
                }
        }

        // distances of this slab: the lane's best (two best) of its 4 neurons, per document
        const int col = j0 + lane * 4;
        const float4 n = __ldg(reinterpret_cast<const float4 *>(a.norms + col));
        const float n4[4] = {n.x, n.y, n.z, n.w};
        Keys<TOP2> k[T];
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const float s4[4] = {lo_f(acc[t][0]), hi_f(acc[t][0]), lo_f(acc[t][1]), hi_f(acc[t][1])};
            Best<TOP2> bst;
            bst.init();
#pragma unroll
            for (int c = 0; c < 4; ++c) bst.push(fmaf(-2.f, s4[c], n4[c]), col + c);
            k[t].k1 = make_key(bst.d1, bst.j1);
            k[t].k2 = TOP2 ? make_key(bst.d2, bst.j2) : KEY_WORST;
        }
        // transposing butterfly: halve the documents a lane is responsible for at each step
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const Keys<TOP2> send = (lane & 1) ? k[i] : k[i + 4];
            const Keys<TOP2> keep = (lane & 1) ? k[i + 4] : k[i];
            k[i] = keep;
            k[i].absorb(send.xchg(1));
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const Keys<TOP2> send = (lane & 2) ? k[i] : k[i + 2];
            const Keys<TOP2> keep = (lane & 2) ? k[i + 2] : k[i];
            k[i] = keep;
            k[i].absorb(send.xchg(2));
        }
        {
            const Keys<TOP2> send = (lane & 4) ? k[0] : k[1];
            const Keys<TOP2> keep = (lane & 4) ? k[1] : k[0];
            k[0] = keep;
            k[0].absorb(send.xchg(4));
        }
        k[0].absorb(k[0].xchg(8));
        k[0].absorb(k[0].xchg(16));
        run.absorb(k[0]);
    }

    if (lane < T && orig >= 0)
        Best<TOP2>::commit(run.k1, run.k2, a.state, a.state2, orig, a.first);
}

int launch_sweep_tiles(const TileArgs &a, const bmu_opts &o, cudaStream_t s)
{
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    if ((a.j_hi - a.j_lo) % 128 != 0) {
        set_error("tiled kernel handles whole 128-neuron slabs only");
        return BMU_ERR_INVALID_ARG;
    }
    const int NW = o.warps ? o.warps : 4;
#define BMU_CASE(nw)                                                                        \
    if (NW == nw) {                                                                         \
        const unsigned blocks = (unsigned)((a.n_tiles + nw - 1) / nw);                      \
        if (a.state2) { sweep_tiles_kernel<nw, true><<<blocks, nw * 32, 0, s>>>(a); BMU_LAUNCHED(); }           \
        else { sweep_tiles_kernel<nw, false><<<blocks, nw * 32, 0, s>>>(a); BMU_LAUNCHED(); }                   \
        BMU_CUDA(cudaGetLastError());                                                       \
        return BMU_OK;                                                                      \
    }
    BMU_CASE(2) BMU_CASE(4) BMU_CASE(8) BMU_CASE(16) BMU_CASE(32)
#undef BMU_CASE
    set_error("tiled kernel: warps must be 2, 4, 8, 16 or 32");
    return BMU_ERR_INVALID_ARG;
}

}  // namespace bmu
