// Direct gather-accumulate sweep with the argmin fused in (Section 3; levers of
// Section 4: vector loads, neuron-axis chunking).
//
// One warp carries K documents through the neuron chunk [j_lo, j_hi) slab by
// slab.  A slab is 32*V consecutive neurons: every lane owns V of them and adds,
// for each active feature f of the document, its piece of the codebook row
// W[f*M + slab] -- a 128-bit load per lane, 512 contiguous bytes per warp --
// into fp32 accumulators (x is binary, so there is no multiply).  The rows come
// through L1/L2: all warps of a block walk the slabs in the same order, so the
// rows of frequent features are shared in L1, and the host keeps one chunk of
// the codebook (D * chunk * 4 bytes) resident in L2 by launching chunk by chunk.
// After the last feature each lane turns its sums into distances
// n_j - 2 s_ij (|x_i| is added once at the end), keeps a running minimum with
// a strict "<" over ascending j, and after the last slab the warp reduces
// (distance, index) lexicographically by shuffles and merges it into the
// per-document state that persists across chunks.
#include "common.cuh"

#include <cuda_fp16.h>
#include <math_constants.h>

namespace bmu {

template <int V, int K, int NW, bool VEC, bool TOP2>
__global__ void __launch_bounds__(NW * 32)
sweep_direct_kernel(const SweepArgs a)
{
    static_assert(!VEC || V % 4 == 0, "vector path owns whole float4s");
    constexpr int H = VEC ? V / 4 : V;            // loads per lane per row
    constexpr int STEP = VEC ? 4 : 1;             // floats per load
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t doc0 = ((int64_t)blockIdx.x * NW + warp) * K;
#ifndef BMU_SLAB_SYNC
    if (doc0 >= a.N) return;
#endif

    int beg[K], end[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int64_t i = doc0 + k;
        beg[k] = i < a.N ? __ldg(a.rowptr + i) : 0;
        end[k] = i < a.N ? __ldg(a.rowptr + i + 1) : 0;
    }
    Best<TOP2> best[K];
#pragma unroll
    for (int k = 0; k < K; ++k) best[k].init();

    const uint32_t rowbytes = (uint32_t)(a.M * 4);

    for (int j0 = a.j_lo; j0 < a.j_hi; j0 += 32 * V) {
#ifdef BMU_SLAB_SYNC
        __syncthreads();
#endif
        // this lane's columns of the slab
        int col[H];
        bool act[H];
        const char *base[H];
#pragma unroll
        for (int h = 0; h < H; ++h) {
            col[h] = VEC ? j0 + h * 128 + lane * 4 : j0 + h * 32 + lane;
            act[h] = col[h] < a.j_hi;
            base[h] = reinterpret_cast<const char *>(a.W + (act[h] ? col[h] : a.j_lo));
        }
        float nrm[H][STEP];
#pragma unroll
        for (int h = 0; h < H; ++h)
#pragma unroll
            for (int c = 0; c < STEP; ++c)
                nrm[h][c] = act[h] ? __ldg(a.norms + col[h] + c) : CUDART_INF_F;

#pragma unroll
        for (int k = 0; k < K; ++k) {
            if (doc0 + k >= a.N) continue;             // warp-uniform
            float s[H][STEP];
            if constexpr (VEC) {
                u64 acc[H][2];
#pragma unroll
                for (int h = 0; h < H; ++h) acc[h][0] = acc[h][1] = 0ull;
                for (int eb = beg[k]; eb < end[k]; eb += 32) {
                    const int myf = (eb + lane < end[k]) ? __ldg(a.colidx + eb + lane) : 0;
                    const int c = min(32, end[k] - eb);
                    int q = 0;
                    for (; q + 4 <= c; q += 4) {
                        ulonglong2 w[4][H];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const uint32_t f = (uint32_t)__shfl_sync(0xffffffffu, myf, q + u);
                            const u64 off = (u64)BMU_IDX(f, a.D, a.status) * rowbytes;
#pragma unroll
                            for (int h = 0; h < H; ++h)
                                w[u][h] = act[h]
                                    ? __ldg(reinterpret_cast<const ulonglong2 *>(base[h] + off))
                                    : make_ulonglong2(0ull, 0ull);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
#pragma unroll
                            for (int h = 0; h < H; ++h) {
                                add2(acc[h][0], w[u][h].x);
                                add2(acc[h][1], w[u][h].y);
                            }
                    }
                    for (; q < c; ++q) {
                        const uint32_t f = (uint32_t)__shfl_sync(0xffffffffu, myf, q);
                        const u64 off = (u64)BMU_IDX(f, a.D, a.status) * rowbytes;
#pragma unroll
                        for (int h = 0; h < H; ++h) {
                            const ulonglong2 w = act[h]
                                ? __ldg(reinterpret_cast<const ulonglong2 *>(base[h] + off))
                                : make_ulonglong2(0ull, 0ull);
                            add2(acc[h][0], w.x);
                            add2(acc[h][1], w.y);
                        }
                    }
                }
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    s[h][0] = lo_f(acc[h][0]); s[h][1] = hi_f(acc[h][0]);
                    s[h][2] = lo_f(acc[h][1]); s[h][3] = hi_f(acc[h][1]);
                }
            } else {
#pragma unroll
                for (int h = 0; h < H; ++h) s[h][0] = 0.f;
                for (int eb = beg[k]; eb < end[k]; eb += 32) {
                    const int myf = (eb + lane < end[k]) ? __ldg(a.colidx + eb + lane) : 0;
                    const int c = min(32, end[k] - eb);
                    for (int q = 0; q < c; ++q) {
                        const uint32_t f = (uint32_t)__shfl_sync(0xffffffffu, myf, q);
                        const u64 off = (u64)BMU_IDX(f, a.D, a.status) * rowbytes;
#pragma unroll
                        for (int h = 0; h < H; ++h)
                            if (act[h])
                                s[h][0] += __ldg(reinterpret_cast<const float *>(base[h] + off));
                    }
                }
            }
            // distances of this slab, running minimum over ascending neuron index
#pragma unroll
            for (int h = 0; h < H; ++h)
#pragma unroll
                for (int c = 0; c < STEP; ++c) {
                    best[k].push(fmaf(-2.f, s[h][c], nrm[h][c]), col[h] + c);
                }
        }
    }

#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (doc0 + k >= a.N) continue;
        u64 k1, k2;
        best[k].warp_keys(k1, k2);
        if (lane == 0) Best<TOP2>::commit(k1, k2, a.state, a.state2, doc0 + k, a.first);
    }
}

// ---------------------------------------------------------------------------
// Planned variant of the same sweep: a warp per document, but the feature ids
// come from the tiling pass (ascending 16-bit ids, eight per aligned 128-bit
// word, see plan.cu).  All lanes read the same word, so one broadcast load
// yields eight ids, no shuffle is needed, and the row address is one
// multiply-add.  Only whole slabs are handled here (no per-lane guards in the
// loop); a ragged last slab goes through the generic kernel above.
template <int V, int NW, bool TOP2>
__global__ void __launch_bounds__(NW * 32)
sweep_rows_kernel(const RowsArgs a)
{
    constexpr int H = V / 4;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t p = (int64_t)blockIdx.x * NW + warp;
    if (p >= a.N || (__ldg(a.status) & PLAN_STATUS_OVERFLOW)) return;
    const int32_t orig = __ldg(a.perm + p);
    const int len = __ldg(a.rowptr + orig + 1) - __ldg(a.rowptr + orig);
    const uint4 *gp = a.ids + BMU_IDX((size_t)__ldg(a.doc_off + p) + 1, a.id_groups_cap, a.status);
    [[maybe_unused]] const size_t room = a.id_groups_cap - (size_t)(gp - a.ids);
    const int full = len >> 3, rem = len & 7;
    const uint32_t rowbytes = (uint32_t)(a.M * 4);
    Best<TOP2> best;
    best.init();

    for (int j0 = a.j_lo; j0 < a.j_hi; j0 += 32 * V) {
        const char *base = reinterpret_cast<const char *>(a.W + j0 + lane * 4);
        u64 acc[H][2];
#pragma unroll
        for (int h = 0; h < H; ++h) acc[h][0] = acc[h][1] = 0ull;

        for (int g = 0; g < full; ++g) {
            const uint4 t = __ldg(gp + BMU_IDX(g, room, a.status));
            const uint32_t f[8] = {t.x & 0xffffu, t.x >> 16, t.y & 0xffffu, t.y >> 16,
                                   t.z & 0xffffu, t.z >> 16, t.w & 0xffffu, t.w >> 16};
            ulonglong2 w[8][H];
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int h = 0; h < H; ++h)
                    w[u][h] = __ldg(reinterpret_cast<const ulonglong2 *>(
                        base + (u64)BMU_IDX(f[u], a.D, a.status) * rowbytes + h * 512));
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int h = 0; h < H; ++h) {
                    add2(acc[h][0], w[u][h].x);
                    add2(acc[h][1], w[u][h].y);
                }
        }
        if (rem) {
            const uint4 t = __ldg(gp + BMU_IDX(full, room, a.status));
            const uint32_t f[8] = {t.x & 0xffffu, t.x >> 16, t.y & 0xffffu, t.y >> 16,
                                   t.z & 0xffffu, t.z >> 16, t.w & 0xffffu, t.w >> 16};
#pragma unroll
            for (int u = 0; u < 7; ++u)
                if (u < rem) {
#pragma unroll
                    for (int h = 0; h < H; ++h) {
                        const ulonglong2 w = __ldg(reinterpret_cast<const ulonglong2 *>(
                            base + (u64)BMU_IDX(f[u], a.D, a.status) * rowbytes + h * 512));
                        add2(acc[h][0], w.x);
                        add2(acc[h][1], w.y);
                    }
                }
        }
#pragma unroll
        for (int h = 0; h < H; ++h) {
            const int col = j0 + h * 128 + lane * 4;
            const float4 n = __ldg(reinterpret_cast<const float4 *>(a.norms + col));
            const float s4[4] = {lo_f(acc[h][0]), hi_f(acc[h][0]), lo_f(acc[h][1]), hi_f(acc[h][1])};
            const float n4[4] = {n.x, n.y, n.z, n.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) best.push(fmaf(-2.f, s4[c], n4[c]), col + c);
        }
    }
    u64 k1, k2;
    best.warp_keys(k1, k2);
    if (lane == 0) Best<TOP2>::commit(k1, k2, a.state, a.state2, orig, a.first);
}

// ---------------------------------------------------------------------------
// Half-precision codebook (the paper's own storage, Section 4.2/4.3: 2 bytes per
// weight, loaded as pairs of halves): the planned kernel with rows of
// fp16, eight neurons per 128-bit load, widened to fp32 in registers and
// accumulated in fp32.  Slab = 256 neurons.
template <int NW, bool TOP2>
__global__ void __launch_bounds__(NW * 32)
sweep_rows_f16_kernel(const RowsArgs a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t p = (int64_t)blockIdx.x * NW + warp;
    if (p >= a.N || (__ldg(a.status) & PLAN_STATUS_OVERFLOW)) return;
    const int32_t orig = __ldg(a.perm + p);
    const int len = __ldg(a.rowptr + orig + 1) - __ldg(a.rowptr + orig);
    const uint4 *gp = a.ids + BMU_IDX((size_t)__ldg(a.doc_off + p) + 1, a.id_groups_cap, a.status);
    [[maybe_unused]] const size_t room = a.id_groups_cap - (size_t)(gp - a.ids);
    const int full = len >> 3, rem = len & 7;
    const uint32_t rowbytes = (uint32_t)(a.M * 2);
    const __half *W16 = reinterpret_cast<const __half *>(a.W);
    Best<TOP2> best;
    best.init();

    for (int j0 = a.j_lo; j0 < a.j_hi; j0 += 256) {
        const char *base = reinterpret_cast<const char *>(W16 + j0 + lane * 8);
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        // fp32 sum + fp16 weight in one instruction (the mixed-precision add of sm_100; the
        // widening is exact, so this equals convert-then-add bit for bit)
        auto add_row = [&](const uint4 h) {
            const uint32_t w[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint16_t h0, h1;
                asm("mov.b32 {%0, %1}, %2;" : "=h"(h0), "=h"(h1) : "r"(w[i]));
                asm("add.rn.f32.f16 %0, %1, %0;" : "+f"(acc[2 * i]) : "h"(h0));
                asm("add.rn.f32.f16 %0, %1, %0;" : "+f"(acc[2 * i + 1]) : "h"(h1));
            }
        };
        for (int g = 0; g < full; ++g) {
            const uint4 t = __ldg(gp + BMU_IDX(g, room, a.status));
            const uint32_t f[8] = {t.x & 0xffffu, t.x >> 16, t.y & 0xffffu, t.y >> 16,
                                   t.z & 0xffffu, t.z >> 16, t.w & 0xffffu, t.w >> 16};
            uint4 w[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                w[u] = __ldg(reinterpret_cast<const uint4 *>(base + (u64)BMU_IDX(f[u], a.D, a.status) * rowbytes));
#pragma unroll
            for (int u = 0; u < 8; ++u) add_row(w[u]);
        }
        if (rem) {
            const uint4 t = __ldg(gp + BMU_IDX(full, room, a.status));
            const uint32_t f[8] = {t.x & 0xffffu, t.x >> 16, t.y & 0xffffu, t.y >> 16,
                                   t.z & 0xffffu, t.z >> 16, t.w & 0xffffu, t.w >> 16};
#pragma unroll
            for (int u = 0; u < 7; ++u)
                if (u < rem)
                    add_row(__ldg(reinterpret_cast<const uint4 *>(base + (u64)BMU_IDX(f[u], a.D, a.status) * rowbytes)));
        }
        const int col = j0 + lane * 8;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 n = __ldg(reinterpret_cast<const float2 *>(a.norms + col + 2 * i));
            best.push(fmaf(-2.f, acc[2 * i], n.x), col + 2 * i);
            best.push(fmaf(-2.f, acc[2 * i + 1], n.y), col + 2 * i + 1);
        }
    }
    u64 k1, k2;
    best.warp_keys(k1, k2);
    if (lane == 0) Best<TOP2>::commit(k1, k2, a.state, a.state2, orig, a.first);
}

int launch_sweep_rows_f16(const RowsArgs &a, const bmu_opts &o, cudaStream_t s)
{
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    if ((a.j_hi - a.j_lo) % 256 != 0) {
        set_error("half-precision kernel handles whole 256-neuron slabs only");
        return BMU_ERR_INVALID_ARG;
    }
    const int NW = o.warps ? o.warps : 8;
#define BMU_CASE(nw)                                                                      \
    if (NW == nw) {                                                                       \
        const unsigned blocks = (unsigned)((a.N + nw - 1) / nw);                          \
        if (a.state2) { sweep_rows_f16_kernel<nw, true><<<blocks, nw * 32, 0, s>>>(a); BMU_LAUNCHED(); }      \
        else { sweep_rows_f16_kernel<nw, false><<<blocks, nw * 32, 0, s>>>(a); BMU_LAUNCHED(); }              \
        BMU_CUDA(cudaGetLastError());                                                     \
        return BMU_OK;                                                                    \
    }
    BMU_CASE(8) BMU_CASE(16) BMU_CASE(32)
#undef BMU_CASE
    set_error("half-precision kernel: warps must be 8, 16 or 32");
    return BMU_ERR_INVALID_ARG;
}

template <int V>
static int launch_rows_v(const RowsArgs &a, int NW, cudaStream_t s)
{
#define BMU_CASE(nw)                                                                   \
    if (NW == nw) {                                                                    \
        const unsigned blocks = (unsigned)((a.N + nw - 1) / nw);                       \
        if (a.state2) { sweep_rows_kernel<V, nw, true><<<blocks, nw * 32, 0, s>>>(a); BMU_LAUNCHED(); }    \
        else { sweep_rows_kernel<V, nw, false><<<blocks, nw * 32, 0, s>>>(a); BMU_LAUNCHED(); }            \
        BMU_CUDA(cudaGetLastError());                                                  \
        return BMU_OK;                                                                 \
    }
    BMU_CASE(4) BMU_CASE(8) BMU_CASE(16) BMU_CASE(32)
#undef BMU_CASE
    set_error("planned kernel: warps must be 4, 8, 16 or 32");
    return BMU_ERR_INVALID_ARG;
}

// defaults measured on B200: two 128-bit loads per lane and row, 16 warps per block
int rows_slab_width(const bmu_opts &o) { return 32 * (o.vec ? o.vec : 8); }

int launch_sweep_rows(const RowsArgs &a, const bmu_opts &o, cudaStream_t s)
{
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    const int NW = o.warps ? o.warps : 16;
    const int V = o.vec ? o.vec : 8;
    if ((a.j_hi - a.j_lo) % (32 * V) != 0) {
        set_error("planned kernel handles whole slabs only");
        return BMU_ERR_INVALID_ARG;
    }
    return V == 8 ? launch_rows_v<8>(a, NW, s) : launch_rows_v<4>(a, NW, s);
}

// state -> outputs: out_dist = |x_i| + min_j (n_j - 2 s_ij)
// (a second-best unit that does not exist, M == 1, comes out as index -1 at distance +inf)
__global__ void finalize_kernel(const u64 *__restrict__ state, const u64 *__restrict__ state2,
                                const int32_t *__restrict__ rowptr, int64_t N,
                                int32_t *__restrict__ out_bmu, float *__restrict__ out_dist,
                                int32_t *__restrict__ out_bmu2, float *__restrict__ out_dist2)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const u64 key = state[i];
    const float nx = (float)(rowptr[i + 1] - rowptr[i]);
    out_bmu[i] = (int32_t)(uint32_t)key;
    out_dist[i] = nx + ordered_to_float((uint32_t)(key >> 32));
    if (state2) {
        const u64 k2 = state2[i];
        const bool none = (uint32_t)k2 == 0x7fffffffu;
        out_bmu2[i] = none ? -1 : (int32_t)(uint32_t)k2;
        out_dist2[i] = none ? CUDART_INF_F : nx + ordered_to_float((uint32_t)(k2 >> 32));
    }
}

int launch_finalize(const u64 *state, const u64 *state2, const int32_t *rowptr, int64_t N,
                    int32_t *out_bmu, float *out_dist, int32_t *out_bmu2, float *out_dist2,
                    cudaStream_t s)
{
    if (N == 0) return BMU_OK;
    { finalize_kernel<<<(unsigned)((N + 255) / 256), 256, 0, s>>>(state, state2, rowptr, N, out_bmu,
                                                                out_dist, out_bmu2, out_dist2); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

template <int V, int K, int NW, bool VEC>
static int launch_one(const SweepArgs &a, cudaStream_t s)
{
    const int64_t per_block = (int64_t)NW * K;
    const int64_t blocks = (a.N + per_block - 1) / per_block;
    if (a.state2)
        { sweep_direct_kernel<V, K, NW, VEC, true><<<(unsigned)blocks, NW * 32, 0, s>>>(a); BMU_LAUNCHED(); }
    else
        { sweep_direct_kernel<V, K, NW, VEC, false><<<(unsigned)blocks, NW * 32, 0, s>>>(a); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

template <int V, bool VEC>
static int launch_vk(const SweepArgs &a, int K, int NW, cudaStream_t s)
{
#define BMU_CASE(k, nw) if (K == k && NW == nw) return launch_one<V, k, nw, VEC>(a, s);
    BMU_CASE(1, 8) BMU_CASE(1, 16) BMU_CASE(1, 32)
    BMU_CASE(2, 8) BMU_CASE(2, 16) BMU_CASE(2, 32)
    BMU_CASE(4, 8) BMU_CASE(4, 16) BMU_CASE(4, 32)
#undef BMU_CASE
    set_error("direct kernel: docs_per_warp must be 1, 2 or 4 and warps 8, 16 or 32");
    return BMU_ERR_INVALID_ARG;
}

int launch_sweep_direct(const SweepArgs &a, const bmu_opts &o, cudaStream_t s)
{
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    const int K = o.docs_per_warp ? o.docs_per_warp : 4;
    const int NW = o.warps ? o.warps : 16;
    const bool vec = (a.M % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.W) & 15) == 0) &&
                     (a.j_lo % 4 == 0);
    if (!vec) return launch_vk<4, false>(a, K, NW, s);
    const int V = o.vec ? o.vec : 4;
    if (V == 4) return launch_vk<4, true>(a, K, NW, s);
    if (V == 8) return launch_vk<8, true>(a, K, NW, s);
    set_error("vec must be 4 or 8");
    return BMU_ERR_INVALID_ARG;
}

}  // namespace bmu
