// The rest of a batch epoch after the search (Table 4: "scatter", "blur",
// "write-back"; Section 6: the scatter into accumulators is O(N.nnz), the blur is
// the O(M) term).  The paper times these steps without printing formulas; this is
// the textbook batch update on a rectangular, non-periodic map of edge_y rows by
// edge_x columns (neuron j = y * edge_x + x):
//
//   scatter     num[f][j] = #{ i : bmu_i = j and f in x_i },  cnt[j] = #{ i : bmu_i = j }
//               -- integer counters, exact
//   blur        B[f][j] = sum_k h(j, k) num[f][k],  c[j] = sum_k h(j, k) cnt[k],
//               h = exp(-(dx^2 + dy^2) / (2 sigma^2)) for |dx|, |dy| <= R = ceil(3 sigma)
//   write-back  W[f][j] = B[f][j] / c[j] where c[j] > 0, otherwise unchanged
//
// All three are bound by HBM: the scatter by its scattered 4-byte atomics, the
// blur and the write-back by one read and one write of a D x M plane set.
#include "common.cuh"

#include <math.h>

namespace bmu {

// One warp per document: its unit's counter, then one atomic per listed feature.
__global__ void __launch_bounds__(256)
update_scatter_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                      int64_t N, const int32_t *__restrict__ bmu, int64_t M,
                      uint32_t *__restrict__ num, uint32_t *__restrict__ cnt)
{
    const int lane = threadIdx.x & 31;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= N) return;
    const int64_t j = __ldg(bmu + i);
    const int beg = __ldg(rowptr + i), end = __ldg(rowptr + i + 1);
    if (lane == 0) atomicAdd(cnt + j, 1u);
    for (int e = beg + lane; e < end; e += 32)
        atomicAdd(num + (int64_t)__ldg(colidx + e) * M + j, 1u);
}

static const int BLUR_TX = 64, BLUR_TY = 32;   // outputs per block
static const int BLUR_RMAX = 24;               // sigma <= 8

// taps g[-R..R] at gp[3 .. 3 + 2R], three zeros on either side so that a window value can be
// offered to four neighbouring outputs without a range test
struct BlurTaps { int32_t R; float gp[2 * BLUR_RMAX + 1 + 6]; };

// One block per 32 x 64 tile of one plane: the tile and its halo (zero outside the map) into
// shared memory; the row pass there, four neighbouring outputs per thread from 128-bit
// shared-memory loads; the column pass into the output, four outputs down a column per thread.
// Planes 0 .. D-1 are the feature planes of `num`, plane D is `cnt`.
__global__ void __launch_bounds__(256)
update_blur_kernel(const uint32_t *__restrict__ num, const uint32_t *__restrict__ cnt, int64_t D,
                   int32_t edge_x, int32_t edge_y, const BlurTaps taps, float *__restrict__ num_blur,
                   float *__restrict__ cnt_blur)
{
    extern __shared__ __align__(16) float sm[];
    const int R = taps.R, span_y = BLUR_TY + 2 * R;
    const int pitch = (BLUR_TX + 2 * R + 3) / 4 * 4 + 4;     // floats per staged row (16-byte rows)
    float *in = sm;                          // span_y x pitch
    float *mid = sm + span_y * pitch;        // span_y x BLUR_TX
    const int64_t plane = blockIdx.z, M = (int64_t)edge_x * edge_y;
    const uint32_t *src = plane < D ? num + plane * M : cnt;
    float *dst = plane < D ? num_blur + plane * M : cnt_blur;
    const int x0 = blockIdx.x * BLUR_TX, y0 = blockIdx.y * BLUR_TY;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;

    for (int r = ty; r < span_y; r += 8) {
        const int y = y0 - R + r;
        const bool row_in = y >= 0 && y < edge_y;
        for (int c = tx; c < pitch; c += 32) {
            const int x = x0 - R + c;
            in[r * pitch + c] = (row_in && x >= 0 && x < edge_x)
                                    ? (float)__ldg(src + (int64_t)y * edge_x + x) : 0.f;
        }
    }
    __syncthreads();
    // row pass: item = (row r, group of four outputs c4); output x = 4 c4 + o reads in[r][x + d]
    const int groups = BLUR_TX / 4;
    for (int item = threadIdx.x; item < span_y * groups; item += 256) {
        const int r = item / groups, c4 = item - r * groups;
        const float4 *win = reinterpret_cast<const float4 *>(in + r * pitch + 4 * c4);
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        const int pieces = (4 + 2 * R + 3) / 4;
        for (int k = 0; k < pieces; ++k) {
            const float4 v = win[k];
            const float *g = taps.gp + 4 * k;                // value e = 4k + i serves output o with
            a0 = fmaf(g[3], v.x, a0); a1 = fmaf(g[2], v.x, a1);   // tap d = e - o: gp[e - o + 3]
            a2 = fmaf(g[1], v.x, a2); a3 = fmaf(g[0], v.x, a3);
            a0 = fmaf(g[4], v.y, a0); a1 = fmaf(g[3], v.y, a1);
            a2 = fmaf(g[2], v.y, a2); a3 = fmaf(g[1], v.y, a3);
            a0 = fmaf(g[5], v.z, a0); a1 = fmaf(g[4], v.z, a1);
            a2 = fmaf(g[3], v.z, a2); a3 = fmaf(g[2], v.z, a3);
            a0 = fmaf(g[6], v.w, a0); a1 = fmaf(g[5], v.w, a1);
            a2 = fmaf(g[4], v.w, a2); a3 = fmaf(g[3], v.w, a3);
        }
        *reinterpret_cast<float4 *>(mid + r * BLUR_TX + 4 * c4) = make_float4(a0, a1, a2, a3);
    }
    __syncthreads();
    // column pass: item = (group of four rows r4, column c)
    for (int item = threadIdx.x; item < (BLUR_TY / 4) * BLUR_TX; item += 256) {
        const int r4 = item / BLUR_TX, c = item - r4 * BLUR_TX;
        const float *col = mid + (4 * r4) * BLUR_TX + c;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        for (int e = 0; e < 4 + 2 * R; ++e) {
            const float v = col[e * BLUR_TX];
            const float *g = taps.gp + e;
            a0 = fmaf(g[3], v, a0); a1 = fmaf(g[2], v, a1);
            a2 = fmaf(g[1], v, a2); a3 = fmaf(g[0], v, a3);
        }
        const int x = x0 + c, y = y0 + 4 * r4;
        if (x < edge_x) {
            if (y < edge_y) dst[(int64_t)y * edge_x + x] = a0;
            if (y + 1 < edge_y) dst[(int64_t)(y + 1) * edge_x + x] = a1;
            if (y + 2 < edge_y) dst[(int64_t)(y + 2) * edge_x + x] = a2;
            if (y + 3 < edge_y) dst[(int64_t)(y + 3) * edge_x + x] = a3;
        }
    }
}


// ---- the same blur for radii 1 .. 8 on maps whose rows are whole 16-byte pieces ----------
// One block per 64 x 64 tile of one plane, radius a template parameter so that every loop
// unrolls and the taps sit in registers.  Packed fp32 arithmetic throughout (fma.rn.f32x2):
// the row pass works on two map rows at once (the tile is staged as (row 2p, row 2p+1) pairs),
// the column pass on two neighbouring columns at once, and the outputs leave as 8-byte stores:
// 47 warp instructions per 32 outputs against 84 for the general kernel above.
__device__ __forceinline__ void fma2(u64 &acc, u64 a, u64 b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ u64 pack2(float lo, float hi)
{
    return ((u64)__float_as_uint(hi) << 32) | __float_as_uint(lo);
}

template <int R> struct BlurFast {
    static constexpr int TX = 64, TY = 64;
    static constexpr int RP = (R + 3) / 4 * 4;          // halo in x, whole 16-byte pieces
    static constexpr int SPAN = TY + 2 * R;             // staged rows (even)
    static constexpr int NRP = SPAN / 2;                // staged row pairs
    static constexpr int NC = (TX + 2 * RP) / 4;        // 16-byte pieces per staged row
    static constexpr int PX = TX + 2 * RP + 1;          // pairs per staged row pair (odd pitch:
                                                        // lanes over row pairs hit distinct banks)
    static constexpr int PM = TX + 4;                   // floats per row of the row-pass result
    static constexpr size_t SMEM = (size_t)SPAN * PM * 4 + (size_t)NRP * PX * 8;
};

template <int R>
__global__ void __launch_bounds__(256)
update_blur_fast_kernel(const uint32_t *__restrict__ num, const uint32_t *__restrict__ cnt, int64_t D,
                        int32_t edge_x, int32_t edge_y, const BlurTaps taps,
                        float *__restrict__ num_blur, float *__restrict__ cnt_blur)
{
    using F = BlurFast<R>;
    extern __shared__ __align__(16) unsigned char smraw[];
    float *mid = reinterpret_cast<float *>(smraw);                          // SPAN x PM
    float2 *in2 = reinterpret_cast<float2 *>(smraw + (size_t)F::SPAN * F::PM * 4);   // NRP x PX
    const int64_t plane = blockIdx.z, M = (int64_t)edge_x * edge_y;
    const uint32_t *src = plane < D ? num + plane * M : cnt;
    float *dst = plane < D ? num_blur + plane * M : cnt_blur;
    const int x0 = blockIdx.x * F::TX, y0 = blockIdx.y * F::TY;

    // taps g[-R .. R] are symmetric: ts[k] = (g[k], g[k]) for k = |d|
    u64 ts[R + 1];
#pragma unroll
    for (int k = 0; k <= R; ++k) ts[k] = pack2(taps.gp[3 + R + k], taps.gp[3 + R + k]);

    // stage the tile and its halo as pairs of rows, zero outside the map
    for (int item = threadIdx.x; item < F::NRP * F::NC; item += 256) {
        const int rp = item / F::NC, q = item - rp * F::NC;
        const int x = x0 - F::RP + 4 * q, y = y0 - R + 2 * rp;
        uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
        if (x >= 0 && x < edge_x) {
            if (y >= 0 && y < edge_y)
                a = __ldcs(reinterpret_cast<const uint4 *>(src + (int64_t)y * edge_x + x));
            if (y + 1 >= 0 && y + 1 < edge_y)
                b = __ldcs(reinterpret_cast<const uint4 *>(src + (int64_t)(y + 1) * edge_x + x));
        }
        float2 *o = in2 + rp * F::PX + 4 * q;
        const float2 v[4] = {make_float2((float)a.x, (float)b.x), make_float2((float)a.y, (float)b.y),
                             make_float2((float)a.z, (float)b.z), make_float2((float)a.w, (float)b.w)};
        // neighbouring lanes sit 32 bytes apart: lane l stores its four pairs starting with
        // pair (l / 4) % 4, so that 16 lanes hit 16 different bank pairs at every step
        const int rot = (threadIdx.x >> 2) & 3;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int kk = (k + rot) & 3;
            const float2 lo = (kk & 1) ? v[1] : v[0], hi = (kk & 1) ? v[3] : v[2];
            o[kk] = (kk & 2) ? hi : lo;
        }
    }
    __syncthreads();
    // row pass: item = (group of four outputs g4, row pair rp), lanes over row pairs
    for (int item = threadIdx.x; item < F::NRP * (F::TX / 4); item += 256) {
        const int g4 = item / F::NRP, rp = item - g4 * F::NRP;
        const u64 *win = reinterpret_cast<const u64 *>(in2 + rp * F::PX + (F::RP - R) + 4 * g4);
        u64 acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
        for (int e = 0; e < 4 + 2 * R; ++e) {
            const u64 v = win[e];
#pragma unroll
            for (int o = 0; o < 4; ++o) {
                const int d = e - o - R;                 // tap offset of input e for output o
                if (d >= -R && d <= R) fma2(acc[o], ts[d < 0 ? -d : d], v);
            }
        }
        float *m0 = mid + (2 * rp) * F::PM + 4 * g4;
        *reinterpret_cast<float4 *>(m0) = make_float4(lo_f(acc[0]), lo_f(acc[1]), lo_f(acc[2]), lo_f(acc[3]));
        *reinterpret_cast<float4 *>(m0 + F::PM) =
            make_float4(hi_f(acc[0]), hi_f(acc[1]), hi_f(acc[2]), hi_f(acc[3]));
    }
    __syncthreads();
    // column pass: a thread takes two neighbouring columns and eight rows
    {
        const int c2 = threadIdx.x & 31, rg = threadIdx.x >> 5;
        const float *col = mid + (8 * rg) * F::PM + 2 * c2;
        u64 acc[8] = {0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull};
#pragma unroll
        for (int e = 0; e < 8 + 2 * R; ++e) {
            const u64 v = *reinterpret_cast<const u64 *>(col + e * F::PM);
#pragma unroll
            for (int o = 0; o < 8; ++o) {
                const int d = e - o - R;
                if (d >= -R && d <= R) fma2(acc[o], ts[d < 0 ? -d : d], v);
            }
        }
        const int x = x0 + 2 * c2, y = y0 + 8 * rg;
        if (x < edge_x) {
#pragma unroll
            for (int o = 0; o < 8; ++o)
                if (y + o < edge_y)
                    __stcs(reinterpret_cast<float2 *>(dst + (int64_t)(y + o) * edge_x + x),
                           make_float2(lo_f(acc[o]), hi_f(acc[o])));
        }
    }
}

template <int R>
static int launch_blur_fast(const uint32_t *num, const uint32_t *cnt, int64_t D, int32_t edge_x,
                            int32_t edge_y, const BlurTaps &t, float *num_blur, float *cnt_blur,
                            cudaStream_t s)
{
    using F = BlurFast<R>;
    static bool configured[64];
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        BMU_CUDA(cudaFuncSetAttribute(update_blur_fast_kernel<R>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)F::SMEM));
        configured[dev] = true;
    }
    const dim3 grid((unsigned)((edge_x + F::TX - 1) / F::TX), (unsigned)((edge_y + F::TY - 1) / F::TY),
                    (unsigned)(D + 1));
    { update_blur_fast_kernel<R><<<grid, 256, F::SMEM, s>>>(num, cnt, D, edge_x, edge_y, t, num_blur,
                                                         cnt_blur); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

// One row of W per blockIdx.y; float4 pieces when the row pitch allows.
template <bool VEC>
__global__ void __launch_bounds__(256)
update_writeback_kernel(const float *__restrict__ num_blur, const float *__restrict__ cnt_blur,
                        int64_t M, float *__restrict__ W)
{
    const int64_t row = (int64_t)blockIdx.y * M;
    if (VEC) {
        const int64_t n4 = M / 4;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
             i += (int64_t)gridDim.x * blockDim.x) {
            const float4 c = __ldg(reinterpret_cast<const float4 *>(cnt_blur) + i);
            const float4 b = __ldcs(reinterpret_cast<const float4 *>(num_blur + row) + i);
            float4 w = reinterpret_cast<float4 *>(W + row)[i];
            if (c.x > 0.f) w.x = __fdiv_rn(b.x, c.x);
            if (c.y > 0.f) w.y = __fdiv_rn(b.y, c.y);
            if (c.z > 0.f) w.z = __fdiv_rn(b.z, c.z);
            if (c.w > 0.f) w.w = __fdiv_rn(b.w, c.w);
            reinterpret_cast<float4 *>(W + row)[i] = w;
        }
    } else {
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < M;
             i += (int64_t)gridDim.x * blockDim.x) {
            const float c = __ldg(cnt_blur + i);
            if (c > 0.f) W[row + i] = __fdiv_rn(__ldcs(num_blur + row + i), c);
        }
    }
}


// Stopping metrics of an epoch (Table 4 "stopping metric"; Section 5: the second-best unit feeds
// the topographic error): mean d, mean sqrt(max(d, 0)) and the fraction of documents whose best
// and second-best units are not neighbours on the map.  fp64 sums in a fixed order (grid-stride
// partition, shuffle tree, warps in order, blocks in order by the last block to finish), so a
// call gives the same bits every time.
static const int ME_BLOCKS = 592, ME_THREADS = 256;

__global__ void __launch_bounds__(ME_THREADS)
map_errors_kernel(const int32_t *__restrict__ bmu, const int32_t *__restrict__ bmu2,
                  const float *__restrict__ dist, int64_t N, int32_t edge_x, int32_t adjacency,
                  double *__restrict__ part, unsigned int *__restrict__ ticket,
                  double *__restrict__ out)
{
    double sd = 0.0, sr = 0.0, er = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * ME_THREADS + threadIdx.x; i < N;
         i += (int64_t)ME_BLOCKS * ME_THREADS) {
        const double d = (double)__ldg(dist + i);
        sd += d;
        sr += d > 0.0 ? sqrt(d) : 0.0;
        const int32_t b2 = __ldg(bmu2 + i);
        if (b2 >= 0) {
            const int32_t b1 = __ldg(bmu + i);
            const int32_t dx = abs(b1 % edge_x - b2 % edge_x), dy = abs(b1 / edge_x - b2 / edge_x);
            const bool near = adjacency == 8 ? max(dx, dy) == 1 : dx + dy == 1;
            er += near ? 0.0 : 1.0;
        }
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        sd += __shfl_xor_sync(0xffffffffu, sd, m);
        sr += __shfl_xor_sync(0xffffffffu, sr, m);
        er += __shfl_xor_sync(0xffffffffu, er, m);
    }
    __shared__ double wsum[3][ME_THREADS / 32];
    __shared__ bool last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { wsum[0][warp] = sd; wsum[1][warp] = sr; wsum[2][warp] = er; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0, e = 0.0;
        for (int w = 0; w < ME_THREADS / 32; ++w) { a += wsum[0][w]; b += wsum[1][w]; e += wsum[2][w]; }
        part[blockIdx.x] = a;
        part[ME_BLOCKS + blockIdx.x] = b;
        part[2 * ME_BLOCKS + blockIdx.x] = e;
        __threadfence();
        last = atomicAdd(ticket, 1u) == ME_BLOCKS - 1;
    }
    __syncthreads();
    if (last && threadIdx.x < 3) {
        __threadfence();
        const volatile double *p = part + threadIdx.x * ME_BLOCKS;
        double s = 0.0;
        for (int b = 0; b < ME_BLOCKS; ++b) s += p[b];
        out[threadIdx.x] = s / (double)N;
    }
}

int launch_update_scatter(const int32_t *rowptr, const int32_t *colidx, int64_t N,
                          const int32_t *bmu, int64_t M, uint32_t *num, uint32_t *cnt,
                          cudaStream_t s)
{
    if (N == 0) return BMU_OK;
    { update_scatter_kernel<<<(unsigned)((N * 32 + 255) / 256), 256, 0, s>>>(rowptr, colidx, N, bmu,
                                                                          M, num, cnt); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

int launch_update_blur(const uint32_t *num, const uint32_t *cnt, int64_t D, int32_t edge_x,
                       int32_t edge_y, float sigma, float *num_blur, float *cnt_blur,
                       cudaStream_t s)
{
    BlurTaps t;
    t.R = sigma > 0.f ? (int)ceil(3.0 * (double)sigma) : 0;
    if (t.R > BLUR_RMAX) {
        set_error("blur: sigma %.3f needs a radius of %d cells, the kernel holds %d (sigma <= 8)",
                  (double)sigma, t.R, BLUR_RMAX);
        return BMU_ERR_UNSUPPORTED;
    }
    for (int i = 0; i < 2 * BLUR_RMAX + 1 + 6; ++i) t.gp[i] = 0.f;
    for (int d = -t.R; d <= t.R; ++d)
        t.gp[d + t.R + 3] = sigma > 0.f
            ? (float)exp(-(double)(d * d) / (2.0 * (double)sigma * (double)sigma)) : 1.f;
    // radii 1 .. 8 on maps whose rows are whole, aligned 16-byte pieces: the unrolled kernel
    const bool aligned = edge_x % 4 == 0 &&
                         ((reinterpret_cast<uintptr_t>(num) | reinterpret_cast<uintptr_t>(cnt) |
                           reinterpret_cast<uintptr_t>(num_blur) | reinterpret_cast<uintptr_t>(cnt_blur)) & 15) == 0;
    if (aligned && t.R >= 1 && t.R <= 8) {
        switch (t.R) {
        case 1: return launch_blur_fast<1>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        case 2: return launch_blur_fast<2>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        case 3: return launch_blur_fast<3>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        case 4: return launch_blur_fast<4>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        case 5: return launch_blur_fast<5>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        case 6: return launch_blur_fast<6>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        case 7: return launch_blur_fast<7>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        default: return launch_blur_fast<8>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur, s);
        }
    }
    const int span_y = BLUR_TY + 2 * t.R;
    const int pitch = (BLUR_TX + 2 * t.R + 3) / 4 * 4 + 4;
    const size_t smem = (size_t)(span_y * pitch + span_y * BLUR_TX) * sizeof(float);
    static bool configured[64];
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        BMU_CUDA(cudaFuncSetAttribute(update_blur_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      64 * 1024));
        configured[dev] = true;
    }
    const dim3 grid((unsigned)((edge_x + BLUR_TX - 1) / BLUR_TX),
                    (unsigned)((edge_y + BLUR_TY - 1) / BLUR_TY), (unsigned)(D + 1));
    { update_blur_kernel<<<grid, 256, smem, s>>>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

int launch_update_writeback(const float *num_blur, const float *cnt_blur, int64_t D, int64_t M,
                            float *W, cudaStream_t s)
{
    if (D * M == 0) return BMU_OK;
    const bool vec = M % 4 == 0 && ((reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(num_blur) |
                                     reinterpret_cast<uintptr_t>(cnt_blur)) & 15) == 0;
    const int64_t per_row = vec ? M / 4 : M;
    const dim3 grid((unsigned)((per_row + 255) / 256 < 64 ? (per_row + 255) / 256 : 64), (unsigned)D);
    if (vec) { update_writeback_kernel<true><<<grid, 256, 0, s>>>(num_blur, cnt_blur, M, W); BMU_LAUNCHED(); }
    else { update_writeback_kernel<false><<<grid, 256, 0, s>>>(num_blur, cnt_blur, M, W); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

size_t map_errors_workspace_bytes() { return 256 + (size_t)3 * ME_BLOCKS * sizeof(double); }

int launch_map_errors(const int32_t *bmu, const int32_t *bmu2, const float *dist, int64_t N,
                      int32_t edge_x, int32_t adjacency, double *out, void *ws, cudaStream_t s)
{
    if (N == 0) {
        BMU_CUDA(cudaMemsetAsync(out, 0, 3 * sizeof(double), s));
        return BMU_OK;
    }
    unsigned int *ticket = static_cast<unsigned int *>(ws);
    double *part = reinterpret_cast<double *>(static_cast<char *>(ws) + 256);
    BMU_CUDA(cudaMemsetAsync(ticket, 0, sizeof(unsigned int), s));
    { map_errors_kernel<<<ME_BLOCKS, ME_THREADS, 0, s>>>(bmu, bmu2, dist, N, edge_x, adjacency, part,
                                                      ticket, out); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
