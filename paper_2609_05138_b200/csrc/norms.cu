// Codebook norms: norms[j] = sum_f W[f*M + j]^2   (the "norms" step, Table 4).
//
// A pure HBM stream over the D x M codebook.  One thread block owns a band of
// columns; its warps take the feature rows round-robin, square and sum in fp64,
// and the per-warp partials are added in a fixed order in shared memory, so
// the result does not depend on scheduling.  No scratch memory.
#include "common.cuh"

#include <cuda_fp16.h>

namespace bmu {

static const int NORM_WARPS = 16;

// VEC: a lane owns 4 consecutive columns (one 16-byte load per row); otherwise a lane owns
// one column.  LX lanes of a warp lie side by side along the columns and 32 / LX along the
// rows: LX = 32 for wide codebooks (a warp reads 512 contiguous bytes of one row), LX = 8 or 2
// for narrow ones, where 128 columns per block would leave most SMs without a block.
template <bool VEC, int LX>
__global__ void __launch_bounds__(NORM_WARPS * 32)
norms_kernel(const float *__restrict__ W, int64_t D, int64_t M, float *__restrict__ norms)
{
    constexpr int C = VEC ? 4 : 1;
    constexpr int LY = 32 / LX;                    // rows a warp reads per step
    constexpr int RSTEP = NORM_WARPS * LY;         // rows the block reads per step
    __shared__ double part[NORM_WARPS][32 * C];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lx = lane % LX, ly = lane / LX;
    const int64_t col = (int64_t)blockIdx.x * (LX * C) + lx * C;
    const bool act = col < M;
    double a[C];
#pragma unroll
    for (int c = 0; c < C; ++c) a[c] = 0.0;

    if (act) {
        const float *p = W + col;
        int64_t f = warp * LY + ly;
        // four rows in flight per thread
        for (; f + 3 * RSTEP < D; f += 4 * RSTEP) {
            float v[4][C];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float *q = p + (f + (int64_t)u * RSTEP) * M;
                if constexpr (VEC) {
                    float4 t = __ldcs(reinterpret_cast<const float4 *>(q));
                    v[u][0] = t.x; v[u][1] = t.y; v[u][2] = t.z; v[u][3] = t.w;
                } else {
                    v[u][0] = __ldcs(q);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    double w = (double)v[u][c];
                    a[c] = fma(w, w, a[c]);
                }
        }
        for (; f < D; f += RSTEP) {
            const float *q = p + f * M;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                double w = (double)q[c];
                a[c] = fma(w, w, a[c]);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < C; ++c) part[warp][lane * C + c] = a[c];
    __syncthreads();
    if (threadIdx.x < LX * C) {
        const int64_t j = (int64_t)blockIdx.x * (LX * C) + threadIdx.x;
        if (j < M) {
            double s = 0.0;               // fixed order: warps, then the row lanes of a warp
#pragma unroll
            for (int w = 0; w < NORM_WARPS; ++w)
#pragma unroll
                for (int r = 0; r < LY; ++r) s += part[w][r * LX * C + threadIdx.x];
            norms[j] = (float)s;
        }
    }
}

// fp16 codebook: a lane owns 8 consecutive columns (one 16-byte load per row)
__global__ void __launch_bounds__(NORM_WARPS * 32)
norms_f16_kernel(const __half *__restrict__ W, int64_t D, int64_t M, float *__restrict__ norms)
{
    __shared__ double part[NORM_WARPS][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t col = (int64_t)blockIdx.x * 256 + lane * 8;
    double a[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) a[c] = 0.0;
    if (col < M) {
        for (int64_t f = warp; f < D; f += NORM_WARPS) {
            const uint4 t = __ldcs(reinterpret_cast<const uint4 *>(W + f * M + col));
            const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 v = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
                a[2 * i] = fma((double)v.x, (double)v.x, a[2 * i]);
                a[2 * i + 1] = fma((double)v.y, (double)v.y, a[2 * i + 1]);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) part[warp][lane * 8 + c] = a[c];
    __syncthreads();
    if (threadIdx.x < 256) {
        const int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x;
        if (j < M) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < NORM_WARPS; ++w) s += part[w][threadIdx.x];
            norms[j] = (float)s;
        }
    }
}

int launch_norms_f16(const void *W16, int64_t D, int64_t M, float *norms, cudaStream_t s)
{
    if (M == 0) return BMU_OK;
    { norms_f16_kernel<<<(unsigned)((M + 255) / 256), NORM_WARPS * 32, 0, s>>>(
        static_cast<const __half *>(W16), D, M, norms); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

int launch_norms(const float *W, int64_t D, int64_t M, float *norms, cudaStream_t s)
{
    if (M == 0) return BMU_OK;
    const bool vec = (M % 4 == 0) && ((reinterpret_cast<uintptr_t>(W) & 15) == 0);
    const int c = vec ? 4 : 1;
    // narrow codebooks: 8 or 2 lanes across the columns instead of 32, so that there are blocks
    // for every SM (M = 1024: 128 blocks of 8 columns instead of 8 blocks of 128)
    const int64_t wide_blocks = (M + 32 * c - 1) / (32 * c);
    const int lx = wide_blocks >= 296 ? 32 : wide_blocks >= 16 ? 8 : 2;
    const int cols = lx * c;
    const unsigned blocks = (unsigned)((M + cols - 1) / cols);
#define BMU_NORMS(V, L) { norms_kernel<V, L><<<blocks, NORM_WARPS * 32, 0, s>>>(W, D, M, norms); BMU_LAUNCHED(); }
    if (vec) {
        if (lx == 32) BMU_NORMS(true, 32) else if (lx == 8) BMU_NORMS(true, 8) else BMU_NORMS(true, 2)
    } else {
        if (lx == 32) BMU_NORMS(false, 32) else if (lx == 8) BMU_NORMS(false, 8) else BMU_NORMS(false, 2)
    }
#undef BMU_NORMS
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
