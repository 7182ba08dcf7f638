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

// VEC: a lane owns 4 consecutive columns (one 16-byte load per row);
// otherwise a lane owns one column.
template <bool VEC>
__global__ void __launch_bounds__(NORM_WARPS * 32)
norms_kernel(const float *__restrict__ W, int64_t D, int64_t M, float *__restrict__ norms)
{
    constexpr int C = VEC ? 4 : 1;
    __shared__ double part[NORM_WARPS][32 * C];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t col = (int64_t)blockIdx.x * (32 * C) + lane * C;
    const bool act = col < M;
    double a[C];
#pragma unroll
    for (int c = 0; c < C; ++c) a[c] = 0.0;

    if (act) {
        const float *p = W + col;
        int64_t f = warp;
        // four rows in flight per thread
        for (; f + 3 * NORM_WARPS < D; f += 4 * NORM_WARPS) {
            float v[4][C];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float *q = p + (f + (int64_t)u * NORM_WARPS) * M;
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
        for (; f < D; f += NORM_WARPS) {
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
    if (threadIdx.x < 32 * C) {
        const int64_t j = (int64_t)blockIdx.x * (32 * C) + threadIdx.x;
        if (j < M) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < NORM_WARPS; ++w) s += part[w][threadIdx.x];
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
    norms_f16_kernel<<<(unsigned)((M + 255) / 256), NORM_WARPS * 32, 0, s>>>(
        static_cast<const __half *>(W16), D, M, norms);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

int launch_norms(const float *W, int64_t D, int64_t M, float *norms, cudaStream_t s)
{
    if (M == 0) return BMU_OK;
    const bool vec = (M % 4 == 0) && ((reinterpret_cast<uintptr_t>(W) & 15) == 0);
    const int cols = vec ? 128 : 32;
    const int64_t blocks = (M + cols - 1) / cols;
    if (vec)
        norms_kernel<true><<<(unsigned)blocks, NORM_WARPS * 32, 0, s>>>(W, D, M, norms);
    else
        norms_kernel<false><<<(unsigned)blocks, NORM_WARPS * 32, 0, s>>>(W, D, M, norms);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
