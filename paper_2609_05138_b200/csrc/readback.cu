// Arg-min read-back over a materialised score block: the second half of the OTHER way to do
// the search (Section 3: a sparse-dense product writes the whole document-by-neuron score
// block, a separate kernel then reads it back and reduces each row; Section 4.4 tunes that
// read-back from a thread per row to a warp per row with vector loads).  It exists here so
// that the fused search can be compared with a tuned version of that route on the same GPU.
//
// One warp per document row.  A lane reads 16 bytes at a time (4 fp32 or 8 fp16 scores), the
// warp 512 contiguous bytes per step, four steps in flight; the distance n_j - 2 s_ij is formed
// on the fly, each lane keeps its best in ascending j (strict <), the warp reduces the packed
// (distance, index) keys, |x_i| is added once at the end.  Pure stream: the block is read once.
#include "common.cuh"

#include <cuda_fp16.h>

namespace bmu {

static const int RB_WARPS = 8;

template <bool HALF>
__global__ void __launch_bounds__(RB_WARPS * 32)
readback_argmin_kernel(const void *__restrict__ scores, int64_t n_rows, int64_t M,
                       const float *__restrict__ norms, const int32_t *__restrict__ rowptr,
                       int32_t *__restrict__ out_bmu, float *__restrict__ out_dist)
{
    constexpr int E = HALF ? 8 : 4;                    // scores per 16-byte load
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * RB_WARPS + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    const uint4 *src = reinterpret_cast<const uint4 *>(
        static_cast<const char *>(scores) + (size_t)row * (size_t)M * (HALF ? 2 : 4));
    const int64_t n_vec = M / E;                       // M is a multiple of E
    Best<false> best;
    best.init();
    auto take = [&](const uint4 v, int64_t i) {
        const int j0 = (int)(i * E);
        float s[E];
        if constexpr (HALF) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[k]));
                s[2 * k] = f.x;
                s[2 * k + 1] = f.y;
            }
        } else {
            s[0] = __uint_as_float(v.x); s[1] = __uint_as_float(v.y);
            s[2] = __uint_as_float(v.z); s[3] = __uint_as_float(v.w);
        }
#pragma unroll
        for (int k = 0; k < E; k += 4) {
            const float4 n = __ldg(reinterpret_cast<const float4 *>(norms + j0 + k));
            best.push(fmaf(-2.f, s[k], n.x), j0 + k);
            best.push(fmaf(-2.f, s[k + 1], n.y), j0 + k + 1);
            best.push(fmaf(-2.f, s[k + 2], n.z), j0 + k + 2);
            best.push(fmaf(-2.f, s[k + 3], n.w), j0 + k + 3);
        }
    };
    int64_t i = lane;
    for (; i + 96 < n_vec; i += 128) {                 // four loads in flight per lane
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldcs(src + i + 32 * u);
#pragma unroll
        for (int u = 0; u < 4; ++u) take(v[u], i + 32 * u);
    }
    for (; i < n_vec; i += 32) take(__ldcs(src + i), i);
    u64 k1, k2;
    best.warp_keys(k1, k2);
    if (lane == 0) {
        const float nx = (float)(rowptr[row + 1] - rowptr[row]);
        out_bmu[row] = (int32_t)(uint32_t)k1;
        out_dist[row] = nx + ordered_to_float((uint32_t)(k1 >> 32));
    }
}

int launch_readback_argmin(const void *scores, int half, int64_t n_rows, int64_t M,
                           const float *norms, const int32_t *rowptr, int32_t *out_bmu,
                           float *out_dist, cudaStream_t s)
{
    if (n_rows == 0) return BMU_OK;
    const unsigned blocks = (unsigned)((n_rows + RB_WARPS - 1) / RB_WARPS);
    if (half) { readback_argmin_kernel<true><<<blocks, RB_WARPS * 32, 0, s>>>(scores, n_rows, M, norms, rowptr, out_bmu, out_dist); BMU_LAUNCHED(); }
    else { readback_argmin_kernel<false><<<blocks, RB_WARPS * 32, 0, s>>>(scores, n_rows, M, norms, rowptr, out_bmu, out_dist); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
