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

static const int BLUR_TILE = 32;
static const int BLUR_RMAX = 24;           // sigma <= 8

struct BlurTaps { int32_t R; float g[2 * BLUR_RMAX + 1]; };

// One block per 32 x 32 tile of one plane: the tile and its halo (zero outside the map) into
// shared memory, the row pass there, the column pass into the output.  Planes 0 .. D-1 are the
// feature planes of `num`, plane D is `cnt`.
__global__ void __launch_bounds__(256)
update_blur_kernel(const uint32_t *__restrict__ num, const uint32_t *__restrict__ cnt, int64_t D,
                   int32_t edge_x, int32_t edge_y, const BlurTaps taps, float *__restrict__ num_blur,
                   float *__restrict__ cnt_blur)
{
    extern __shared__ float sm[];
    const int R = taps.R, span = BLUR_TILE + 2 * R;
    float *in = sm;                          // span x span
    float *mid = sm + span * span;           // span rows x BLUR_TILE columns
    const int64_t plane = blockIdx.z, M = (int64_t)edge_x * edge_y;
    const uint32_t *src = plane < D ? num + plane * M : cnt;
    float *dst = plane < D ? num_blur + plane * M : cnt_blur;
    const int x0 = blockIdx.x * BLUR_TILE, y0 = blockIdx.y * BLUR_TILE;

    for (int idx = threadIdx.x; idx < span * span; idx += blockDim.x) {
        const int r = idx / span, c = idx - r * span;
        const int y = y0 - R + r, x = x0 - R + c;
        in[idx] = (y >= 0 && y < edge_y && x >= 0 && x < edge_x)
                      ? (float)__ldg(src + (int64_t)y * edge_x + x) : 0.f;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < span * BLUR_TILE; idx += blockDim.x) {
        const int r = idx / BLUR_TILE, c = idx - r * BLUR_TILE;
        const float *row = in + r * span + c;
        float s = 0.f;
        for (int d = 0; d <= 2 * R; ++d) s = fmaf(taps.g[d], row[d], s);
        mid[idx] = s;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < BLUR_TILE * BLUR_TILE; idx += blockDim.x) {
        const int r = idx / BLUR_TILE, c = idx - r * BLUR_TILE;
        const int y = y0 + r, x = x0 + c;
        if (y >= edge_y || x >= edge_x) continue;
        const float *col = mid + r * BLUR_TILE + c;
        float s = 0.f;
        for (int d = 0; d <= 2 * R; ++d) s = fmaf(taps.g[d], col[d * BLUR_TILE], s);
        dst[(int64_t)y * edge_x + x] = s;
    }
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

int launch_update_scatter(const int32_t *rowptr, const int32_t *colidx, int64_t N,
                          const int32_t *bmu, int64_t M, uint32_t *num, uint32_t *cnt,
                          cudaStream_t s)
{
    if (N == 0) return BMU_OK;
    update_scatter_kernel<<<(unsigned)((N * 32 + 255) / 256), 256, 0, s>>>(rowptr, colidx, N, bmu,
                                                                          M, num, cnt);
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
    for (int d = -t.R; d <= t.R; ++d)
        t.g[d + t.R] = sigma > 0.f
            ? (float)exp(-(double)(d * d) / (2.0 * (double)sigma * (double)sigma)) : 1.f;
    const int span = BLUR_TILE + 2 * t.R;
    const size_t smem = (size_t)(span * span + span * BLUR_TILE) * sizeof(float);
    const dim3 grid((unsigned)((edge_x + BLUR_TILE - 1) / BLUR_TILE),
                    (unsigned)((edge_y + BLUR_TILE - 1) / BLUR_TILE), (unsigned)(D + 1));
    update_blur_kernel<<<grid, 256, smem, s>>>(num, cnt, D, edge_x, edge_y, t, num_blur, cnt_blur);
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
    if (vec) update_writeback_kernel<true><<<grid, 256, 0, s>>>(num_blur, cnt_blur, M, W);
    else update_writeback_kernel<false><<<grid, 256, 0, s>>>(num_blur, cnt_blur, M, W);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
