// The document-tiling pass (Section 4.1 "tile size", Section 4.2 "tile
// membership"): turns the caller's CSR into the form the staged sweep walks.
//
// The staged sweep gives every lane of a thread block one document, so a
// "tile" here is the 992 documents of one block, which share every staged
// codebook row.  The pass
//   1. orders documents by length (longest first) so that the 32 lanes of a
//      warp, which step through their feature lists together, carry similar
//      numbers of features;
//   2. re-packs every row as ascending 16-bit feature ids in 16-byte groups
//      (8 ids), padded with the sentinel 0xFFFF and closed by one all-sentinel
//      group, so a lane fetches eight ids with one aligned 128-bit load and
//      stops by itself at the end of its row.
// Integer work only; the order of documents never changes any result because
// every document is reduced by one lane on its own.
#include "common.cuh"

#include <cub/device/device_scan.cuh>

namespace bmu {

static const int PLAN_BINS = 1024;

__global__ void plan_hist_kernel(const int32_t *__restrict__ rowptr, int64_t N,
                                 uint32_t *__restrict__ hist)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int len = rowptr[i + 1] - rowptr[i];
    const int bin = PLAN_BINS - 1 - min(len, PLAN_BINS - 1);      // longest rows first
    atomicAdd(hist + bin, 1u);
}

// exclusive scan of the PLAN_BINS counters (one block)
__global__ void plan_scan_bins_kernel(uint32_t *__restrict__ hist, uint32_t *__restrict__ cursor)
{
    __shared__ uint32_t s[PLAN_BINS];
    const int t = threadIdx.x;
    s[t] = hist[t];
    __syncthreads();
    for (int off = 1; off < PLAN_BINS; off <<= 1) {
        const uint32_t v = t >= off ? s[t - off] : 0u;
        __syncthreads();
        s[t] += v;
        __syncthreads();
    }
    cursor[t] = s[t] - hist[t];
}

__global__ void plan_scatter_kernel(const int32_t *__restrict__ rowptr, int64_t N,
                                    uint32_t *__restrict__ cursor, int32_t *__restrict__ perm)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int len = rowptr[i + 1] - rowptr[i];
    const int bin = PLAN_BINS - 1 - min(len, PLAN_BINS - 1);
    perm[atomicAdd(cursor + bin, 1u)] = (int32_t)i;
}

__global__ void plan_identity_kernel(int64_t N, int32_t *__restrict__ perm)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) perm[i] = (int32_t)i;
}

// groups of 8 ids the row at planned position p needs (plus its closing sentinel group)
__global__ void plan_groups_kernel(const int32_t *__restrict__ rowptr,
                                   const int32_t *__restrict__ perm, int64_t N,
                                   uint32_t *__restrict__ ngroups)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= N) return;
    const int32_t i = perm[p];
    const int len = rowptr[i + 1] - rowptr[i];
    ngroups[p] = (uint32_t)((len + 7) / 8 + 1);
}

// One warp per planned document: writes its ascending 16-bit id list.  Rows that
// are not already ascending are ordered by counting, for each id, the ids that
// must precede it (quadratic in the row length, rows are short).
__global__ void __launch_bounds__(256)
plan_fill_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                 const int32_t *__restrict__ perm, const uint32_t *__restrict__ doc_off,
                 int64_t N, uint16_t *__restrict__ ids16)
{
    const int lane = threadIdx.x & 31;
    const int64_t p = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (p >= N) return;
    const int32_t i = perm[p];
    const int beg = rowptr[i], len = rowptr[i + 1] - beg;
    const int32_t *row = colidx + beg;
    uint16_t *dst = ids16 + ((size_t)doc_off[p] + 1) * 8;          // group 0 is the global sentinel
    const int padded = ((len + 7) / 8 + 1) * 8;

    bool sorted = true;
    for (int e = lane; e + 1 < len; e += 32) sorted &= row[e] < row[e + 1];
    sorted = __all_sync(0xffffffffu, sorted);
    if (sorted) {
        for (int e = lane; e < padded; e += 32) dst[e] = e < len ? (uint16_t)row[e] : 0xFFFFu;
    } else {
        for (int e = lane; e < padded; e += 32)
            if (e >= len) dst[e] = 0xFFFFu;
        for (int e = lane; e < len; e += 32) {
            const int32_t f = row[e];
            int rank = 0;
            for (int k = 0; k < len; ++k) {
                const int32_t g = row[k];
                rank += (g < f) || (g == f && k < e);
            }
            dst[rank] = (uint16_t)f;
        }
    }
    if (p == 0 && lane < 8) ids16[lane] = 0xFFFFu;                  // global sentinel group
    if (p == N - 1 && lane < 16) dst[padded + lane] = 0xFFFFu;      // two groups of slack at the end
}

size_t plan_bytes(int64_t N, int64_t nnz, PlanLayout *l)
{
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    size_t off = 0;
    PlanLayout t;
    t.perm_off = off; off = up(off + (size_t)N * 4);
    t.docoff_off = off; off = up(off + (size_t)(N + 1) * 4);
    t.ngroups_off = off; off = up(off + (size_t)(N + 1) * 4);
    t.bins_off = off; off = up(off + (size_t)PLAN_BINS * 4 * 2);
    const size_t groups = (size_t)nnz / 8 + 2 * (size_t)N + 4;
    t.ids_off = off; off = up(off + groups * 16);
    size_t scan_tmp = 0;
    cub::DeviceScan::ExclusiveSum(nullptr, scan_tmp, (uint32_t *)nullptr, (uint32_t *)nullptr,
                                  (int)(N + 1));
    t.scan_off = off; t.scan_bytes = scan_tmp; off = up(off + scan_tmp);
    t.total = off;
    if (l) *l = t;
    return off;
}

int launch_plan(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                int order_by_length, char *ws, const PlanLayout &l, cudaStream_t s)
{
    (void)nnz;
    int32_t *perm = reinterpret_cast<int32_t *>(ws + l.perm_off);
    uint32_t *doc_off = reinterpret_cast<uint32_t *>(ws + l.docoff_off);
    uint32_t *ngroups = reinterpret_cast<uint32_t *>(ws + l.ngroups_off);
    uint32_t *hist = reinterpret_cast<uint32_t *>(ws + l.bins_off);
    uint32_t *cursor = hist + PLAN_BINS;
    uint16_t *ids16 = reinterpret_cast<uint16_t *>(ws + l.ids_off);
    const unsigned blocks = (unsigned)((N + 255) / 256);
    if (order_by_length) {
        BMU_CUDA(cudaMemsetAsync(hist, 0, PLAN_BINS * 4, s));
        plan_hist_kernel<<<blocks, 256, 0, s>>>(rowptr, N, hist);
        plan_scan_bins_kernel<<<1, PLAN_BINS, 0, s>>>(hist, cursor);
        plan_scatter_kernel<<<blocks, 256, 0, s>>>(rowptr, N, cursor, perm);
    } else {
        plan_identity_kernel<<<blocks, 256, 0, s>>>(N, perm);
    }
    plan_groups_kernel<<<blocks, 256, 0, s>>>(rowptr, perm, N, ngroups);
    BMU_CUDA(cudaMemsetAsync(ngroups + N, 0, 4, s));
    size_t tmp = l.scan_bytes;
    BMU_CUDA(cub::DeviceScan::ExclusiveSum(ws + l.scan_off, tmp, ngroups, doc_off, (int)(N + 1), s));
    plan_fill_kernel<<<(unsigned)((N * 32 + 255) / 256), 256, 0, s>>>(rowptr, colidx, perm,
                                                                       doc_off, N, ids16);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
