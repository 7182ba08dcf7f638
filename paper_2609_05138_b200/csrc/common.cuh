// Shared device/host helpers of the BMU library (CUDA path only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "bmu.h"

namespace bmu {

typedef unsigned long long u64;

// ---- error plumbing -------------------------------------------------------
void set_error(const char *fmt, ...);
int cuda_fail(cudaError_t e, const char *what);

#define BMU_CUDA(call)                                       \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) return bmu::cuda_fail(e__, #call); \
    } while (0)

// kernels of this library that the calling thread has launched (bmu_kernel_launches)
extern thread_local unsigned long long g_kernel_launches;
#define BMU_LAUNCHED() (++bmu::g_kernel_launches)

// ---- bounds-checked build (-DBMU_BOUNDS_CHECK) -------------------------------
// Every address a kernel derives from a feature id, a neuron index or a scanned
// offset is checked before it is used.  A violation sets STATUS_BOUNDS in the
// status word and the access goes to element 0 of the same array instead (never
// a trap, never an access outside the array); the results of that call are then
// invalid, which the status word says.  In the normal build the macros cost nothing.
static const uint32_t STATUS_BOUNDS = 128u;
#ifdef __CUDACC__
#ifdef BMU_BOUNDS_CHECK
__device__ __forceinline__ uint32_t checked_index(unsigned long long i, unsigned long long n,
                                                  uint32_t *status)
{
    if (i < n) return (uint32_t)i;
    if (status) atomicOr(status, STATUS_BOUNDS);
    return 0u;
}
#define BMU_IDX(i, n, status) bmu::checked_index((unsigned long long)(i), (unsigned long long)(n), (status))
#define BMU_EXPECT(cond, status) do { if (!(cond) && (status)) atomicOr((status), bmu::STATUS_BOUNDS); } while (0)
#else
#define BMU_IDX(i, n, status) (i)
#define BMU_EXPECT(cond, status) do { } while (0)
#endif
#endif

// ---- (distance, index) keys ----------------------------------------------
// A 64-bit key whose unsigned order is the lexicographic order of (distance,
// neuron index): the smallest key is the smallest distance and, among equal
// distances, the lowest index -- the tie rule of the search.  The float is
// mapped to an unsigned int that sorts like the float does.
__host__ __device__ __forceinline__ uint32_t float_to_ordered(float x)
{
#ifdef __CUDA_ARCH__
    uint32_t b = __float_as_uint(x);
#else
    union { float f; uint32_t u; } c; c.f = x; uint32_t b = c.u;
#endif
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__host__ __device__ __forceinline__ float ordered_to_float(uint32_t o)
{
    uint32_t b = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
#ifdef __CUDA_ARCH__
    return __uint_as_float(b);
#else
    union { float f; uint32_t u; } c; c.u = b; return c.f;
#endif
}

__host__ __device__ __forceinline__ u64 make_key(float d, int32_t j)
{
    return ((u64)float_to_ordered(d) << 32) | (uint32_t)j;
}

static const u64 KEY_WORST = ~0ull;

#ifdef __CUDACC__
// Running minimum of one lane / warp / document: the best unit, and with TOP2 also
// the second-best unit (Table 5: the paper's kernel tracks it for topographic
// error).  push() must see a lane's neurons in ascending index order; ties then
// keep the lower index.  Across lanes and chunks the 64-bit keys decide.
template <bool TOP2>
struct Best {
    float d1, d2;
    int j1, j2;
    __device__ __forceinline__ void init()
    {
        d1 = d2 = __int_as_float(0x7f800000);
        j1 = j2 = 0x7fffffff;
    }
    __device__ __forceinline__ void push(float d, int j)
    {
        if (d < d1) {
            if (TOP2) { d2 = d1; j2 = j1; }
            d1 = d; j1 = j;
        } else if (TOP2 && d < d2) {
            d2 = d; j2 = j;
        }
    }
    static __device__ __forceinline__ void merge(u64 &a1, u64 &a2, u64 b1, u64 b2)
    {
        const u64 lo = a1 < b1 ? a1 : b1, mid = a1 < b1 ? b1 : a1;
        const u64 rest = a2 < b2 ? a2 : b2;
        a1 = lo;
        a2 = mid < rest ? mid : rest;
    }
    // warp-wide result into (k1, k2) on every lane
    __device__ __forceinline__ void warp_keys(u64 &k1, u64 &k2) const
    {
        k1 = make_key(d1, j1);
        k2 = TOP2 ? make_key(d2, j2) : KEY_WORST;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const u64 o1 = __shfl_xor_sync(0xffffffffu, k1, off);
            if (TOP2) {
                const u64 o2 = __shfl_xor_sync(0xffffffffu, k2, off);
                merge(k1, k2, o1, o2);
            } else {
                k1 = o1 < k1 ? o1 : k1;
            }
        }
    }
    // merge the warp's result into the per-document state (one owner per document)
    static __device__ __forceinline__ void commit(u64 k1, u64 k2, u64 *state, u64 *state2,
                                                  int64_t doc, bool first)
    {
        if (!first) {
            if (TOP2) merge(k1, k2, state[doc], state2[doc]);
            else { const u64 old = state[doc]; k1 = old < k1 ? old : k1; }
        }
        state[doc] = k1;
        if (TOP2) state2[doc] = k2;
    }
};

// packed fp32 pair add: two IEEE round-to-nearest adds in one issue slot (sm_100a)
__device__ __forceinline__ void add2(u64 &acc, u64 w)
{
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc) : "l"(w));
}
__device__ __forceinline__ float lo_f(u64 p) { return __uint_as_float((uint32_t)p); }
__device__ __forceinline__ float hi_f(u64 p) { return __uint_as_float((uint32_t)(p >> 32)); }
#endif

// ---- kernels' host launchers (one per .cu file) ---------------------------
int launch_norms(const float *W, int64_t D, int64_t M, float *norms, cudaStream_t s);
int launch_norms_f16(const void *W16, int64_t D, int64_t M, float *norms, cudaStream_t s);

struct SweepArgs {
    const float *W;
    int64_t D, M;
    const float *norms;
    const int32_t *rowptr;
    const int32_t *colidx;
    int64_t N;
    u64 *state;           // per-document running (distance, index) key
    u64 *state2;          // same for the second-best unit (NULL unless it is wanted)
    uint32_t *status;     // status word (bounds-checked build: violations are recorded here)
    int32_t j_lo, j_hi;   // neuron chunk [j_lo, j_hi)
    int32_t first;        // 1: this chunk initialises the state, 0: merges into it
};
int launch_sweep_direct(const SweepArgs &a, const bmu_opts &o, cudaStream_t s);
int launch_finalize(const u64 *state, const u64 *state2, const int32_t *rowptr, int64_t N,
                    int32_t *out_bmu, float *out_dist, int32_t *out_bmu2, float *out_dist2,
                    cudaStream_t s);
// ---- tiling plan (plan.cu) ---------------------------------------------------
struct PlanLayout {
    size_t perm_off, docoff_off, ngroups_off, bins_off, ids_off, scan_off, scan_bytes, total;
    size_t tilelen_off, tilerows_off, tileoff_off, tilehead_off, tileids_off, tile_rows_cap;
    size_t id_groups_cap;                                                   // 16-byte id groups
    size_t cluster_off, cluster_tmp_off, cluster_tmp_bytes;                 // ordering by content
    size_t rank_off, feat_off, fsort_off, fsort_tmp_off, fsort_tmp_bytes;   // feature ranks
};
static const int TILE_HEAD_ROWS = 32;    // ids below this are swept densely, once per tile
static const int HEAD_ROWS_MAX = 2048;   // widest dense head (the tensor-core sweep's)
// status-word bit set when a scanned offset of the tiling pass exceeds its reserved room
static const uint32_t PLAN_STATUS_OVERFLOW = 64u;
int launch_plan_tiles(const int32_t *rowptr, int64_t N, int interleave, int head, int relabel,
                      int64_t D, char *ws, const PlanLayout &l, uint32_t *status, cudaStream_t s);

// tiled sweep (sweep_tiles.cu): a warp carries 8 documents, 128-neuron slabs
struct TileArgs {
    const float *W;
    int64_t M, N, n_tiles;
    const float *norms;
    const int32_t *perm;
    const uint32_t *tile_len;   // longest | shortest << 16 row of the tile
    const uint32_t *tile_off;   // first row of the tile's id matrix
    const uint4 *tile_ids;      // row r: the r-th id (behind the head) of each of the 8 documents
    const uint32_t *tile_head;  // 8 masks per tile: which of the ids < head_rows a document has
    int32_t head_rows;          // 0 or TILE_HEAD_ROWS
    u64 *state;
    u64 *state2;
    uint32_t *status;           // the sweep does nothing if the tiling pass flagged an overflow
    int64_t D;                  // rows of W, rows of the id matrices: for the bounds-checked build
    size_t tile_rows_cap;
    int32_t j_lo, j_hi, first;
};
int launch_sweep_tiles(const TileArgs &a, const bmu_opts &o, cudaStream_t s);

// tensor-core head + gathered tail (sweep_mma2.cu, sweep_mma2_f16.cu): a block carries 128
// documents through slabs of 256 neurons; launches cover whole multiples of MMA_SLAB neurons
static const int MMA_SLAB = 256;         // granularity of a launch's neuron range (the kernel's slab)
static const int MMA_DOCS = 128;         // documents per block
static const size_t MMA_STAGE_BYTES = 16384;                  // 128 neurons x 64 features x fp16
struct MmaArgs {
    const float *W;
    int64_t M, N, n_tiles;
    const float *norms;
    const int32_t *perm;
    const uint32_t *tile_len;
    const uint32_t *tile_off;
    const uint4 *tile_ids;
    int32_t head;               // features summed on the tensor cores (a multiple of 64)
    const uint32_t *tile_head;  // head / 32 mask words per planned document
    const unsigned char *head_img;  // split head of slab j_lo / 256 onwards (head_image2_bytes)
    const uint32_t *head_max;   // bit pattern of max |W[f][j]| over the head rows
    u64 *state;
    u64 *state2;                // second-best unit (NULL unless wanted)
    uint32_t *status;           // set non-zero if a bounded wait ran out
    int64_t D;                  // rows of W, rows of the id matrices: for the bounds-checked build
    size_t tile_rows_cap;
    int32_t j_lo, j_hi, first;
    int32_t f16;                // W is an fp16 codebook (row pitch 2 * M bytes)
};
// `feat` (may be NULL = identity): the feature whose row of W is head row r
int launch_head_absmax(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                       uint32_t *head_max, cudaStream_t s);
// writes the fp16 (hi, lo) split of the `head` most frequent rows of W, scaled by a power of
// two, as the shared-memory images the sweep copies; whole slabs of [0, m_full) only
size_t head_image2_bytes(int64_t M, int head);
int launch_head_split2(const float *W, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                       uint32_t *head_max, unsigned char *head_img, cudaStream_t s);
int launch_sweep_mma2(const MmaArgs &a, const bmu_opts &o, cudaStream_t s);
int launch_sweep_mma2_f16(const MmaArgs &a, const bmu_opts &o, cudaStream_t s);
int launch_head_split2_f16(const void *W16, int64_t M, int64_t m_full, int head, const uint16_t *feat,
                           unsigned char *head_img, cudaStream_t s);
size_t plan_bytes(int64_t N, int64_t nnz, int head, int64_t D, int cluster, PlanLayout *l);
int launch_plan(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                int order_by_length, int head, int relabel, int64_t D, char *ws, const PlanLayout &l,
                uint32_t *status, cudaStream_t s);

static const int LANES_MAX_D = 65024;    // 16-bit ids with 0xFFFF as the end marker

int launch_wait_timeout_selftest(uint32_t *status, cudaStream_t s);

// planned warp-per-document sweep (sweep_direct.cu): whole slabs of [j_lo, j_hi) only
struct RowsArgs {
    const float *W;
    int64_t M, N;
    const float *norms;
    const int32_t *rowptr;
    const int32_t *perm;
    const uint32_t *doc_off;
    const uint4 *ids;
    u64 *state;
    u64 *state2;          // NULL unless the second-best unit is wanted
    uint32_t *status;     // the sweep does nothing if the tiling pass flagged an overflow
    int64_t D;            // rows of W, 16-byte id groups: for the bounds-checked build
    size_t id_groups_cap;
    int32_t j_lo, j_hi, first;
};
int rows_slab_width(const bmu_opts &o);
int launch_sweep_rows(const RowsArgs &a, const bmu_opts &o, cudaStream_t s);
// same with W pointing at an fp16 codebook (row pitch 2*M bytes), 256-neuron slabs
int launch_sweep_rows_f16(const RowsArgs &a, const bmu_opts &o, cudaStream_t s);

// update step (update.cu): scatter, neighbourhood blur, write-back
int launch_update_scatter(const int32_t *rowptr, const int32_t *colidx, int64_t N,
                          const int32_t *bmu, int64_t M, uint32_t *num, uint32_t *cnt,
                          cudaStream_t s);
int launch_update_blur(const uint32_t *num, const uint32_t *cnt, int64_t D, int32_t edge_x,
                       int32_t edge_y, float sigma, float *num_blur, float *cnt_blur,
                       cudaStream_t s);
size_t map_errors_workspace_bytes();
int launch_map_errors(const int32_t *bmu, const int32_t *bmu2, const float *dist, int64_t N,
                      int32_t edge_x, int32_t adjacency, double *out, void *ws, cudaStream_t s);
int launch_update_writeback(const float *num_blur, const float *cnt_blur, int64_t D, int64_t M,
                            float *W, cudaStream_t s);

// arg-min read-back over a materialised score block (readback.cu)
int launch_readback_argmin(const void *scores, int half, int64_t n_rows, int64_t M,
                           const float *norms, const int32_t *rowptr, int32_t *out_bmu,
                           float *out_dist, cudaStream_t s);

int launch_validate_csr(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                        int64_t D, int32_t *flags, cudaStream_t s);

}  // namespace bmu
