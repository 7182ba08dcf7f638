/*
 * bmu.h -- C ABI of the B200 (sm_100a) best-matching-unit search library.
 *
 * The operation (paper Section 3: the nearest-neuron search of self-organizing
 * map training, with the arg-min taken inside the sparse-dense product so that
 * no document-by-neuron score matrix is ever written): for every document i of
 * a sparse binary corpus and every neuron j of an M-neuron codebook
 *
 *     d_ij = |x_i| + ||w_j||^2 - 2 * sum_{f in x_i} W[f*M + j]
 *
 * and the library returns, per document, the lowest j attaining min_j d_ij and
 * that minimum (the SQUARED distance, not clamped, not rooted).
 *
 * Layouts (all arrays are DEVICE memory unless the name says "host"; the
 * caller owns every buffer it passes and keeps it alive until the stream has
 * finished the call):
 *   W       float32 [D][M], feature-major: the M weights of feature f are
 *           contiguous at W + f*M (the feature-major layout of Section 3).  The fast path needs
 *           W 16-byte aligned and M % 4 == 0; any other M takes a scalar path.
 *   rowptr  int32 [N+1], rowptr[0] == 0, non-decreasing; row i is
 *           colidx[rowptr[i] .. rowptr[i+1])            (CSR of the binary corpus)
 *   colidx  int32 [nnz], feature ids in [0, D); distinct inside a row (a
 *           repeated id is simply added twice and counted twice in |x_i|);
 *           any order inside a row; at most 65535 ids in a row (more is only
 *           possible with repeats; the planned and tile kernels keep row lengths
 *           in 16 bits).
 *   norms   float32 [M], ||w_j||^2.
 *   out_bmu int32 [N], out_dist float32 [N], in the caller's document order.
 * Limits: M < 2^30; N, D < 2^31; nnz < 2^31 per call (int32 rowptr).  Ids out of
 * range, rows of more than 65535 ids and non-finite weights are preconditions
 * that the hot path does not check (bmu_validate_csr checks the first two).  An empty row is legal: its
 * distances are the norms.  N == 0 is legal and does nothing.
 *
 * Every call is asynchronous on `stream` (a cudaStream_t passed as void*, NULL =
 * the legacy default stream) unless stated otherwise, and returns a bmu_status;
 * errors detected at launch time are returned, nothing throws or aborts.
 * bmu_last_error() gives a thread-local detail string for the last failure.
 * There is no CPU fallback: without a CUDA device every compute call returns
 * BMU_ERR_CUDA.
 */
#ifndef BMU_H
#define BMU_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BMU_API __attribute__((visibility("default")))
#else
#define BMU_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BMU_OK = 0,
    BMU_ERR_INVALID_ARG = 1,   /* null pointer, negative size, bad option */
    BMU_ERR_UNSUPPORTED = 2,   /* size beyond a stated limit */
    BMU_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or too small */
    BMU_ERR_CUDA = 4,          /* a CUDA runtime call failed (see bmu_last_error) */
    BMU_ERR_TIMEOUT = 5        /* a bounded device-side wait ran out */
} bmu_status;

/*
 * Tunables of the search (the paper's levers, Section 4: tile size, tile
 * membership, neuron-axis chunking, vector width).  0 in any field = choose
 * automatically.  Unknown combinations return BMU_ERR_INVALID_ARG.
 */
typedef struct bmu_opts {
    int32_t kernel;         /* 0 auto; 1 generic (a warp per document, ids straight from the
                               CSR, any D and M); 3 planned (a warp per document, ids from
                               the tiling pass; needs M % 4 == 0, M >= 32 * vec, D <= 65024);
                               4 tiled (a warp carries 8 documents; frequent rows loaded once
                               per tile; the warps of a block walk the feature axis in step
                               so that L1 serves the rows they share; needs what 3 needs and
                               length-ordered documents); 6 tensor-core head (the sum over
                               the head_rows most frequent features is a dense contraction
                               on tcgen05 tensor cores with fp32 accumulation into
                               double-buffered tensor memory, the remaining ids are gathered
                               as in 4; needs what 4 needs, D >= head_rows and M >= 256; the
                               automatic choice for large sweeps).  Other values are
                               refused. */
    int32_t chunk_neurons;  /* neurons per L2-resident chunk of the codebook (Section 4.2,
                               "neuron-axis chunking"); rounded to the slab width */
    int32_t vec;            /* warp-per-document kernels: floats per lane per row, 4 or 8 */
    int32_t docs_per_warp;  /* generic kernel: documents a warp carries through one slab */
    int32_t warps;          /* warp-per-document kernels: warps per thread block */
    int32_t cluster;        /* tile membership (Section 4.2): 1 order the documents by
                               length before cutting tiles, so that the documents of a tile
                               finish together (0 = 3 for the tensor-core sweep, 1 for the
                               other kernels); 3 by length, and among equally long
                               documents by their two rarest features and their most frequent
                               gathered one, so that documents sharing features fall in the
                               same tile; 4 the same with the three most frequent gathered
                               features as the key (3 and 4: fp32 codebook, and the tensor-core
                               sweep of the half-precision one); 2 keep the corpus order
                               (generic and planned kernels only) */
    int32_t stage_rows;     /* unused, must be 0 */
    int32_t stages;         /* unused, must be 0 */
    int32_t tile_order;     /* order of the gathered ids inside a tile: 1 ascending; 2 dealt
                               alternately from the frequent and the rare half of each list
                               (so that a warp mixes loads that hit L1 with loads that go to
                               L2); 0 = 2 for the tiled kernel, 1 for the tensor-core sweep
                               (its dense head has taken the frequent ids already; ascending
                               measured 0.7 % faster on config 4) */
    int32_t tile_head;      /* tiled kernel: 0 sweep the 32 most frequent features (ids < 32)
                               densely, one load per tile, 1 treat them like all other ids */
    int32_t head_rows;      /* tensor-core sweep: how many of the most frequent features
                               are summed by the tensor cores: a multiple of 64 up to 2048;
                               0 = 640 (half-precision codebook: 576) */
    int32_t repack;         /* tensor-core sweep: 0/1 gather from a compact [D][chunk] copy
                               of the chunk's columns, made before each launch, 2 gather
                               from the codebook itself */
    int32_t relabel;        /* tensor-core sweep: which features form the dense head.
                               1 the head_rows features listed by the most documents of
                               this corpus (ranked inside the tiling pass; the caller's ids
                               stay as they are); 2 the ids below head_rows (a vocabulary
                               already labelled by frequency, as the paper's is, Table 8);
                               0 decide: keep the ids if they cover at least 98 % of what
                               the most frequent features would */
    int32_t reserved[3];    /* must be 0 */
} bmu_opts;

BMU_API const char *bmu_status_string(int status);
BMU_API const char *bmu_last_error(void);

/* Library version as major*10000 + minor*100 + patch. */
BMU_API int bmu_version(void);

/*
 * How many kernels of this library the calling thread has launched so far (the
 * library's own kernels; the sort and scan of the tiling pass, which come from
 * a CUDA library, and memsets are not counted).  The difference across a region
 * is the number of launches in it.
 */
BMU_API uint64_t bmu_kernel_launches(void);

/*
 * What bmu_search_ws would do for a problem of this size with these options on
 * the current device (Section 4: tile, chunking and vector-width choices), without
 * doing it: which kernel (as in bmu_opts.kernel; never 0), the tensor-core head
 * (0 for the other kernels), the neurons a block carries at a time, the documents
 * that share a block, whether a compact copy of the chunk's columns precedes each
 * launch, the neurons per launch (one L2-resident chunk), the number of sweep
 * launches, and how many neurons beyond the last whole slab go to the generic
 * kernel in one more launch.  Assumes W 16-byte aligned.  Same errors as
 * bmu_search_ws for sizes and options it would refuse.
 */
typedef struct bmu_search_desc {
    int32_t kernel, head_rows, slab, docs_per_block, repack, sweep_launches, ragged_neurons;
    int32_t reserved;
    int64_t chunk_neurons;
} bmu_search_desc;
BMU_API int bmu_describe_search(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                const bmu_opts *opts, bmu_search_desc *out);

/*
 * Codebook norms, the "norms" step of an epoch (Table 4): norms[j] = sum_f
 * W[f*M+j]^2.  Products and the running sum are taken in fp64 and rounded to
 * fp32 once.  Deterministic.  Uses no scratch memory.
 */
BMU_API int bmu_codebook_norms(const float *W, int64_t D, int64_t M, float *norms, void *stream);

/*
 * Scratch bytes bmu_search_ws needs for a problem of this size (norms, the
 * per-document running minimum merged across neuron chunks, the tiling plan,
 * the split image of the frequent rows (4 * head_rows bytes per neuron) and the
 * compact chunk copy of the tensor-core sweep).  `nnz` is the length of colidx.
 */
BMU_API size_t bmu_search_workspace_bytes(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                  const bmu_opts *opts);

/*
 * The whole search (norms -> tiling -> gather-accumulate sweep over neuron
 * chunks with the argmin fused in -> outputs in document order; Section 3 and
 * Section 4) with caller-supplied scratch.  `norms` may be NULL (computed into
 * the workspace) or a device array from bmu_codebook_norms.  `workspace` must be
 * 256-byte aligned device memory of at least bmu_search_workspace_bytes(...)
 * bytes; its contents are undefined afterwards, except that its first 32-bit
 * word is a status word: 0 after a clean run, non-zero if a bounded device-side
 * wait of the tensor-core sweep ran out or a size check of the tiling pass
 * failed (results are then invalid).  Allocates nothing.  Calls that share a workspace must not overlap on the GPU.
 */
BMU_API int bmu_search_ws(const float *W, int64_t D, int64_t M, const float *norms,
                  const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                  int32_t *out_bmu, float *out_dist, const bmu_opts *opts,
                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * Reusable tiling plan.  The paper's epochs run over a frozen, pre-ordered corpus
 * (Section 5: the corpus is clustered once, offline; Section 4.2, tile
 * membership), so the document-tiling pass -- ordering, id re-packing, tile
 * matrices, head masks -- can be done once and reused by every epoch's search.
 *   bmu_plan_workspace_bytes  bytes of 256-byte aligned device memory a plan needs
 *       (the plan itself plus the scratch of the searches that use it).
 *   bmu_plan_create  runs the tiling pass into `workspace` on `stream`, waits for
 *       it, checks its status word (BMU_ERR_WORKSPACE if a size check of the pass
 *       failed) and returns a host handle in *plan.  rowptr, colidx and the
 *       workspace stay owned by the caller and must stay alive and unchanged
 *       until bmu_plan_destroy; `nnz` is the length of colidx.
 *   bmu_search_planned  the search of bmu_search_ws without its tiling pass:
 *       norms (NULL = computed), sweep, outputs.  W must be 16-byte aligned.
 *       Allocates nothing, asynchronous on `stream`; searches that share a plan
 *       must not overlap on the GPU.  Results equal bmu_search_ws with the same
 *       options bit for bit.
 *   bmu_plan_order  copies the order the tiling pass put the documents in
 *       (Section 4.2, tile membership) to out_order[N], device memory: the
 *       document at planned position p is out_order[p]; consecutive positions
 *       form the tiles (8) and blocks (128) of the tiled and tensor-core sweeps.
 *       For inspection and measurement (tile reuse); the searches do not need it.
 *       BMU_ERR_UNSUPPORTED for the generic kernel, which plans nothing.
 *   bmu_plan_destroy  frees the host handle (not the workspace).
 */
typedef struct bmu_plan bmu_plan;
BMU_API size_t bmu_plan_workspace_bytes(int64_t N, int64_t nnz, int64_t D, int64_t M,
                                        const bmu_opts *opts);
BMU_API int bmu_plan_create(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                            int64_t D, int64_t M, const bmu_opts *opts, void *workspace,
                            size_t workspace_bytes, bmu_plan **plan, void *stream);
BMU_API int bmu_search_planned(const bmu_plan *plan, const float *W, const float *norms,
                               int32_t *out_bmu, float *out_dist, void *stream);
BMU_API int bmu_plan_order(const bmu_plan *plan, int32_t *out_order, void *stream);
BMU_API void bmu_plan_destroy(bmu_plan *plan);

/*
 * The same search that also returns the second-best unit, which the paper's
 * kernel tracks because topographic error -- gated on by its stopping rules --
 * needs it (Table 5, "bmu1-only").  out_bmu2[i] is the lowest index j !=
 * out_bmu[i] attaining the second-smallest distance, out_dist2[i] that distance
 * (-1 and +inf when M == 1).  Same tie rule, same options, workspace of bmu_search_top2_workspace_bytes(...).
 */
BMU_API size_t bmu_search_top2_workspace_bytes(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                               const bmu_opts *opts);
BMU_API int bmu_search_top2_ws(const float *W, int64_t D, int64_t M, const float *norms,
                               const int32_t *rowptr, const int32_t *colidx, int64_t N,
                               int64_t nnz, int32_t *out_bmu, float *out_dist,
                               int32_t *out_bmu2, float *out_dist2, const bmu_opts *opts,
                               void *workspace, size_t workspace_bytes, void *stream);

/*
 * Half-precision codebook, the paper's own storage (Section 4.2 counts its
 * working set at 2 bytes per weight; Section 4.3 loads pairs of halves).  W16 is IEEE fp16
 * [D][M], feature-major, 16-byte aligned; sums and distances are still fp32
 * (norms: fp64 accumulate).  Needs M % 256 == 0 (M % 8 == 0 for the norms
 * alone) and D <= 65024.  out_bmu2 / out_dist2 may both be NULL, or both given
 * to get the second-best unit as in bmu_search_top2_ws.  bmu_opts.kernel: 3 the
 * planned kernel, 6 the wide tensor-core sweep (needs D >=
 * head_rows; the weights being fp16 already, its head image has one part), 0
 * the tensor-core sweep for large sweeps, else the planned kernel; head_rows
 * defaults to 576 here.  Workspace: bmu_search_f16_workspace_bytes(...) with the
 * same sizes and options (enough with or without the second-best outputs).
 */
BMU_API size_t bmu_search_f16_workspace_bytes(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                              const bmu_opts *opts);
BMU_API int bmu_codebook_norms_f16(const void *W16, int64_t D, int64_t M, float *norms,
                                   void *stream);
BMU_API int bmu_search_f16_ws(const void *W16, int64_t D, int64_t M, const float *norms,
                              const int32_t *rowptr, const int32_t *colidx, int64_t N,
                              int64_t nnz, int32_t *out_bmu, float *out_dist, int32_t *out_bmu2,
                              float *out_dist2, const bmu_opts *opts, void *workspace,
                              size_t workspace_bytes, void *stream);

/*
 * One-shot form.  Same as bmu_search_ws with norms == NULL and default options,
 * but the scratch is a library-owned buffer per device that only ever grows
 * (cudaMalloc on first use or growth; freed by bmu_release_scratch or at
 * process exit).  Reads rowptr[N] back to size the scratch, so the call
 * synchronises the stream once before the kernels are queued.  Calls on
 * different streams of one device share the scratch and must not overlap.
 * The status word of the search (see bmu_search_ws) sits in that scratch:
 * bmu_last_status reads it.
 */
BMU_API int bmu_search(const float *W, int64_t D, int64_t M, const int32_t *rowptr,
               const int32_t *colidx, int64_t N, int32_t *out_bmu, float *out_dist,
               void *stream);

/*
 * What a status word (the first 32-bit word of a search workspace, read back by the
 * caller after the stream has finished) means: BMU_OK for 0, BMU_ERR_WORKSPACE if
 * a size check of the tiling pass failed (bit 64), BMU_ERR_TIMEOUT if a bounded
 * device-side wait ran out (any other bit; bit 128 is set by the bounds-checked
 * build for an address it refused).  The detail string names the word.  Host-side only.
 */
BMU_API int bmu_status_of_word(uint32_t status_word);

/*
 * Status word of the last bmu_search (or bmu_search_host, bmu_search_batches_host)
 * on the current device: synchronises `stream`, copies the word to *out_status and
 * returns BMU_OK if it is 0, BMU_ERR_TIMEOUT if a bounded device-side wait ran
 * out, BMU_ERR_WORKSPACE if a size check of the tiling pass failed (the results
 * of that search are then invalid).  0 if no search has run yet.
 */
BMU_API int bmu_last_status(uint32_t *out_status, void *stream);

/*
 * End-to-end form for a corpus batch that lives in HOST memory (pinned for
 * full copy speed): copies rowptr_host[N+1] and colidx_host[nnz] to the device,
 * runs bmu_search against the device-resident codebook W, and copies the N
 * results back into out_bmu_host / out_dist_host.  Synchronous: returns when
 * the results are in host memory.  Device staging buffers come from the same
 * grow-only library scratch as bmu_search.
 */
BMU_API int bmu_search_host(const float *W, int64_t D, int64_t M, const int32_t *rowptr_host,
                    const int32_t *colidx_host, int64_t N, int32_t *out_bmu_host,
                    float *out_dist_host, void *stream);

/*
 * A corpus streamed in batches from HOST memory against one device-resident
 * codebook (the corpus-scale epoch is fed this way: one CSR per batch, because a
 * whole corpus exceeds the int32 row pointers).  The norms are computed once;
 * the status words of all batches are collected and checked at the end
 * (BMU_ERR_TIMEOUT / BMU_ERR_WORKSPACE as in bmu_last_status);
 * two device staging buffers let a copy stream upload batch k+1 and download the
 * results of batch k-1 while `stream` searches batch k.  Arrays of n_batches
 * host pointers: rowptr_host[k] has N[k]+1 entries, colidx_host[k] has
 * rowptr_host[k][N[k]], out_*_host[k] have N[k]; pinned memory lets the copies
 * overlap.  Synchronous: returns when every result is in host memory.  Staging
 * comes from the grow-only library scratch (sized for the largest batch).
 */
BMU_API int bmu_search_batches_host(const float *W, int64_t D, int64_t M, int32_t n_batches,
                                    const int32_t *const *rowptr_host,
                                    const int32_t *const *colidx_host, const int64_t *N,
                                    int32_t *const *out_bmu_host, float *const *out_dist_host,
                                    void *stream);

/*
 * Self-test of the failure path of device-side waits.  The tensor-core sweep's
 * producer, MMA issuer and tail warps wait on shared-memory barriers; every such wait has an
 * iteration limit, after which the kernel records a status word and returns
 * instead of trapping or spinning forever.  This call runs a one-block kernel
 * that waits (limit: 4096 polls) on a barrier nothing ever arrives on and hands
 * the outcome back the way bmu_search_host does: it returns BMU_ERR_TIMEOUT, and
 * the CUDA context stays usable.  Synchronises the stream.
 */
BMU_API int bmu_selftest_wait_timeout(void *stream);

/* Frees the library-owned scratch of the current device (synchronises it). */
BMU_API int bmu_release_scratch(void);

/*
 * Checks the CSR preconditions on the device: rowptr[0] == 0, rowptr
 * non-decreasing, rowptr[N] == nnz, 0 <= colidx < D, no row of more than 65535
 * ids.  Synchronises the stream.
 * Returns BMU_ERR_INVALID_ARG (detail in bmu_last_error) when one fails.
 */
BMU_API int bmu_validate_csr(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                     int64_t D, void *stream);

/*
 * Search for callers that must not allocate.  (The paper has no counterpart:
 * this entry point exists for integration, not for the method.)  Some hosts of
 * this library cannot call cudaMalloc at the point where they need a search --
 * code running inside a memory pool that owns the whole device, a real-time
 * loop that forbids allocation after start-up, a plug-in that is only handed
 * its inputs and outputs.  bmu_search_ws already allocates nothing but wants a
 * workspace from the caller; this form needs none: its scratch (the codebook
 * norms and the per-document running minimum that is merged across neuron
 * chunks) lives in a fixed 8 MiB array that is part of the library image, so
 * every GPU that loads the library carries those 8 MiB until the process ends.
 * It runs the generic warp-per-document kernel (bmu_opts.kernel == 1) and gives
 * the same results as bmu_search_ws with that option.
 *   Limit: 256 + roundup256(4*M) + roundup256(8*N) <= 8 MiB, else
 *   BMU_ERR_UNSUPPORTED with the sizes in bmu_last_error().  For example
 *   M = 262144 leaves room for about 917,000 documents per call; split larger
 *   batches.
 *   First call on a device: looks up the device address of the array (once per
 *   device, with that device current) -- make that first call outside any
 *   stream capture.  No call ever invokes cudaMalloc, cudaFree or an allocating
 *   library routine.
 *   The array is shared by every call on the device and keeps what the last
 *   call left in it; the entry point re-initialises what it reads, so stale
 *   contents are harmless, but two calls that overlap on the GPU (different
 *   streams, or another thread) race on it and corrupt each other's results.
 * `nnz` is the length of colidx.  Asynchronous on `stream` like bmu_search_ws.
 */
BMU_API int bmu_search_static(const float *W, int64_t D, int64_t M, const int32_t *rowptr,
                              const int32_t *colidx, int64_t N, int64_t nnz, int32_t *out_bmu,
                              float *out_dist, void *stream);

/*
 * The rest of a batch epoch after the search (Table 4 columns "scatter", "blur",
 * "write-back"; Section 6 gives their cost: the scatter grows with the listings,
 * N times nnz per document, the blur with the map size M).  The paper times these steps and prints no formula;
 * they are the textbook batch update of a self-organizing map on a rectangular,
 * non-periodic map of edge_y rows by edge_x columns, neuron j = y * edge_x + x.
 * All arrays are device memory, feature-major like W; every call is
 * asynchronous on `stream` and uses no scratch.
 *
 * bmu_update_scatter: for every document i, cnt[bmu[i]] += 1 and, for every
 *   listed feature f, num[f*M + bmu[i]] += 1 (a repeated id counts twice).
 *   num uint32 [D][M] and cnt uint32 [M] are accumulated into: zero them at the
 *   start of an epoch, call once per corpus batch.  Exact integer counters.
 *   bmu[i] must lie in [0, M) (unchecked, like colidx).
 * bmu_update_blur: num_blur[f][j] = sum_k h(j, k) * num[f][k] and cnt_blur[j] =
 *   sum_k h(j, k) * cnt[k] in fp32, h(j, k) = exp(-(dx^2 + dy^2) / (2 sigma^2))
 *   for |dx|, |dy| <= ceil(3 sigma) and 0 beyond (no wrap-around, no
 *   normalisation: the write-back divides it out); sigma == 0 copies.  Limits:
 *   sigma <= 8, D <= 65024.  Outputs must not alias inputs.
 * bmu_update_writeback: W[f*M + j] = num_blur[f*M + j] / cnt_blur[j] where
 *   cnt_blur[j] > 0; other neurons keep their weights.  D <= 65535.
 * The norms of the new codebook are bmu_codebook_norms.
 */
BMU_API int bmu_update_scatter(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                               const int32_t *bmu, int64_t D, int64_t M, uint32_t *num,
                               uint32_t *cnt, void *stream);
BMU_API int bmu_update_blur(const uint32_t *num, const uint32_t *cnt, int64_t D, int32_t edge_x,
                            int32_t edge_y, float sigma, float *num_blur, float *cnt_blur,
                            void *stream);
BMU_API int bmu_update_writeback(const float *num_blur, const float *cnt_blur, int64_t D, int64_t M,
                                 float *W, void *stream);

/*
 * Stopping metrics of an epoch (Table 4 column "stopping metric"; Section 5: the
 * second-best unit feeds the topographic error, which the stopping rules gate on
 * together with the quantisation error).  The paper names the measures and
 * prints no formula; these are the textbook definitions over the outputs of
 * bmu_search_top2_ws for a batch of (held-out) documents, on the map of edge_y
 * rows by edge_x columns (neuron j = y * edge_x + x):
 *   out[0] = mean of dist[i]               (mean squared quantisation error)
 *   out[1] = mean of sqrt(max(dist[i], 0)) (quantisation error)
 *   out[2] = fraction of documents whose bmu[i] and bmu2[i] are not neighbours
 *            (topographic error): adjacency 4 = the units share an edge, 8 = an
 *            edge or a corner; bmu2[i] < 0 (one-neuron map) is not an error.
 * bmu, bmu2 int32[N], dist fp32[N], out double[3]: device memory.  Sums are
 * fp64 in a fixed order (same bits on every call).  N == 0 gives zeros.
 * workspace: bmu_map_errors_workspace_bytes() bytes of device memory, 256-byte
 * aligned, contents irrelevant.  Asynchronous on `stream`; BMU_ERR_INVALID_ARG for
 * an adjacency other than 4 or 8, edges < 1 or null pointers.
 */
BMU_API size_t bmu_map_errors_workspace_bytes(void);
BMU_API int bmu_map_errors(const int32_t *bmu, const int32_t *bmu2, const float *dist, int64_t N,
                           int32_t edge_x, int32_t edge_y, int32_t adjacency, double *out,
                           void *workspace, size_t workspace_bytes, void *stream);

/*
 * Arg-min read-back over a MATERIALISED score block: the second half of the other
 * route to the same search (Section 3: a sparse-dense product writes all
 * n_rows x M scores s_ij = sum_{f in x_i} W[f][j], a separate pass reads them
 * back; Section 4.4 tunes that pass to a warp per row with vector loads).  Not
 * used by bmu_search; it is here so that the fused search can be compared with a
 * tuned version of that route.  scores: n_rows x M, row-major, fp32 (half == 0)
 * or IEEE fp16 (half != 0), 16-byte aligned, M % 4 == 0 (fp16: M % 8 == 0);
 * rowptr: the n_rows + 1 row pointers of these documents (only differences are
 * used, for |x_i|).  out_bmu[i] = lowest j attaining min_j (norms[j] - 2 s_ij),
 * out_dist[i] = |x_i| + that minimum.  Reads the block once; no scratch.
 */
BMU_API int bmu_score_block_argmin(const void *scores, int32_t half, int64_t n_rows, int64_t M,
                                   const float *norms, const int32_t *rowptr, int32_t *out_bmu,
                                   float *out_dist, void *stream);

/*
 * Measures one on-chip ceiling of the current device with a microbenchmark, so
 * that achieved throughput can be quoted against the roof that binds (the paper
 * quotes its kernel against the L2 roof of its card, Section 6 / Table 3).
 *   which 0  L2 -> SM read bandwidth, 128-bit loads bypassing L1      [bytes/s]
 *         1  L2 -> shared memory by bulk asynchronous copies of `piece` bytes
 *            (multiple of 16, <= 24576)                                [bytes/s]
 *         2  shared memory -> registers, conflict-free 128-bit loads   [bytes/s]
 *         3  L1-resident global loads -> registers, 128-bit            [bytes/s]
 *         4  fp32 adds, scalar instructions                            [adds/s]
 *         5  fp32 adds, packed two-wide instructions                   [adds/s]
 *         6  L2 -> SM by 128-bit loads and bulk copies of `piece` bytes (multiple
 *            of 16 in [256, 16384]; up to sixteen issuing threads per block, as many
 *            as 64 KB of buffers allow) running together, both counted: the way the
 *            tensor-core sweep pulls bytes (gathered rows by loads, head image by
 *            bulk copies)                                              [bytes/s]
 * `buffer` is 256-byte aligned device memory the benchmark may overwrite; for
 * 0, 1 and 6 its size is the footprint that is swept (keep it well inside L2), for
 * 3 it must hold 64 KiB per SM.  Synchronous; the result goes to *out_value.
 */
BMU_API int bmu_measure_roof(int which, void *buffer, size_t buffer_bytes, int piece,
                             double *out_value, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* BMU_H */
