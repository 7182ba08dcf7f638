// Host side of the C ABI: argument checks, workspace layout, neuron-axis
// chunking (Section 4.2) and the order in which the kernels are queued.
#include "common.cuh"

#include <stdarg.h>
#include <string.h>

#include <mutex>
#include <new>

namespace bmu {

static thread_local char g_err[512] = "";
thread_local unsigned long long g_kernel_launches = 0;

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char *what)
{
    set_error("%s: %s", what, cudaGetErrorString(e));
    return BMU_ERR_CUDA;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static const int64_t MAX_M = (int64_t)1 << 30;   // row pitch M*4 must fit 32 bits
static const int64_t MAX_I32 = 0x7fffffff;

// ---- workspace layout -----------------------------------------------------
struct Layout {
    size_t status_off, norms_off, state_off, state2_off, head_off, repack_off, plan_off, total;
    PlanLayout plan;
};

// Neurons per launch of the tensor-core sweep: whole 256-neuron slabs whose rows take about
// 0.4 of L2 (768 neurons at D = 16384 on a 126 MB L2).  Measured on config 4: 768 beats 1024 by
// 2 % and 512 by 3 %; at 1024 the chunk (67 MB) no longer stays resident in the two-part L2 and
// its rows are fetched from DRAM five times over.
static int64_t mma_auto_chunk(int64_t D, int64_t M)
{
    int dev = 0, l2 = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess || l2 <= 0)
        l2 = 64 << 20;
    int64_t c = (int64_t)((double)l2 * 0.42) / (D * 4) / MMA_SLAB * MMA_SLAB;
    if (c < MMA_SLAB) c = MMA_SLAB;
    if (c > M) c = M / MMA_SLAB * MMA_SLAB;
    return c;
}

static int64_t mma_chunk(const bmu_opts &o, int64_t D, int64_t M)
{
    return o.chunk_neurons ? ((int64_t)o.chunk_neurons + MMA_SLAB - 1) / MMA_SLAB * MMA_SLAB
                           : mma_auto_chunk(D, M);
}

// Bytes of the compact chunk copy: unless told otherwise the tensor-core sweeps gather from a
// [D][chunk] copy of the chunk's columns (4 KB row pitch at a chunk of 1024), made before each
// launch, instead of from the codebook itself (row pitch 4 * M bytes), so that the rows of a
// chunk share pages: 2-7 % faster on every benchmark shape for 0.2 % more traffic.
static size_t mma_repack_bytes(const bmu_opts &o, int64_t D, int64_t M, int64_t N, int64_t nnz,
                               bool top2)
{
    if (o.repack == 2 || (o.kernel != 0 && o.kernel != 6)) return 0;
    if (D > LANES_MAX_D || M < MMA_SLAB) return 0;
    const int64_t chunk = mma_chunk(o, D, M);
    if (M <= chunk) return 0;                      // one launch: the codebook is the chunk
    (void)N; (void)nnz;
    return (size_t)D * (size_t)(chunk < M ? chunk : M) * sizeof(float);
}

// one block per codebook row: `width_bytes` (a multiple of 16) from byte `off_bytes` of the row
__global__ void __launch_bounds__(256)
repack_chunk_kernel(const char *__restrict__ W, int64_t pitch_bytes, int64_t off_bytes,
                    int32_t width_bytes, char *__restrict__ out)
{
    const uint4 *src = reinterpret_cast<const uint4 *>(W + (int64_t)blockIdx.x * pitch_bytes + off_bytes);
    uint4 *dst = reinterpret_cast<uint4 *>(out + (int64_t)blockIdx.x * width_bytes);
    for (int i = threadIdx.x; i < width_bytes / 16; i += 256) dst[i] = __ldcs(src + i);
}

// Features summed on the tensor cores: 640 (measured best of 512 .. 1024 on configs 2-5 in
// full-length runs, where the board sits at its power cap: 768 wins short runs at boost clocks
// and loses 1-2 % once the cap binds), less if the vocabulary is smaller.
static int mma_head_rows(const bmu_opts &o, int64_t D)
{
    if (o.head_rows) return o.head_rows;
    const int64_t cap = D / 64 * 64, want = 640;
    return (int)(cap < want ? (cap < 64 ? 64 : cap) : want);
}

static Layout layout_for(int64_t D, int64_t M, int64_t N, int64_t nnz, int kernel,
                         bool top2 = false, int head = 640, size_t repack_bytes = 0, int cluster = 0)
{
    Layout l;
    size_t off = 0;
    l.status_off = off; off = 256;
    l.norms_off = off; off = align_up(off + (size_t)M * sizeof(float), 256);
    l.state_off = off; off = align_up(off + (size_t)N * sizeof(u64), 256);
    l.state2_off = off;
    if (top2) off = align_up(off + (size_t)N * sizeof(u64), 256);
    // split image of the frequent rows for the tensor-core sweep (it may be the automatic choice)
    l.head_off = off;
    if ((kernel == 0 || kernel == 6) && D >= head && D <= LANES_MAX_D && M >= MMA_SLAB)
        off = align_up(off + head_image2_bytes(M, head), 256);
    l.repack_off = off;                  // compact copy of the codebook chunk being swept
    off = align_up(off + repack_bytes, 256);
    l.plan_off = off;
    memset(&l.plan, 0, sizeof(l.plan));
    if (kernel != 1 && D <= LANES_MAX_D) off += plan_bytes(N, nnz, head, D, cluster, &l.plan);
    l.total = off;
    return l;
}

// How the tiling pass orders the documents: 0 corpus order, 1 by length, 3 / 4 by length and
// content.  The tensor-core sweep takes 3 unless told otherwise (measured on configs 2-4: 0.5,
// 2.8 and 2.5 % faster than by length alone, the extra sort included; 4 gains less).
static int plan_order(const bmu_opts &o, bool tensor_core_sweep)
{
    if (o.cluster == 2) return 0;
    if (o.cluster >= 3) return o.cluster;
    return (o.cluster == 0 && tensor_core_sweep) ? 3 : 1;
}

// the layout search_impl uses for these options (the workspace-size queries must agree with it)
static Layout layout_of(const bmu_opts &o, int64_t D, int64_t M, int64_t N, int64_t nnz, bool top2)
{
    return layout_for(D, M, N, nnz, o.kernel, top2, mma_head_rows(o, D),
                      mma_repack_bytes(o, D, M, N, nnz, top2), plan_order(o, true));
}

static int check_sizes(int64_t D, int64_t M, int64_t N, int64_t nnz)
{
    if (D < 0 || M < 0 || N < 0 || nnz < 0) {
        set_error("negative size (D=%lld M=%lld N=%lld nnz=%lld)", (long long)D, (long long)M,
                  (long long)N, (long long)nnz);
        return BMU_ERR_INVALID_ARG;
    }
    if (M >= MAX_M || D > MAX_I32 || N >= MAX_I32 || nnz > MAX_I32) {
        set_error("size beyond the limits (M < 2^30; D, N, nnz < 2^31)");
        return BMU_ERR_UNSUPPORTED;
    }
    return BMU_OK;
}

static int check_opts(const bmu_opts &o)
{
    if (o.tile_order < 0 || o.tile_order > 2) { set_error("bmu_opts.tile_order must be 0, 1 or 2"); return BMU_ERR_INVALID_ARG; }
    if (o.tile_head < 0 || o.tile_head > 1) { set_error("bmu_opts.tile_head must be 0 or 1"); return BMU_ERR_INVALID_ARG; }
    if (o.head_rows < 0 || o.head_rows > HEAD_ROWS_MAX || o.head_rows % 64 != 0) {
        set_error("bmu_opts.head_rows must be 0 or a multiple of 64 up to %d", HEAD_ROWS_MAX);
        return BMU_ERR_INVALID_ARG;
    }
    if (o.repack < 0 || o.repack > 2) { set_error("bmu_opts.repack must be 0, 1 or 2"); return BMU_ERR_INVALID_ARG; }
    if (o.relabel < 0 || o.relabel > 2) { set_error("bmu_opts.relabel must be 0, 1 or 2"); return BMU_ERR_INVALID_ARG; }
    for (int i = 0; i < 3; ++i)
        if (o.reserved[i] != 0) { set_error("bmu_opts.reserved must be zero"); return BMU_ERR_INVALID_ARG; }
    if (o.kernel != 0 && o.kernel != 1 && o.kernel != 3 && o.kernel != 4 && o.kernel != 6) {
        set_error("bmu_opts.kernel must be 0, 1, 3, 4 or 6");
        return BMU_ERR_INVALID_ARG;
    }
    if (o.stage_rows != 0 || o.stages != 0) {
        set_error("bmu_opts.stage_rows and bmu_opts.stages must be zero");
        return BMU_ERR_INVALID_ARG;
    }
    if (o.cluster < 0 || o.cluster > 4) { set_error("bmu_opts.cluster must be 0 .. 4"); return BMU_ERR_INVALID_ARG; }
    if (o.chunk_neurons < 0) { set_error("bmu_opts.chunk_neurons < 0"); return BMU_ERR_INVALID_ARG; }
    if (o.vec != 0 && o.vec != 4 && o.vec != 8) { set_error("bmu_opts.vec must be 0, 4 or 8"); return BMU_ERR_INVALID_ARG; }
    return BMU_OK;
}

// Neurons per L2-resident chunk: the chunk's share of the codebook,
// D * chunk * 4 bytes, is kept to about half of L2 so that the rows of one
// chunk stay cached while every document passes over them.
static int64_t auto_chunk(int64_t D, int64_t M, int slab)
{
    int dev = 0, l2 = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess || l2 <= 0)
        l2 = 64 << 20;
    int64_t c = D > 0 ? ((int64_t)l2 / 2) / (D * 4) : M;
    c = c / slab * slab;
    if (c < slab) c = slab;
    if (c > M) c = (M + slab - 1) / slab * slab;
    return c;
}

// Which kernel a search takes and how it is cut into launches.
struct Route {
    int kernel;            // 1 generic, 3 planned, 4 tiled, 6 tensor-core head + gathered tail
    int head;              // features summed on the tensor cores (kernel 6), else 0
    int slab;              // neurons a block (or warp) carries at a time
    int docs_per_block;    // documents that share a block
    int64_t chunk;         // neurons per launch (one L2-resident chunk)
    int64_t m_full;        // neurons covered by whole slabs; the rest takes the generic kernel
    int repack;            // 1: a compact copy of the chunk's columns precedes each launch
};

static int route_search(const bmu_opts &o, int64_t D, int64_t M, int64_t nnz, uintptr_t w_addr,
                        Route &r)
{
    const int head = mma_head_rows(o, D);
    // the planned warp-per-document kernel needs 16-bit ids and whole 16-byte row pieces
    const bool planned_ok = D <= LANES_MAX_D && M % 4 == 0 && M >= rows_slab_width(o) &&
                            (w_addr & 15) == 0;
    if (o.kernel == 3 && !planned_ok) {
        set_error("planned kernel needs M %% 4 == 0, M >= 128, D <= %d and W 16-byte aligned",
                  LANES_MAX_D);
        return BMU_ERR_UNSUPPORTED;
    }
    const bool tiled_ok = planned_ok && M >= 128 && o.cluster != 2;
    // tensor-core head: additionally at least one whole 256-neuron slab and `head` features
    const bool mma_ok = tiled_ok && D >= head && M >= MMA_SLAB;
    if (o.kernel == 6 && !mma_ok) {
        set_error("tensor-core sweep needs what the tiled kernel needs, D >= %d and M >= %d",
                  head, MMA_SLAB);
        return BMU_ERR_UNSUPPORTED;
    }
    // automatic choice for large sweeps: the tensor-core sweep where it applies, else the tiled
    // kernel; both repay their extra preparation only when there is enough to sweep
    const bool big = (double)nnz * (double)M >= 2e10;
    const bool mma = o.kernel == 6 || (o.kernel == 0 && mma_ok && big);
    const bool tiled = !mma && (o.kernel == 4 || (o.kernel == 0 && tiled_ok && big));
    if (tiled && !tiled_ok) {
        set_error("tiled kernel needs M %% 4 == 0, M >= 128, D <= %d, W 16-byte aligned and "
                  "length-ordered documents (cluster != 2)", LANES_MAX_D);
        return BMU_ERR_UNSUPPORTED;
    }
    const bool planned = !tiled && !mma && (o.kernel == 3 || (o.kernel == 0 && planned_ok));
    r.head = 0; r.repack = 0;
    if (mma) {
        r.kernel = 6; r.head = head; r.slab = 256; r.docs_per_block = MMA_DOCS;
        r.chunk = mma_chunk(o, D, M);
        r.m_full = M / MMA_SLAB * MMA_SLAB;
        r.repack = o.repack != 2 && M > r.chunk;
    } else if (tiled) {
        r.kernel = 4; r.slab = 128; r.docs_per_block = 8 * (o.warps ? o.warps : 4);
        r.chunk = o.chunk_neurons ? (o.chunk_neurons + 127) / 128 * 128 : auto_chunk(D, M, 128);
        r.m_full = M / 128 * 128;
    } else if (planned) {
        r.kernel = 3; r.slab = rows_slab_width(o); r.docs_per_block = o.warps ? o.warps : 16;
        r.chunk = o.chunk_neurons ? (o.chunk_neurons + r.slab - 1) / r.slab * r.slab
                                  : auto_chunk(D, M, r.slab);
        r.m_full = M / r.slab * r.slab;
    } else {
        r.kernel = 1; r.slab = 32 * (o.vec ? o.vec : 4);
        r.docs_per_block = (o.warps ? o.warps : 16) * (o.docs_per_warp ? o.docs_per_warp : 4);
        r.chunk = o.chunk_neurons ? (o.chunk_neurons + r.slab - 1) / r.slab * r.slab
                                  : auto_chunk(D, M, r.slab);
        r.m_full = M;
    }
    return BMU_OK;
}

// Cuts [0, m_full) into the launches of the tensor-core sweep: as many as chunks of `chunk`
// neurons need, the 256-neuron slabs dealt evenly among them (so that the last launch is not a
// single slab whose MMAs nothing overlaps).  Launch k covers [cut(k), cut(k + 1)).
struct LaunchCuts {
    int64_t slabs, n, base, rem;
    LaunchCuts(int64_t m_full, int64_t chunk)
    {
        slabs = m_full / MMA_SLAB;
        n = (m_full + chunk - 1) / chunk;
        base = n ? slabs / n : 0;
        rem = n ? slabs % n : 0;
    }
    int64_t cut(int64_t k) const { return (k * base + (k < rem ? k : rem)) * MMA_SLAB; }
};

static int search_impl(const float *W, int64_t D, int64_t M, const float *norms,
                       const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                       int32_t *out_bmu, float *out_dist, const bmu_opts *opts_in, void *ws,
                       size_t ws_bytes, cudaStream_t s, int32_t *out_bmu2 = nullptr,
                       float *out_dist2 = nullptr, int phase = 0)
{
    // phase 0: the whole search; 1: only the tiling pass (bmu_plan_create); 2: everything but
    // the tiling pass, whose results are still in the workspace (bmu_search_planned)
    const bool top2 = out_bmu2 != nullptr || out_dist2 != nullptr;
    int rc = check_sizes(D, M, N, nnz);
    if (rc) return rc;
    bmu_opts o;
    memset(&o, 0, sizeof(o));
    if (opts_in) o = *opts_in;
    if ((rc = check_opts(o))) return rc;
    if (N == 0) return BMU_OK;
    if (!rowptr || (nnz > 0 && !colidx) ||
        (phase != 1 && (!W || !out_bmu || !out_dist || (top2 && (!out_bmu2 || !out_dist2))))) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    // a plan is made before the codebook is known: it assumes the aligned fast path, and the
    // search that uses it insists on it
    const uintptr_t w_addr = phase == 1 ? 0 : reinterpret_cast<uintptr_t>(W);
    if (phase == 2 && (w_addr & 15) != 0) {
        set_error("a planned search needs W 16-byte aligned");
        return BMU_ERR_UNSUPPORTED;
    }
    if (M == 0 || D == 0) {
        set_error("empty codebook (D=%lld, M=%lld): no neuron to return", (long long)D, (long long)M);
        return BMU_ERR_INVALID_ARG;
    }
    const int head = mma_head_rows(o, D);
    const size_t repack_bytes = mma_repack_bytes(o, D, M, N, nnz, top2);
    const Layout l = layout_of(o, D, M, N, nnz, top2);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < l.total) {
        set_error("workspace missing, not 256-byte aligned, or smaller than %zu bytes", l.total);
        return BMU_ERR_WORKSPACE;
    }
    char *base = static_cast<char *>(ws);
    u64 *state = reinterpret_cast<u64 *>(base + l.state_off);
    u64 *state2 = top2 ? reinterpret_cast<u64 *>(base + l.state2_off) : nullptr;
    if (!norms && phase != 1) {
        float *n = reinterpret_cast<float *>(base + l.norms_off);
        if ((rc = launch_norms(W, D, M, n, s))) return rc;
        norms = n;
    }
    uint32_t *status = reinterpret_cast<uint32_t *>(base + l.status_off);
    BMU_CUDA(cudaMemsetAsync(status, 0, 256, s));
    Route r;
    if ((rc = route_search(o, D, M, nnz, w_addr, r))) return rc;
    const bool mma = r.kernel == 6, tiled = r.kernel == 4, planned = r.kernel == 3;
    char *pw = base + l.plan_off;
    // dense head = the most frequent features by the corpus's own counts (bmu_opts.relabel)
    const int relabel = mma ? o.relabel : 2;        // 0 decide from the counts, 1 always, 2 never
    if ((planned || tiled || mma) && phase != 2)
        if ((rc = launch_plan(rowptr, colidx, N, nnz, plan_order(o, mma),
                              mma ? head : 0, relabel, D, pw, l.plan, status, s)))
            return rc;
    if (mma) {
        if (phase != 2 &&
            (rc = launch_plan_tiles(rowptr, N, o.tile_order == 2, head, relabel, D, pw, l.plan, status, s)))
            return rc;
        if (phase == 1) return BMU_OK;
        const int64_t m_full = r.m_full;
        uint32_t *head_max = status + 16;
        unsigned char *img = reinterpret_cast<unsigned char *>(base + l.head_off);
        const uint16_t *feat = (relabel != 2 && l.plan.fsort_tmp_bytes > 0)
                                   ? reinterpret_cast<const uint16_t *>(pw + l.plan.feat_off) : nullptr;
        if ((rc = launch_head_split2(W, M, m_full, head, feat, head_max, img, s))) return rc;
        MmaArgs a;
        a.W = W; a.M = M; a.N = N; a.n_tiles = (N + 7) / 8; a.norms = norms;
        a.perm = reinterpret_cast<const int32_t *>(pw + l.plan.perm_off);
        a.tile_len = reinterpret_cast<const uint32_t *>(pw + l.plan.tilelen_off);
        a.tile_off = reinterpret_cast<const uint32_t *>(pw + l.plan.tileoff_off);
        a.tile_ids = reinterpret_cast<const uint4 *>(pw + l.plan.tileids_off);
        a.tile_head = reinterpret_cast<const uint32_t *>(pw + l.plan.tilehead_off);
        a.head_max = head_max; a.head = head; a.f16 = 0;
        a.state = state; a.state2 = state2; a.status = status;
        a.D = D; a.tile_rows_cap = l.plan.tile_rows_cap;
        const int64_t chunk = r.chunk;
        float *compact = repack_bytes ? reinterpret_cast<float *>(base + l.repack_off) : nullptr;
        const LaunchCuts cuts(m_full, chunk);
        for (int64_t k = 0; k < cuts.n; ++k) {
            const int64_t j = cuts.cut(k);
            a.j_lo = (int32_t)j;
            a.j_hi = (int32_t)cuts.cut(k + 1);
            a.first = j == 0;
            a.W = W; a.M = M;
            if (compact) {                 // gather from a compact copy of this chunk's columns
                const int32_t width = a.j_hi - a.j_lo;
                { repack_chunk_kernel<<<(unsigned)D, 256, 0, s>>>(
                    reinterpret_cast<const char *>(W), M * 4, j * 4, width * 4,
                    reinterpret_cast<char *>(compact)); BMU_LAUNCHED(); }
                a.W = reinterpret_cast<const float *>(reinterpret_cast<uintptr_t>(compact) -
                                                      (uintptr_t)j * sizeof(float));
                a.M = width;
            }
            // the image takes 4 * head bytes per neuron, slab after slab
            a.head_img = img + (size_t)j * head * 4;
            if ((rc = launch_sweep_mma2(a, o, s))) return rc;
        }
        if (m_full < M) {                      // ragged last slab: generic kernel, merged in
            SweepArgs g;
            g.W = W; g.D = D; g.M = M; g.norms = norms; g.rowptr = rowptr; g.colidx = colidx;
            g.N = N; g.state = state; g.state2 = state2; g.status = status; g.j_lo = (int32_t)m_full;
            g.j_hi = (int32_t)M; g.first = 0;
            bmu_opts go;
            memset(&go, 0, sizeof(go));
            if ((rc = launch_sweep_direct(g, go, s))) return rc;
        }
        return launch_finalize(state, state2, rowptr, N, out_bmu, out_dist, out_bmu2, out_dist2, s);
    }
    if (tiled) {
        const int head = (o.tile_head == 1 || D < TILE_HEAD_ROWS) ? 0 : TILE_HEAD_ROWS;
        if (phase != 2 &&
            (rc = launch_plan_tiles(rowptr, N, o.tile_order != 1, head, 2, D, pw, l.plan, status, s))) return rc;
        if (phase == 1) return BMU_OK;
        TileArgs a;
        a.W = W; a.M = M; a.N = N; a.n_tiles = (N + 7) / 8; a.norms = norms;
        a.perm = reinterpret_cast<const int32_t *>(pw + l.plan.perm_off);
        a.tile_len = reinterpret_cast<const uint32_t *>(pw + l.plan.tilelen_off);
        a.tile_off = reinterpret_cast<const uint32_t *>(pw + l.plan.tileoff_off);
        a.tile_ids = reinterpret_cast<const uint4 *>(pw + l.plan.tileids_off);
        a.tile_head = reinterpret_cast<const uint32_t *>(pw + l.plan.tilehead_off);
        a.head_rows = head;
        a.state = state; a.state2 = state2; a.status = status;
        a.D = D; a.tile_rows_cap = l.plan.tile_rows_cap;
        const int64_t chunk = r.chunk, m_full = r.m_full;
        for (int64_t j = 0; j < m_full; j += chunk) {
            a.j_lo = (int32_t)j;
            a.j_hi = (int32_t)(j + chunk < m_full ? j + chunk : m_full);
            a.first = j == 0;
            if ((rc = launch_sweep_tiles(a, o, s))) return rc;
        }
        if (m_full < M) {                      // ragged last slab: generic kernel, merged in
            SweepArgs g;
            g.W = W; g.D = D; g.M = M; g.norms = norms; g.rowptr = rowptr; g.colidx = colidx;
            g.N = N; g.state = state; g.state2 = state2; g.status = status; g.j_lo = (int32_t)m_full;
            g.j_hi = (int32_t)M; g.first = 0;
            bmu_opts go;
            memset(&go, 0, sizeof(go));
            if ((rc = launch_sweep_direct(g, go, s))) return rc;
        }
        return launch_finalize(state, state2, rowptr, N, out_bmu, out_dist, out_bmu2, out_dist2, s);
    }
    if (phase == 1) return BMU_OK;           // nothing more to prepare for the other kernels
    if (planned) {
        const int slab = rows_slab_width(o);
        RowsArgs a;
        a.W = W; a.M = M; a.N = N; a.norms = norms; a.rowptr = rowptr;
        a.perm = reinterpret_cast<const int32_t *>(pw + l.plan.perm_off);
        a.doc_off = reinterpret_cast<const uint32_t *>(pw + l.plan.docoff_off);
        a.ids = reinterpret_cast<const uint4 *>(pw + l.plan.ids_off);
        a.state = state; a.state2 = state2; a.status = status;
        a.D = D; a.id_groups_cap = l.plan.id_groups_cap;
        const int64_t chunk = r.chunk, m_full = r.m_full;
        for (int64_t j = 0; j < m_full; j += chunk) {
            a.j_lo = (int32_t)j;
            a.j_hi = (int32_t)(j + chunk < m_full ? j + chunk : m_full);
            a.first = j == 0;
            if ((rc = launch_sweep_rows(a, o, s))) return rc;
        }
        if (m_full < M) {                      // ragged last slab: generic kernel, merged in
            SweepArgs g;
            g.W = W; g.D = D; g.M = M; g.norms = norms; g.rowptr = rowptr; g.colidx = colidx;
            g.N = N; g.state = state; g.state2 = state2; g.status = status; g.j_lo = (int32_t)m_full; g.j_hi = (int32_t)M; g.first = 0;
            bmu_opts go;
            memset(&go, 0, sizeof(go));
            if ((rc = launch_sweep_direct(g, go, s))) return rc;
        }
        return launch_finalize(state, state2, rowptr, N, out_bmu, out_dist, out_bmu2, out_dist2, s);
    }
    if (o.warps == 4) { set_error("generic kernel: warps must be 8, 16 or 32"); return BMU_ERR_INVALID_ARG; }
    const int64_t chunk = r.chunk;
    SweepArgs a;
    a.W = W; a.D = D; a.M = M; a.norms = norms; a.rowptr = rowptr; a.colidx = colidx;
    a.N = N; a.state = state; a.state2 = state2; a.status = status;
    for (int64_t j = 0; j < M; j += chunk) {
        a.j_lo = (int32_t)j;
        a.j_hi = (int32_t)(j + chunk < M ? j + chunk : M);
        a.first = j == 0;
        if ((rc = launch_sweep_direct(a, o, s))) return rc;
    }
    return launch_finalize(state, state2, rowptr, N, out_bmu, out_dist, out_bmu2, out_dist2, s);
}

// ---- library-owned grow-only scratch (one per device) ----------------------
struct Scratch { void *p; size_t bytes; };
static Scratch g_scratch[64];
static std::mutex g_mu;

static int scratch_get(size_t bytes, void **out)
{
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) { set_error("device ordinal %d out of range", dev); return BMU_ERR_UNSUPPORTED; }
    std::lock_guard<std::mutex> g(g_mu);
    Scratch &sc = g_scratch[dev];
    if (sc.bytes < bytes) {
        if (sc.p) {
            BMU_CUDA(cudaDeviceSynchronize());
            BMU_CUDA(cudaFree(sc.p));
            sc.p = nullptr; sc.bytes = 0;
        }
        const size_t want = align_up(bytes + bytes / 8, (size_t)1 << 20);
        BMU_CUDA(cudaMalloc(&sc.p, want));
        sc.bytes = want;
    }
    *out = sc.p;
    return BMU_OK;
}

// what a non-zero status word means, for the host entry points that read it back
static int status_error(uint32_t status)
{
    if (status & PLAN_STATUS_OVERFLOW) {
        set_error("the tiling pass found an offset beyond its reserved room (status word %u); "
                  "results are invalid", status);
        return BMU_ERR_WORKSPACE;
    }
    set_error("a bounded device-side wait ran out (status word %u); results are invalid", status);
    return BMU_ERR_TIMEOUT;
}

// ORs the status word of one search into a word that outlives the next search's clearing
__global__ void status_accumulate_kernel(const uint32_t *__restrict__ status,
                                         uint32_t *__restrict__ sticky)
{
    if (*status) atomicOr(sticky, *status);
}

// ---- CSR validation ---------------------------------------------------------
__global__ void validate_kernel(const int32_t *__restrict__ rowptr,
                                const int32_t *__restrict__ colidx, int64_t N, int64_t nnz,
                                int64_t D, int32_t *__restrict__ flags)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    if (t == 0) {
        if (rowptr[0] != 0) atomicOr(flags, 1);
        if ((int64_t)rowptr[N] != nnz) atomicOr(flags, 2);
    }
    for (int64_t i = t; i < N; i += stride) {
        if (rowptr[i + 1] < rowptr[i]) atomicOr(flags, 4);
        if ((int64_t)rowptr[i + 1] - rowptr[i] > 65535) atomicOr(flags, 16);
    }
    for (int64_t e = t; e < nnz; e += stride) {
        const int32_t f = colidx[e];
        if (f < 0 || (int64_t)f >= D) atomicOr(flags, 8);
    }
}

int launch_validate_csr(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                        int64_t D, int32_t *flags, cudaStream_t s)
{
    BMU_CUDA(cudaMemsetAsync(flags, 0, sizeof(int32_t), s));
    { validate_kernel<<<296, 256, 0, s>>>(rowptr, colidx, N, nnz, D, flags); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu

using namespace bmu;

extern "C" {

const char *bmu_status_string(int status)
{
    switch (status) {
    case BMU_OK: return "ok";
    case BMU_ERR_INVALID_ARG: return "invalid argument";
    case BMU_ERR_UNSUPPORTED: return "unsupported size or option";
    case BMU_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case BMU_ERR_CUDA: return "CUDA runtime error";
    case BMU_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
    }
}

const char *bmu_last_error(void) { return g_err; }

int bmu_version(void) { return 200; }

uint64_t bmu_kernel_launches(void) { return g_kernel_launches; }

int bmu_describe_search(int64_t D, int64_t M, int64_t N, int64_t nnz, const bmu_opts *opts,
                        bmu_search_desc *out)
{
    if (!out) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    memset(out, 0, sizeof(*out));
    int rc = check_sizes(D, M, N, nnz);
    if (rc) return rc;
    bmu_opts o;
    memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    if ((rc = check_opts(o))) return rc;
    if (M == 0 || D == 0) { set_error("empty codebook"); return BMU_ERR_INVALID_ARG; }
    Route r;
    if ((rc = route_search(o, D, M, nnz, 0, r))) return rc;
    out->kernel = r.kernel;
    out->head_rows = r.head;
    out->slab = r.slab;
    out->docs_per_block = r.docs_per_block;
    out->repack = r.repack;
    out->chunk_neurons = r.chunk;
    out->sweep_launches = (int32_t)((r.m_full + r.chunk - 1) / r.chunk);
    out->ragged_neurons = (int32_t)(M - r.m_full);
    return BMU_OK;
}

int bmu_codebook_norms(const float *W, int64_t D, int64_t M, float *norms, void *stream)
{
    int rc = check_sizes(D, M, 0, 0);
    if (rc) return rc;
    if (M == 0) return BMU_OK;
    if (!norms || (D > 0 && !W)) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    return launch_norms(W, D, M, norms, static_cast<cudaStream_t>(stream));
}

size_t bmu_search_workspace_bytes(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                  const bmu_opts *opts)
{
    if (D < 0 || M < 0 || N < 0 || nnz < 0) return 0;
    bmu_opts o;
    memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    return layout_of(o, D, M, N, nnz, false).total;
}

int bmu_search_ws(const float *W, int64_t D, int64_t M, const float *norms,
                  const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                  int32_t *out_bmu, float *out_dist, const bmu_opts *opts, void *workspace,
                  size_t workspace_bytes, void *stream)
{
    return search_impl(W, D, M, norms, rowptr, colidx, N, nnz, out_bmu, out_dist, opts,
                       workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

size_t bmu_search_top2_workspace_bytes(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                       const bmu_opts *opts)
{
    if (D < 0 || M < 0 || N < 0 || nnz < 0) return 0;
    bmu_opts o;
    memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    return layout_of(o, D, M, N, nnz, true).total;
}

int bmu_search_top2_ws(const float *W, int64_t D, int64_t M, const float *norms,
                       const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                       int32_t *out_bmu, float *out_dist, int32_t *out_bmu2, float *out_dist2,
                       const bmu_opts *opts, void *workspace, size_t workspace_bytes,
                       void *stream)
{
    if (N > 0 && (!out_bmu2 || !out_dist2)) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    return search_impl(W, D, M, norms, rowptr, colidx, N, nnz, out_bmu, out_dist, opts, workspace,
                       workspace_bytes, static_cast<cudaStream_t>(stream), out_bmu2, out_dist2);
}

int bmu_codebook_norms_f16(const void *W16, int64_t D, int64_t M, float *norms, void *stream)
{
    int rc = check_sizes(D, M, 0, 0);
    if (rc) return rc;
    if (M == 0) return BMU_OK;
    if (!norms || (D > 0 && !W16)) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    if (M % 8 != 0 || (reinterpret_cast<uintptr_t>(W16) & 15) != 0) {
        set_error("half-precision codebook needs M %% 8 == 0 and 16-byte alignment");
        return BMU_ERR_UNSUPPORTED;
    }
    return launch_norms_f16(W16, D, M, norms, static_cast<cudaStream_t>(stream));
}

// Which kernel a half-precision search takes: large sweeps the wide tensor-core sweep (whole
// 256-neuron slabs only), the rest the planned kernel.  `ow` = the options of the wide sweep, its
// head resolved (576 by default: with 2-byte rows the gathered tail is cheap, so the balance
// point sits lower than the fp32 sweep's 640; config 4 at full length: 2364 / 2348 / 2331 / 2473
// ms per step at 448 / 512 / 576 / 704).
static bool f16_route(const bmu_opts &o, int64_t D, int64_t M, int64_t nnz, bmu_opts &ow, bool &wide)
{
    ow = o;
    ow.kernel = 6;
    if (!ow.head_rows) {
        const int64_t cap = D / 64 * 64;
        ow.head_rows = (int32_t)(cap < 576 ? (cap < 64 ? 64 : cap) : 576);
    }
    const bool wide_ok = M % MMA_SLAB == 0 && D >= ow.head_rows && o.cluster != 2;
    wide = wide_ok && (o.kernel == 6 || (o.kernel == 0 && (double)nnz * (double)M >= 2e10));
    return wide_ok;
}

size_t bmu_search_f16_workspace_bytes(int64_t D, int64_t M, int64_t N, int64_t nnz,
                                      const bmu_opts *opts)
{
    if (D < 0 || M < 0 || N < 0 || nnz < 0) return 0;
    bmu_opts o, ow;
    memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    bool wide = false;
    f16_route(o, D, M, nnz, ow, wide);
    return (wide ? layout_of(ow, D, M, N, nnz, true) : layout_for(D, M, N, nnz, 3, true)).total;
}

int bmu_search_f16_ws(const void *W16, int64_t D, int64_t M, const float *norms,
                      const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                      int32_t *out_bmu, float *out_dist, int32_t *out_bmu2, float *out_dist2,
                      const bmu_opts *opts, void *ws, size_t ws_bytes, void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = check_sizes(D, M, N, nnz);
    if (rc) return rc;
    bmu_opts o;
    memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    if ((rc = check_opts(o))) return rc;
    if (N == 0) return BMU_OK;
    const bool top2 = out_bmu2 != nullptr || out_dist2 != nullptr;
    if (!W16 || !rowptr || !out_bmu || !out_dist || (nnz > 0 && !colidx) ||
        (top2 && (!out_bmu2 || !out_dist2))) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    if (M % 256 != 0 || D < 1 || D > LANES_MAX_D || (reinterpret_cast<uintptr_t>(W16) & 15) != 0 ||
        (o.kernel != 0 && o.kernel != 3 && o.kernel != 6)) {
        set_error("half-precision search needs M %% 256 == 0, 1 <= D <= %d, 16-byte alignment and "
                  "the planned (3) or the wide tensor-core (6) kernel", LANES_MAX_D);
        return BMU_ERR_UNSUPPORTED;
    }
    bmu_opts ow;
    bool wide = false;
    const bool wide_ok = f16_route(o, D, M, nnz, ow, wide);
    const int head = ow.head_rows;
    if (o.kernel == 6 && !wide_ok) {
        set_error("half-precision tensor-core sweep needs M %% %d == 0, D >= %d and length-ordered "
                  "documents", MMA_SLAB, head);
        return BMU_ERR_UNSUPPORTED;
    }
    const Layout l = wide ? layout_of(ow, D, M, N, nnz, top2) : layout_for(D, M, N, nnz, 3, top2);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < l.total) {
        set_error("workspace missing, not 256-byte aligned, or smaller than %zu bytes", l.total);
        return BMU_ERR_WORKSPACE;
    }
    char *base = static_cast<char *>(ws);
    u64 *state = reinterpret_cast<u64 *>(base + l.state_off);
    u64 *state2 = top2 ? reinterpret_cast<u64 *>(base + l.state2_off) : nullptr;
    if (!norms) {
        float *n = reinterpret_cast<float *>(base + l.norms_off);
        if ((rc = launch_norms_f16(W16, D, M, n, s))) return rc;
        norms = n;
    }
    if (wide) {
        uint32_t *status = reinterpret_cast<uint32_t *>(base + l.status_off);
        BMU_CUDA(cudaMemsetAsync(status, 0, 256, s));
        char *pw = base + l.plan_off;
        const int relabel = o.relabel;
        if ((rc = launch_plan(rowptr, colidx, N, nnz, plan_order(o, true), head, relabel, D, pw, l.plan,
                              status, s))) return rc;
        if ((rc = launch_plan_tiles(rowptr, N, o.tile_order == 2, head, relabel, D, pw, l.plan, status, s))) return rc;
        unsigned char *img = reinterpret_cast<unsigned char *>(base + l.head_off);
        const uint16_t *feat = (relabel != 2 && l.plan.fsort_tmp_bytes > 0)
                                   ? reinterpret_cast<const uint16_t *>(pw + l.plan.feat_off) : nullptr;
        if ((rc = launch_head_split2_f16(W16, M, M, head, feat, img, s))) return rc;
        MmaArgs a;
        a.W = static_cast<const float *>(W16); a.M = M; a.N = N; a.n_tiles = (N + 7) / 8; a.norms = norms;
        a.perm = reinterpret_cast<const int32_t *>(pw + l.plan.perm_off);
        a.tile_len = reinterpret_cast<const uint32_t *>(pw + l.plan.tilelen_off);
        a.tile_off = reinterpret_cast<const uint32_t *>(pw + l.plan.tileoff_off);
        a.tile_ids = reinterpret_cast<const uint4 *>(pw + l.plan.tileids_off);
        a.tile_head = reinterpret_cast<const uint32_t *>(pw + l.plan.tilehead_off);
        a.head_max = status + 16; a.head = head; a.f16 = 1;
        a.state = state; a.state2 = state2; a.status = status;
        a.D = D; a.tile_rows_cap = l.plan.tile_rows_cap;
        // twice the neurons per L2-resident chunk: the rows are half as wide
        const int64_t chunk = o.chunk_neurons ? mma_chunk(o, D, M) : 2 * mma_auto_chunk(D, M);
        const size_t repack_bytes = mma_repack_bytes(ow, D, M, N, nnz, top2);
        char *compact = (repack_bytes && M > chunk) ? base + l.repack_off : nullptr;
        const LaunchCuts cuts(M, chunk);
        for (int64_t k = 0; k < cuts.n; ++k) {
            const int64_t j = cuts.cut(k);
            a.j_lo = (int32_t)j;
            a.j_hi = (int32_t)cuts.cut(k + 1);
            a.first = j == 0;
            a.W = static_cast<const float *>(W16); a.M = M;
            if (compact) {                 // a compact copy of this chunk's columns (2 bytes each)
                const int32_t width = a.j_hi - a.j_lo;
                { repack_chunk_kernel<<<(unsigned)D, 256, 0, s>>>(static_cast<const char *>(W16), M * 2,
                                                              j * 2, width * 2, compact); BMU_LAUNCHED(); }
                a.W = reinterpret_cast<const float *>(reinterpret_cast<uintptr_t>(compact) -
                                                      (uintptr_t)j * 2);
                a.M = width;
            }
            a.head_img = img + (size_t)j * head * 2;     // one part: 2 * head bytes per neuron
            if ((rc = launch_sweep_mma2_f16(a, o, s))) return rc;
        }
        return launch_finalize(state, state2, rowptr, N, out_bmu, out_dist, out_bmu2, out_dist2, s);
    }
    uint32_t *status = reinterpret_cast<uint32_t *>(base + l.status_off);
    BMU_CUDA(cudaMemsetAsync(status, 0, 256, s));
    char *pw = base + l.plan_off;
    if ((rc = launch_plan(rowptr, colidx, N, nnz, o.cluster != 2, 0, 2, D, pw, l.plan, status, s))) return rc;
    RowsArgs a;
    a.status = status; a.D = D; a.id_groups_cap = l.plan.id_groups_cap;
    a.W = static_cast<const float *>(W16); a.M = M; a.N = N; a.norms = norms; a.rowptr = rowptr;
    a.perm = reinterpret_cast<const int32_t *>(pw + l.plan.perm_off);
    a.doc_off = reinterpret_cast<const uint32_t *>(pw + l.plan.docoff_off);
    a.ids = reinterpret_cast<const uint4 *>(pw + l.plan.ids_off);
    a.state = state; a.state2 = state2;
    // twice the neurons per L2-resident chunk: the rows are half as wide
    const int64_t chunk = o.chunk_neurons ? (o.chunk_neurons + 255) / 256 * 256
                                          : auto_chunk(D, M, 256) * 2;
    for (int64_t j = 0; j < M; j += chunk) {
        a.j_lo = (int32_t)j;
        a.j_hi = (int32_t)(j + chunk < M ? j + chunk : M);
        a.first = j == 0;
        if ((rc = launch_sweep_rows_f16(a, o, s))) return rc;
    }
    return launch_finalize(state, state2, rowptr, N, out_bmu, out_dist, out_bmu2, out_dist2, s);
}

int bmu_search(const float *W, int64_t D, int64_t M, const int32_t *rowptr,
               const int32_t *colidx, int64_t N, int32_t *out_bmu, float *out_dist,
               void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = check_sizes(D, M, N, 0);
    if (rc) return rc;
    if (N == 0) return BMU_OK;
    if (!rowptr) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    int32_t nnz = 0;
    BMU_CUDA(cudaMemcpyAsync(&nnz, rowptr + N, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    const size_t need = bmu_search_workspace_bytes(D, M, N, nnz, nullptr);
    void *ws = nullptr;
    if ((rc = scratch_get(need, &ws))) return rc;
    return search_impl(W, D, M, nullptr, rowptr, colidx, N, nnz, out_bmu, out_dist, nullptr, ws,
                       need, s);
}

int bmu_search_host(const float *W, int64_t D, int64_t M, const int32_t *rowptr_host,
                    const int32_t *colidx_host, int64_t N, int32_t *out_bmu_host,
                    float *out_dist_host, void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = check_sizes(D, M, N, 0);
    if (rc) return rc;
    if (N == 0) return BMU_OK;
    if (!rowptr_host || !out_bmu_host || !out_dist_host) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    const int64_t nnz = rowptr_host[N];
    if (nnz < 0 || (nnz > 0 && !colidx_host)) { set_error("bad rowptr[N] or null colidx"); return BMU_ERR_INVALID_ARG; }
    const size_t ws_need = bmu_search_workspace_bytes(D, M, N, nnz, nullptr);
    const size_t rp_off = align_up(ws_need, 256);
    const size_t ci_off = align_up(rp_off + (size_t)(N + 1) * 4, 256);
    const size_t ob_off = align_up(ci_off + (size_t)nnz * 4, 256);
    const size_t od_off = align_up(ob_off + (size_t)N * 4, 256);
    const size_t total = align_up(od_off + (size_t)N * 4, 256);
    void *p = nullptr;
    if ((rc = scratch_get(total, &p))) return rc;
    char *b = static_cast<char *>(p);
    int32_t *rp = reinterpret_cast<int32_t *>(b + rp_off);
    int32_t *ci = reinterpret_cast<int32_t *>(b + ci_off);
    int32_t *ob = reinterpret_cast<int32_t *>(b + ob_off);
    float *od = reinterpret_cast<float *>(b + od_off);
    BMU_CUDA(cudaMemcpyAsync(rp, rowptr_host, (size_t)(N + 1) * 4, cudaMemcpyHostToDevice, s));
    if (nnz)
        BMU_CUDA(cudaMemcpyAsync(ci, colidx_host, (size_t)nnz * 4, cudaMemcpyHostToDevice, s));
    if ((rc = search_impl(W, D, M, nullptr, rp, ci, N, nnz, ob, od, nullptr, b, ws_need, s)))
        return rc;
    BMU_CUDA(cudaMemcpyAsync(out_bmu_host, ob, (size_t)N * 4, cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaMemcpyAsync(out_dist_host, od, (size_t)N * 4, cudaMemcpyDeviceToHost, s));
    uint32_t status = 0;                               // first word of the workspace
    BMU_CUDA(cudaMemcpyAsync(&status, b, sizeof(status), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    if (status) return status_error(status);
    return BMU_OK;
}

// ---- streamed batches from host memory (config 5: a corpus fed in batches) ----
// Two staging buffers; the copy stream uploads batch k+1 and downloads the results
// of batch k-1 while the caller's stream searches batch k.
struct StreamCtx { cudaStream_t copy; cudaEvent_t h2d[2], done[2], d2h[2]; bool ready; };
static StreamCtx g_stream_ctx[64];

static int stream_ctx_get(int dev, StreamCtx **out)
{
    StreamCtx &c = g_stream_ctx[dev];
    if (!c.ready) {
        BMU_CUDA(cudaStreamCreateWithFlags(&c.copy, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            BMU_CUDA(cudaEventCreateWithFlags(&c.h2d[i], cudaEventDisableTiming));
            BMU_CUDA(cudaEventCreateWithFlags(&c.done[i], cudaEventDisableTiming));
            BMU_CUDA(cudaEventCreateWithFlags(&c.d2h[i], cudaEventDisableTiming));
        }
        c.ready = true;
    }
    *out = &c;
    return BMU_OK;
}

int bmu_search_batches_host(const float *W, int64_t D, int64_t M, int32_t n_batches,
                            const int32_t *const *rowptr_host, const int32_t *const *colidx_host,
                            const int64_t *N, int32_t *const *out_bmu_host,
                            float *const *out_dist_host, void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n_batches < 0 || (n_batches > 0 && (!rowptr_host || !colidx_host || !N || !out_bmu_host ||
                                            !out_dist_host))) {
        set_error("null pointer argument or negative batch count");
        return BMU_ERR_INVALID_ARG;
    }
    int rc;
    int64_t max_n = 0, max_nnz = 0;
    for (int k = 0; k < n_batches; ++k) {
        if (N[k] < 0 || (N[k] > 0 && (!rowptr_host[k] || !out_bmu_host[k] || !out_dist_host[k]))) {
            set_error("batch %d: null pointer or negative size", k);
            return BMU_ERR_INVALID_ARG;
        }
        const int64_t nnz = N[k] > 0 ? rowptr_host[k][N[k]] : 0;
        if ((rc = check_sizes(D, M, N[k], nnz))) return rc;
        if (nnz > 0 && !colidx_host[k]) { set_error("batch %d: null colidx", k); return BMU_ERR_INVALID_ARG; }
        if (N[k] > max_n) max_n = N[k];
        if (nnz > max_nnz) max_nnz = nnz;
    }
    if (max_n == 0) return BMU_OK;
    // layout: status word of the whole call, shared norms | per buffer: workspace, rowptr,
    // colidx, out_bmu, out_dist
    const size_t ws_need = bmu_search_workspace_bytes(D, M, max_n, max_nnz, nullptr);
    const size_t norms_bytes = 256 + align_up((size_t)M * 4, 256);
    const size_t rp_off = align_up(ws_need, 256);
    const size_t ci_off = align_up(rp_off + (size_t)(max_n + 1) * 4, 256);
    const size_t ob_off = align_up(ci_off + (size_t)max_nnz * 4, 256);
    const size_t od_off = align_up(ob_off + (size_t)max_n * 4, 256);
    const size_t per_buf = align_up(od_off + (size_t)max_n * 4, 256);
    void *p = nullptr;
    if ((rc = scratch_get(norms_bytes + 2 * per_buf, &p))) return rc;
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    StreamCtx *c = nullptr;
    if ((rc = stream_ctx_get(dev, &c))) return rc;
    char *b = static_cast<char *>(p);
    uint32_t *sticky = reinterpret_cast<uint32_t *>(b);
    float *norms = reinterpret_cast<float *>(b + 256);
    BMU_CUDA(cudaMemsetAsync(sticky, 0, 256, s));
    if ((rc = launch_norms(W, D, M, norms, s))) return rc;
    for (int k = 0; k < n_batches; ++k) {
        if (N[k] == 0) continue;
        const int i = k & 1;
        char *buf = b + norms_bytes + (size_t)i * per_buf;
        const int64_t n = N[k], nnz = rowptr_host[k][n];
        int32_t *rp = reinterpret_cast<int32_t *>(buf + rp_off);
        int32_t *ci = reinterpret_cast<int32_t *>(buf + ci_off);
        int32_t *ob = reinterpret_cast<int32_t *>(buf + ob_off);
        float *od = reinterpret_cast<float *>(buf + od_off);
        // upload: the buffer is free once the results of its previous batch are out
        if (k >= 2) BMU_CUDA(cudaStreamWaitEvent(c->copy, c->d2h[i], 0));
        BMU_CUDA(cudaMemcpyAsync(rp, rowptr_host[k], (size_t)(n + 1) * 4, cudaMemcpyHostToDevice, c->copy));
        if (nnz)
            BMU_CUDA(cudaMemcpyAsync(ci, colidx_host[k], (size_t)nnz * 4, cudaMemcpyHostToDevice, c->copy));
        BMU_CUDA(cudaEventRecord(c->h2d[i], c->copy));
        // search on the caller's stream
        BMU_CUDA(cudaStreamWaitEvent(s, c->h2d[i], 0));
        if ((rc = search_impl(W, D, M, norms, rp, ci, n, nnz, ob, od, nullptr, buf, ws_need, s)))
            return rc;
        // the next search of this buffer clears its status word: keep what this one left
        { status_accumulate_kernel<<<1, 1, 0, s>>>(reinterpret_cast<const uint32_t *>(buf), sticky); BMU_LAUNCHED(); }
        BMU_CUDA(cudaEventRecord(c->done[i], s));
        // download on the copy stream
        BMU_CUDA(cudaStreamWaitEvent(c->copy, c->done[i], 0));
        BMU_CUDA(cudaMemcpyAsync(out_bmu_host[k], ob, (size_t)n * 4, cudaMemcpyDeviceToHost, c->copy));
        BMU_CUDA(cudaMemcpyAsync(out_dist_host[k], od, (size_t)n * 4, cudaMemcpyDeviceToHost, c->copy));
        BMU_CUDA(cudaEventRecord(c->d2h[i], c->copy));
    }
    uint32_t status = 0;
    BMU_CUDA(cudaMemcpyAsync(&status, sticky, sizeof(status), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    BMU_CUDA(cudaStreamSynchronize(c->copy));
    if (status) return status_error(status);
    return BMU_OK;
}

int bmu_status_of_word(uint32_t status_word)
{
    return status_word ? status_error(status_word) : BMU_OK;
}

int bmu_last_status(uint32_t *out_status, void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!out_status) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    *out_status = 0;
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) { set_error("device ordinal %d out of range", dev); return BMU_ERR_UNSUPPORTED; }
    void *p = nullptr;
    {
        std::lock_guard<std::mutex> g(g_mu);
        p = g_scratch[dev].p;
    }
    if (p) BMU_CUDA(cudaMemcpyAsync(out_status, p, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    if (*out_status) return status_error(*out_status);
    return BMU_OK;
}

int bmu_selftest_wait_timeout(void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void *p = nullptr;
    int rc = scratch_get(512, &p);          // word 0 of the scratch stays the searches' status word
    if (rc) return rc;
    uint32_t *status = reinterpret_cast<uint32_t *>(static_cast<char *>(p) + 256);
    BMU_CUDA(cudaMemsetAsync(status, 0, 256, s));
    if ((rc = launch_wait_timeout_selftest(status, s))) return rc;
    uint32_t h = 0;
    BMU_CUDA(cudaMemcpyAsync(&h, status, sizeof(h), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    if (h) return status_error(h);
    return BMU_OK;
}

int bmu_release_scratch(void)
{
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return BMU_OK;
    std::lock_guard<std::mutex> g(g_mu);
    Scratch &sc = g_scratch[dev];
    if (sc.p) {
        BMU_CUDA(cudaDeviceSynchronize());
        BMU_CUDA(cudaFree(sc.p));
        sc.p = nullptr; sc.bytes = 0;
    }
    return BMU_OK;
}

int bmu_validate_csr(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                     int64_t D, void *stream)
{
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = check_sizes(D, 0, N, nnz);
    if (rc) return rc;
    if (!rowptr || (nnz > 0 && !colidx)) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    void *p = nullptr;
    if ((rc = scratch_get(512, &p))) return rc;   // word 0 stays the searches' status word
    int32_t *flags = reinterpret_cast<int32_t *>(static_cast<char *>(p) + 256);
    if ((rc = launch_validate_csr(rowptr, colidx, N, nnz, D, flags, s))) return rc;
    int32_t h = 0;
    BMU_CUDA(cudaMemcpyAsync(&h, flags, sizeof(h), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    if (h) {
        set_error("invalid CSR:%s%s%s%s%s", (h & 1) ? " rowptr[0] != 0;" : "",
                  (h & 2) ? " rowptr[N] != nnz;" : "", (h & 4) ? " rowptr decreases;" : "",
                  (h & 8) ? " colidx outside [0, D);" : "",
                  (h & 16) ? " a row lists more than 65535 ids;" : "");
        return BMU_ERR_INVALID_ARG;
    }
    return BMU_OK;
}

// ---- reusable tiling plan: a frozen corpus searched once per epoch ------------
struct bmu_plan {
    int64_t D, M, N, nnz;
    bmu_opts opts;
    const int32_t *rowptr, *colidx;
    void *ws;
    size_t ws_bytes;
};

size_t bmu_plan_workspace_bytes(int64_t N, int64_t nnz, int64_t D, int64_t M, const bmu_opts *opts)
{
    return bmu_search_workspace_bytes(D, M, N, nnz, opts);
}

int bmu_plan_create(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz, int64_t D,
                    int64_t M, const bmu_opts *opts, void *workspace, size_t workspace_bytes,
                    bmu_plan **plan, void *stream)
{
    if (!plan) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    *plan = nullptr;
    if (N <= 0) { set_error("a plan needs at least one document"); return BMU_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = search_impl(nullptr, D, M, nullptr, rowptr, colidx, N, nnz, nullptr, nullptr, opts,
                         workspace, workspace_bytes, s, nullptr, nullptr, 1);
    if (rc) return rc;
    // the searches that reuse the plan clear the status word: read the size checks of the
    // tiling pass now
    uint32_t status = 0;
    BMU_CUDA(cudaMemcpyAsync(&status, workspace, sizeof(status), cudaMemcpyDeviceToHost, s));
    BMU_CUDA(cudaStreamSynchronize(s));
    if (status) return status_error(status);
    bmu_plan *p = new (std::nothrow) bmu_plan;
    if (!p) { set_error("out of host memory"); return BMU_ERR_INVALID_ARG; }
    p->D = D; p->M = M; p->N = N; p->nnz = nnz;
    memset(&p->opts, 0, sizeof(p->opts));
    if (opts) p->opts = *opts;
    p->rowptr = rowptr; p->colidx = colidx; p->ws = workspace; p->ws_bytes = workspace_bytes;
    *plan = p;
    return BMU_OK;
}

int bmu_search_planned(const bmu_plan *plan, const float *W, const float *norms, int32_t *out_bmu,
                       float *out_dist, void *stream)
{
    if (!plan) { set_error("null plan"); return BMU_ERR_INVALID_ARG; }
    return search_impl(W, plan->D, plan->M, norms, plan->rowptr, plan->colidx, plan->N, plan->nnz,
                       out_bmu, out_dist, &plan->opts, plan->ws, plan->ws_bytes,
                       static_cast<cudaStream_t>(stream), nullptr, nullptr, 2);
}

int bmu_plan_order(const bmu_plan *plan, int32_t *out_order, void *stream)
{
    if (!plan || !out_order) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    Route r;
    int rc = route_search(plan->opts, plan->D, plan->M, plan->nnz, 0, r);
    if (rc) return rc;
    if (r.kernel == 1) {
        set_error("the generic kernel makes no plan: documents keep the corpus order");
        return BMU_ERR_UNSUPPORTED;
    }
    const Layout l = layout_of(plan->opts, plan->D, plan->M, plan->N, plan->nnz, false);
    const char *perm = static_cast<const char *>(plan->ws) + l.plan_off + l.plan.perm_off;
    BMU_CUDA(cudaMemcpyAsync(out_order, perm, (size_t)plan->N * sizeof(int32_t),
                             cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)));
    return BMU_OK;
}

void bmu_plan_destroy(bmu_plan *plan) { delete plan; }

// ---- the rest of a batch epoch (Table 4: scatter, blur, write-back) -----------
int bmu_update_scatter(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                       const int32_t *bmu, int64_t D, int64_t M, uint32_t *num, uint32_t *cnt,
                       void *stream)
{
    int rc = check_sizes(D, M, N, nnz);
    if (rc) return rc;
    if (N == 0) return BMU_OK;
    if (!rowptr || !bmu || !num || !cnt || (nnz > 0 && !colidx)) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    return launch_update_scatter(rowptr, colidx, N, bmu, M, num, cnt, static_cast<cudaStream_t>(stream));
}

int bmu_update_blur(const uint32_t *num, const uint32_t *cnt, int64_t D, int32_t edge_x,
                    int32_t edge_y, float sigma, float *num_blur, float *cnt_blur, void *stream)
{
    if (D < 0 || edge_x < 0 || edge_y < 0 || !(sigma >= 0.f)) {
        set_error("negative size or sigma");
        return BMU_ERR_INVALID_ARG;
    }
    int rc = check_sizes(D, (int64_t)edge_x * edge_y, 0, 0);
    if (rc) return rc;
    if (D > LANES_MAX_D) { set_error("blur: D beyond %d", LANES_MAX_D); return BMU_ERR_UNSUPPORTED; }
    if ((int64_t)edge_x * edge_y == 0) return BMU_OK;
    if (!cnt || !cnt_blur || (D > 0 && (!num || !num_blur))) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    return launch_update_blur(num, cnt, D, edge_x, edge_y, sigma, num_blur, cnt_blur,
                              static_cast<cudaStream_t>(stream));
}

int bmu_update_writeback(const float *num_blur, const float *cnt_blur, int64_t D, int64_t M,
                         float *W, void *stream)
{
    int rc = check_sizes(D, M, 0, 0);
    if (rc) return rc;
    if (D * M == 0) return BMU_OK;
    if (D > 65535) { set_error("write-back: D beyond 65535"); return BMU_ERR_UNSUPPORTED; }
    if (!num_blur || !cnt_blur || !W) { set_error("null pointer argument"); return BMU_ERR_INVALID_ARG; }
    return launch_update_writeback(num_blur, cnt_blur, D, M, W, static_cast<cudaStream_t>(stream));
}

int bmu_score_block_argmin(const void *scores, int32_t half, int64_t n_rows, int64_t M,
                           const float *norms, const int32_t *rowptr, int32_t *out_bmu,
                           float *out_dist, void *stream)
{
    int rc = check_sizes(0, M, n_rows, 0);
    if (rc) return rc;
    if (n_rows == 0) return BMU_OK;
    if (!scores || !norms || !rowptr || !out_bmu || !out_dist) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    if (M == 0) { set_error("empty score rows: no neuron to return"); return BMU_ERR_INVALID_ARG; }
    if (M % (half ? 8 : 4) != 0 || (reinterpret_cast<uintptr_t>(scores) & 15) != 0 ||
        (reinterpret_cast<uintptr_t>(norms) & 15) != 0) {
        set_error("score read-back needs M %% %d == 0 and 16-byte aligned scores and norms",
                  half ? 8 : 4);
        return BMU_ERR_UNSUPPORTED;
    }
    return launch_readback_argmin(scores, half != 0, n_rows, M, norms, rowptr, out_bmu, out_dist,
                                  static_cast<cudaStream_t>(stream));
}

size_t bmu_map_errors_workspace_bytes(void) { return map_errors_workspace_bytes(); }

int bmu_map_errors(const int32_t *bmu, const int32_t *bmu2, const float *dist, int64_t N,
                   int32_t edge_x, int32_t edge_y, int32_t adjacency, double *out, void *workspace,
                   size_t workspace_bytes, void *stream)
{
    if (N < 0 || N > MAX_I32 || edge_x < 1 || edge_y < 1 || (adjacency != 4 && adjacency != 8)) {
        set_error("map errors: need 0 <= N < 2^31, edges >= 1 and adjacency 4 or 8");
        return BMU_ERR_INVALID_ARG;
    }
    if (!out || (N > 0 && (!bmu || !bmu2 || !dist))) {
        set_error("null pointer argument");
        return BMU_ERR_INVALID_ARG;
    }
    if (N > 0 && (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 ||
                  workspace_bytes < map_errors_workspace_bytes())) {
        set_error("workspace missing, not 256-byte aligned, or smaller than %zu bytes",
                  map_errors_workspace_bytes());
        return BMU_ERR_WORKSPACE;
    }
    return launch_map_errors(bmu, bmu2, dist, N, edge_x, adjacency, out, workspace,
                             static_cast<cudaStream_t>(stream));
}

}  // extern "C"

// ---- search with library-resident scratch (no allocation anywhere) ---------
// The scratch of the generic kernel's search -- norms and the running
// per-document minimum -- in an array that is part of the library image.  The
// name below is only a host-side handle: device code may use it directly, but
// host code must ask the runtime for its device address before handing it to a
// kernel, once per device and with that device current.
static const size_t STATIC_SCRATCH_BYTES = (size_t)8 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];
static void *g_static_scratch_addr[64];
static std::mutex g_static_mu;

extern "C" int bmu_search_static(const float *W, int64_t D, int64_t M, const int32_t *rowptr,
                                 const int32_t *colidx, int64_t N, int64_t nnz, int32_t *out_bmu,
                                 float *out_dist, void *stream)
{
    int rc = bmu::check_sizes(D, M, N, nnz);
    if (rc) return rc;
    if (N == 0) return BMU_OK;
    const size_t need = bmu::layout_for(D, M, N, nnz, 1).total;
    if (need > STATIC_SCRATCH_BYTES) {
        bmu::set_error("bmu_search_static: M=%lld and N=%lld need %zu bytes of scratch, the "
                       "built-in array holds %zu; split the batch or use bmu_search_ws",
                       (long long)M, (long long)N, need, STATIC_SCRATCH_BYTES);
        return BMU_ERR_UNSUPPORTED;
    }
    int dev = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) { bmu::set_error("device ordinal %d out of range", dev); return BMU_ERR_UNSUPPORTED; }
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> g(g_static_mu);
        if (!g_static_scratch_addr[dev]) {
            void *p = nullptr;
            BMU_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
            g_static_scratch_addr[dev] = p;
        }
        scratch = g_static_scratch_addr[dev];
    }
    bmu_opts o;
    memset(&o, 0, sizeof(o));
    o.kernel = 1;
    return bmu::search_impl(W, D, M, nullptr, rowptr, colidx, N, nnz, out_bmu, out_dist, &o,
                            scratch, STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(stream));
}
