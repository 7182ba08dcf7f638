// The document-tiling pass (Section 4.1 "tile size", Section 4.2 "tile
// membership"): turns the caller's CSR into the form the planned, tiled and
// tensor-core sweeps walk.  The pass
//   1. orders documents by length (longest first; by the length of the gathered
//      list when there is a dense head) so that the documents that share a warp,
//      a tile or a block carry similar numbers of features and finish together;
//   2. re-packs every row as ascending 16-bit feature ids in 16-byte groups
//      (8 ids), padded with the sentinel 0xFFFF and closed by one all-sentinel
//      group, so eight ids arrive with one aligned 128-bit load and a list
//      ends by itself;
//   3. (tiled and tensor-core sweeps) cuts the length-ordered documents into tiles
//      of 8 and writes, per tile, an id matrix: row b holds the b-th id of each of
//      the tile's 8 documents (0xFFFF where a document has run out), so one aligned
//      128-bit load hands a warp the next row of all eight documents.
// Integer work only; the order of documents never changes any result because
// every document is reduced on its own.
#include "common.cuh"

#include <cub/device/device_radix_sort.cuh>
#include <cub/device/device_scan.cuh>

namespace bmu {

static const int PLAN_BINS = 65536;      // one bin per row length: documents end up exactly
                                         // length-ordered (ids are 16-bit, so rows are shorter)

// ---- frequency ranks of the features (Table 8: the paper relabels its vocabulary by
// frequency and keeps that as substrate; here the relabelling is internal to the plan, so the
// dense head is the `head` most frequent features whatever ids the caller uses) -------------
// Listings per feature for the ids in [lo, hi): counted in shared memory first (a frequent
// feature is listed by most documents, and that many atomics on one global counter crawl),
// then flushed.
__global__ void __launch_bounds__(1024)
plan_feat_hist_kernel(const int32_t *__restrict__ colidx, int64_t nnz, int32_t lo, int32_t hi,
                      uint32_t *__restrict__ count)
{
    extern __shared__ uint32_t bins[];
    const int n_bins = hi - lo;
    for (int b = threadIdx.x; b < n_bins; b += blockDim.x) bins[b] = 0u;
    __syncthreads();
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < nnz;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int32_t f = __ldg(colidx + e);
        if (f >= lo && f < hi) atomicAdd(bins + (f - lo), 1u);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < n_bins; b += blockDim.x)
        if (bins[b]) atomicAdd(count + lo + b, bins[b]);
}

__global__ void plan_iota_kernel(int32_t D, uint32_t *__restrict__ v)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < D) v[i] = (uint32_t)i;
}

// Is the vocabulary labelled by frequency already?  If the ids below `head` cover at least 98 %
// of the listings that the `head` most frequent features cover, the ids are kept as ranks (rows
// then stay ascending and need no re-sorting).  One block.
__global__ void __launch_bounds__(1024)
plan_rank_decide_kernel(const uint32_t *__restrict__ count, const uint32_t *__restrict__ count_sorted,
                        int32_t D, int32_t head, int force, uint32_t *__restrict__ keep_ids)
{
    __shared__ unsigned long long s_id[32], s_rk[32];
    unsigned long long by_id = 0, by_rank = 0;
    for (int i = threadIdx.x; i < head && i < D; i += 1024) {
        by_id += count[i];
        by_rank += count_sorted[i];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        by_id += __shfl_xor_sync(0xffffffffu, by_id, off);
        by_rank += __shfl_xor_sync(0xffffffffu, by_rank, off);
    }
    if ((threadIdx.x & 31) == 0) { s_id[threadIdx.x >> 5] = by_id; s_rk[threadIdx.x >> 5] = by_rank; }
    __syncthreads();
    if (threadIdx.x == 0) {
        by_id = by_rank = 0;
        for (int w = 0; w < 32; ++w) { by_id += s_id[w]; by_rank += s_rk[w]; }
        *keep_ids = (!force && by_id * 100ull >= by_rank * 98ull) ? 1u : 0u;
    }
}

// sorted[r] = the feature of rank r (most frequent first, ties by ascending id)
__global__ void plan_rank_tables_kernel(const uint32_t *__restrict__ sorted, int32_t D,
                                        const uint32_t *__restrict__ keep_ids,
                                        uint16_t *__restrict__ rank_of_feat,
                                        uint16_t *__restrict__ feat_of_rank)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= D) return;
    const uint32_t f = *keep_ids ? (uint32_t)r : sorted[r];
    feat_of_rank[r] = (uint16_t)f;
    rank_of_feat[f] = (uint16_t)r;
}

// Sorting key of a document: how many of its ids the gather will visit, i.e. the ids at or
// above `head` (all of them when head == 0) -- or the whole list if it repeats an id below
// `head`: such a list keeps multiset semantics by staying out of the dense head altogether
// (plan_tile_len_kernel below), so all of it is gathered.  The key must be the gathered length exactly:
// the room reserved for the tile id matrices counts on documents ordered by it.  With `ckeys`
// the same pass over the row also forms the 64-bit content key (plan_cluster_key_kernel below
// says what it holds).  One warp per document.
__device__ __forceinline__ void plan_min3(uint32_t &a, uint32_t &b, uint32_t &c, uint32_t v)
{
    if (v < a) { c = b; b = a; a = v; } else if (v < b) { c = b; b = v; } else if (v < c) { c = v; }
}

__global__ void __launch_bounds__(256)
plan_key_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                const uint16_t *__restrict__ rank, int64_t N, int32_t head,
                uint32_t *__restrict__ key, [[maybe_unused]] int64_t D,
                [[maybe_unused]] uint32_t *__restrict__ status, int mode,
                u64 *__restrict__ ckeys, uint32_t *__restrict__ cvals)
{
    __shared__ uint32_t seen[8][HEAD_ROWS_MAX / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= N) return;
    for (int w = lane; w < head / 32; w += 32) seen[warp][w] = 0u;
    __syncwarp();
    const int beg = rowptr[i], end = rowptr[i + 1];
    int cnt = 0, repeat = 0;
    uint32_t m1 = 0, m2 = 0;                             // largest and second largest rank
    uint32_t s1 = 0xffffu, s2 = 0xffffu, s3 = 0xffffu;   // three smallest ranks >= head
    for (int e = beg + lane; e < end; e += 32) {
        const int32_t r = rank ? (int32_t)rank[BMU_IDX((uint32_t)colidx[e], D, status)] : colidx[e];
        if (r >= head) {
            ++cnt;
        } else {
            const uint32_t bit = 1u << (r & 31);
            repeat |= (atomicOr(&seen[warp][r >> 5], bit) & bit) != 0u;
        }
        if (ckeys) {
            const uint32_t rr = min((uint32_t)r, 0xfffeu);
            if (rr > m1) { m2 = m1; m1 = rr; } else if (rr > m2) { m2 = rr; }
            if (r >= head) plan_min3(s1, s2, s3, rr);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    repeat = __any_sync(0xffffffffu, repeat);
    const uint32_t len = repeat ? (uint32_t)(end - beg) : (uint32_t)cnt;
    if (lane == 0) key[i] = len;
    if (ckeys) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const uint32_t o1 = __shfl_xor_sync(0xffffffffu, m1, off);
            const uint32_t o2 = __shfl_xor_sync(0xffffffffu, m2, off);
            const uint32_t hi = max(m1, o1), lo = min(m1, o1);
            m2 = max(lo, max(m2, o2));
            m1 = hi;
            const uint32_t t1 = __shfl_xor_sync(0xffffffffu, s1, off);
            const uint32_t t2 = __shfl_xor_sync(0xffffffffu, s2, off);
            const uint32_t t3 = __shfl_xor_sync(0xffffffffu, s3, off);
            plan_min3(s1, s2, s3, t1);
            plan_min3(s1, s2, s3, t2);
            plan_min3(s1, s2, s3, t3);
        }
        if (lane == 0) {
            const u64 top = (u64)(uint32_t)(PLAN_BINS - 1 - min(len, (uint32_t)(PLAN_BINS - 1))) << 48;
            ckeys[i] = mode == 4 ? top | ((u64)s1 << 32) | ((u64)s2 << 16) | (u64)s3
                                 : top | ((u64)m1 << 32) | ((u64)m2 << 16) | (u64)s1;
            cvals[i] = (uint32_t)i;
        }
    }
}

// histogram of the sorting keys, and the largest key (aux[0]) so that the scan below can
// leave out the bins no document falls into
__global__ void plan_hist_kernel(const int32_t *__restrict__ rowptr,
                                 const uint32_t *__restrict__ key, int64_t N,
                                 uint32_t *__restrict__ hist, uint32_t *__restrict__ aux)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int len = 0;
    if (i < N) {
        len = min(key ? (int)key[i] : rowptr[i + 1] - rowptr[i], PLAN_BINS - 1);
        atomicAdd(hist + (PLAN_BINS - 1 - len), 1u);              // longest rows first
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) len = max(len, __shfl_xor_sync(0xffffffffu, len, off));
    if ((threadIdx.x & 31) == 0 && len > 0) atomicMax(aux, (uint32_t)len);
}

// Exclusive scan of the bin counters from the first bin that can hold a document (the one of
// the largest key, aux[0]) to the last.  One block of 32 warps: a warp owns a contiguous run
// of bins and walks it 32 bins at a time (coalesced loads, shuffle scan); first the runs'
// totals, then the scan proper with each run's offset.
__global__ void __launch_bounds__(1024)
plan_scan_bins_kernel(const uint32_t *__restrict__ hist, const uint32_t *__restrict__ aux,
                      uint32_t *__restrict__ cursor)
{
    __shared__ uint32_t s_tot[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lo = PLAN_BINS - 1 - (int)min(aux[0], (uint32_t)(PLAN_BINS - 1));
    const int per = ((PLAN_BINS - lo + 31) / 32 + 31) / 32 * 32;      // bins per warp, whole steps
    const int beg = lo + warp * per, end = min(beg + per, PLAN_BINS);
    uint32_t tot = 0;
    for (int b = beg + lane; b < end; b += 32) tot += hist[b];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, off);
    if (lane == 0) s_tot[warp] = tot;
    __syncthreads();
    uint32_t run = 0;
    for (int w = 0; w < warp; ++w) run += s_tot[w];
    for (int b0 = beg; b0 < end; b0 += 32) {
        const int b = b0 + lane;
        const uint32_t h = b < end ? hist[b] : 0u;
        uint32_t inc = h;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t v = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += v;
        }
        if (b < end) cursor[b] = run + inc - h;
        run += __shfl_sync(0xffffffffu, inc, 31);
    }
}

// a document's planned position, and the groups of 8 ids its row needs there (plus its closing
// sentinel group); ngroups[N] = 0 closes the array for the scan
__global__ void plan_scatter_kernel(const int32_t *__restrict__ rowptr,
                                    const uint32_t *__restrict__ key, int64_t N,
                                    uint32_t *__restrict__ cursor, int32_t *__restrict__ perm,
                                    uint32_t *__restrict__ ngroups)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) ngroups[N] = 0u;
    if (i >= N) return;
    const int row = rowptr[i + 1] - rowptr[i];
    const int len = key ? (int)key[i] : row;
    const int bin = PLAN_BINS - 1 - min(len, PLAN_BINS - 1);
    const uint32_t p = atomicAdd(cursor + bin, 1u);
    perm[p] = (int32_t)i;
    ngroups[p] = (uint32_t)((row + 7) / 8 + 1);
}

// Tile membership by content (Section 4.2: documents that share features are put in the same
// tile).  Sorting key of a document: its length key first -- tiles must stay exactly
// length-ordered -- then a few of its features, so that inside a run of equally long documents
// those with the same features lie next to each other.  Which features (ranks, or ids on a
// vocabulary labelled by frequency):
//   mode 3  the two rarest of the list, then the most frequent one at or above `head`;
//   mode 4  the three most frequent ones at or above `head` (the first three the gather visits).
// Either way the shared features sit at the same step of the lists of a tile (the front, or the
// back of equally long lists), so the loads of one step ask for the same row.  One warp per
// document.
__global__ void __launch_bounds__(256)
plan_cluster_key_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                        const uint16_t *__restrict__ rank, const uint32_t *__restrict__ len_key,
                        int64_t N, int32_t head, int mode, [[maybe_unused]] int64_t D,
                        [[maybe_unused]] uint32_t *status, u64 *__restrict__ keys,
                        uint32_t *__restrict__ vals)
{
    const int lane = threadIdx.x & 31;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= N) return;
    const int beg = rowptr[i], end = rowptr[i + 1];
    uint32_t m1 = 0, m2 = 0;                         // largest and second largest rank
    uint32_t s1 = 0xffffu, s2 = 0xffffu, s3 = 0xffffu;   // three smallest ranks >= head
    for (int e = beg + lane; e < end; e += 32) {
        const uint32_t f = (uint32_t)colidx[e];
        const uint32_t r = rank ? (uint32_t)rank[BMU_IDX(f, D, status)] : min(f, 0xfffeu);
        if (r > m1) { m2 = m1; m1 = r; } else if (r > m2) { m2 = r; }
        if (r >= (uint32_t)head) plan_min3(s1, s2, s3, r);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const uint32_t o1 = __shfl_xor_sync(0xffffffffu, m1, off);
        const uint32_t o2 = __shfl_xor_sync(0xffffffffu, m2, off);
        const uint32_t hi = max(m1, o1), lo = min(m1, o1);
        m2 = max(lo, max(m2, o2));
        m1 = hi;
        const uint32_t t1 = __shfl_xor_sync(0xffffffffu, s1, off);
        const uint32_t t2 = __shfl_xor_sync(0xffffffffu, s2, off);
        const uint32_t t3 = __shfl_xor_sync(0xffffffffu, s3, off);
        plan_min3(s1, s2, s3, t1);
        plan_min3(s1, s2, s3, t2);
        plan_min3(s1, s2, s3, t3);
    }
    if (lane == 0) {
        const int len = min(len_key ? (int)len_key[i] : end - beg, PLAN_BINS - 1);
        const u64 top = (u64)(uint32_t)(PLAN_BINS - 1 - len) << 48;
        keys[i] = mode == 4 ? top | ((u64)s1 << 32) | ((u64)s2 << 16) | (u64)s3
                            : top | ((u64)m1 << 32) | ((u64)m2 << 16) | (u64)s1;
        vals[i] = (uint32_t)i;
    }
}

// groups of 8 ids the row at planned position p needs (plus its closing sentinel group)
__global__ void plan_groups_kernel(const int32_t *__restrict__ rowptr,
                                   const int32_t *__restrict__ perm, int64_t N,
                                   uint32_t *__restrict__ ngroups)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p == 0) ngroups[N] = 0u;
    if (p >= N) return;
    const int32_t i = perm[p];
    ngroups[p] = (uint32_t)((rowptr[i + 1] - rowptr[i] + 7) / 8 + 1);
}

__global__ void plan_identity_kernel(const int32_t *__restrict__ rowptr, int64_t N,
                                     int32_t *__restrict__ perm, uint32_t *__restrict__ ngroups)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) ngroups[N] = 0u;
    if (i >= N) return;
    perm[i] = (int32_t)i;
    ngroups[i] = (uint32_t)((rowptr[i + 1] - rowptr[i] + 7) / 8 + 1);
}

// Size checks of the pass (one thread): the scanned offsets must fit the room that was
// reserved for what they index.  A failure sets bit 64 of the status word; the kernels that
// would write through those offsets, and every sweep, then do nothing.
__global__ void plan_check_kernel(const uint32_t *__restrict__ last_off, uint64_t room,
                                  uint32_t *__restrict__ status)
{
    if ((uint64_t)*last_off > room) atomicOr(status, PLAN_STATUS_OVERFLOW);
}

// One warp per planned document: writes its ascending 16-bit id list.  Rows that
// are not already in non-decreasing order are ordered by counting, for each id, the ids that
// must precede it (quadratic in the row length, rows are short).
__global__ void __launch_bounds__(256)
plan_fill_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                 const uint16_t *__restrict__ rank, const int32_t *__restrict__ perm,
                 const uint32_t *__restrict__ doc_off, int64_t N, uint16_t *__restrict__ ids16,
                 uint32_t *__restrict__ status, [[maybe_unused]] int64_t D)
{
    if (*status & PLAN_STATUS_OVERFLOW) return;
    // with a rank table the list holds ranks (ascending: most frequent first), not ids
#define BMU_PLAN_ID(e) (rank ? (int32_t)rank[BMU_IDX((uint32_t)row[e], D, status)] : row[e])
    const int lane = threadIdx.x & 31;
    const int64_t p = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (p >= N) return;
    const int32_t i = perm[p];
    const int beg = rowptr[i], len = rowptr[i + 1] - beg;
    const int32_t *row = colidx + beg;
    uint16_t *dst = ids16 + ((size_t)doc_off[p] + 1) * 8;          // group 0 is the global sentinel
    const int padded = ((len + 7) / 8 + 1) * 8;

    bool sorted = true;
    for (int e = lane; e + 1 < len; e += 32) sorted &= BMU_PLAN_ID(e) <= BMU_PLAN_ID(e + 1);
    sorted = __all_sync(0xffffffffu, sorted);
    if (sorted) {
        for (int e = lane; e < padded; e += 32) dst[e] = e < len ? (uint16_t)BMU_PLAN_ID(e) : 0xFFFFu;
    } else {
        for (int e = lane; e < padded; e += 32)
            if (e >= len) dst[e] = 0xFFFFu;
        for (int e = lane; e < len; e += 32) {
            const int32_t f = BMU_PLAN_ID(e);
            int pos = 0;
            for (int k = 0; k < len; ++k) {
                const int32_t g = BMU_PLAN_ID(k);
                pos += (g < f) || (g == f && k < e);
            }
            dst[pos] = (uint16_t)f;
        }
    }
#undef BMU_PLAN_ID
    if (p == 0 && lane < 8) ids16[lane] = 0xFFFFu;                  // global sentinel group
    if (p == N - 1 && lane < 16) dst[padded + lane] = 0xFFFFu;      // two groups of slack at the end
}

// ---- tiles of 8 documents -------------------------------------------------
// The ids below `head` (a multiple of 32, at most HEAD_ROWS_MAX) at the front of a document's
// ascending list become a bit mask of head / 32 words, and the list the sweep walks starts
// behind them.  A list that repeats one of them keeps multiset semantics by opting out (mask
// 0, nothing skipped): its ids all stay in the list.
// per tile: longest and shortest list behind the head (max | min << 16), and the head masks
// (head / 32 words per document, document-major).  One block per tile, one warp per document:
// the lanes read the front of the document's ascending list 32 ids at a time and set the mask
// bits in shared memory; a list that repeats a head id opts out (mask 0, nothing skipped).
__global__ void __launch_bounds__(256)
plan_tile_len_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ perm,
                     const uint32_t *__restrict__ doc_off, const uint16_t *__restrict__ ids16,
                     int64_t N, int64_t n_tiles, uint32_t head, uint32_t *__restrict__ tile_rows,
                     uint32_t *__restrict__ tile_len, uint32_t *__restrict__ tile_head)
{
    __shared__ uint32_t s_mask[8][HEAD_ROWS_MAX / 32];
    __shared__ uint32_t s_left[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t tile = blockIdx.x;
    const int64_t p = tile * 8 + warp;                                    // planned position
    const uint32_t words = head ? head / 32 : 1;
    for (uint32_t w = lane; w < words; w += 32) s_mask[warp][w] = 0u;
    __syncwarp();
    uint32_t len = 0, skip = 0;
    if (p < N) {
        const int32_t i = perm[p];
        len = (uint32_t)min(rowptr[i + 1] - rowptr[i], 65535);
        if (head) {
            const uint16_t *ids = ids16 + ((size_t)doc_off[p] + 1) * 8;
            bool repeat = false;
            for (uint32_t e0 = 0; e0 < len && e0 <= head; e0 += 32) {
                const uint32_t e = e0 + lane;
                const uint32_t f = (e < len && e <= head) ? ids[e] : 0xffffu;
                const bool in = f < head;
                if (in) {
                    const uint32_t bit = 1u << (f & 31u);
                    repeat |= (atomicOr(&s_mask[warp][f >> 5], bit) & bit) != 0u;
                }
                const uint32_t got = __ballot_sync(0xffffffffu, in);
                skip += (uint32_t)__popc(got);
                if (got != 0xffffffffu) break;                            // the list left the head
            }
            if (__any_sync(0xffffffffu, repeat)) {
                __syncwarp();
                for (uint32_t w = lane; w < words; w += 32) s_mask[warp][w] = 0u;
                skip = 0;
            }
        }
    }
    __syncwarp();
    {
        uint32_t *mask = tile_head + (size_t)p * words;
        for (uint32_t w = lane; w < words; w += 32) mask[w] = s_mask[warp][w];
    }
    if (lane == 0) s_left[warp] = len - skip;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t mx = 0, mn = 0xffffffffu;
        for (int t = 0; t < 8; ++t) { mx = max(mx, s_left[t]); mn = min(mn, s_left[t]); }
        tile_rows[tile] = mx;
        tile_len[tile] = mx | (mn << 16);
    }
}

// One warp per tile: row r of the matrix = the r-th id, in visiting order, of each of its
// 8 documents behind the head.  Visiting order: ascending, or (interleave) dealt alternately
// from the frequent and the rare half of the document's own list, so that at any moment a
// warp mixes loads that hit L1 with loads that go to L2.  The order depends on the document
// alone, never on its tile mates, so results do not depend on how tiles were cut.
__global__ void __launch_bounds__(256)
plan_tile_fill_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ perm,
                      const uint32_t *__restrict__ doc_off, const uint16_t *__restrict__ ids16,
                      const uint32_t *__restrict__ tile_len, const uint32_t *__restrict__ tile_off,
                      const uint32_t *__restrict__ tile_head, uint32_t head_words,
                      const uint16_t *__restrict__ feat_of_rank, int64_t N, int64_t n_tiles,
                      int interleave, uint4 *__restrict__ tile_ids,
                      uint32_t *__restrict__ status, [[maybe_unused]] int64_t D)
{
    if (*status & PLAN_STATUS_OVERFLOW) return;
    const int lane = threadIdx.x & 31;
    const int64_t tile = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (tile >= n_tiles) return;
    const uint32_t rows = tile_len[tile] & 0xffffu;
    const uint16_t *src[8];
    uint32_t len[8];
    for (int t = 0; t < 8; ++t) {
        const int64_t p = tile * 8 + t;
        len[t] = 0;
        src[t] = ids16;
        if (p < N) {
            const int32_t i = perm[p];
            uint32_t skip = 0;
            for (uint32_t w = 0; w < head_words; ++w)
                skip += (uint32_t)__popc(tile_head[(tile * 8 + t) * head_words + w]);
            len[t] = (uint32_t)min(rowptr[i + 1] - rowptr[i], 65535) - skip;
            src[t] = ids16 + ((size_t)doc_off[p] + 1) * 8 + skip;
        }
    }
    uint4 *dst = tile_ids + tile_off[tile];
    for (uint32_t r = lane; r < rows; r += 32) {
        uint32_t f[8];
        for (int t = 0; t < 8; ++t) {
            uint32_t e = r;
            if (interleave) e = (r & 1u) ? (len[t] + 1) / 2 + r / 2 : r / 2;
            f[t] = r < len[t] ? src[t][e] : 0xffffu;
            if (feat_of_rank && f[t] != 0xffffu)                              // rank -> row of W
                f[t] = feat_of_rank[BMU_IDX(f[t], D, status)];
        }
        dst[r] = make_uint4(f[0] | (f[1] << 16), f[2] | (f[3] << 16), f[4] | (f[5] << 16),
                            f[6] | (f[7] << 16));
    }
}

size_t plan_bytes(int64_t N, int64_t nnz, int head, int64_t D, int cluster, PlanLayout *l)
{
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    size_t off = 0;
    PlanLayout t;
    t.perm_off = off; off = up(off + (size_t)N * 4);
    t.docoff_off = off; off = up(off + (size_t)(N + 1) * 4);
    t.ngroups_off = off; off = up(off + (size_t)(N + 1) * 4);
    t.bins_off = off; off = up(off + (size_t)PLAN_BINS * 4 * 2 + 256);   // counters, cursors, aux
    t.id_groups_cap = (size_t)nnz / 8 + 2 * (size_t)N + 4;
    t.ids_off = off; off = up(off + t.id_groups_cap * 16);
    size_t scan_tmp = 0;
    cub::DeviceScan::ExclusiveSum(nullptr, scan_tmp, (uint32_t *)nullptr, (uint32_t *)nullptr,
                                  (int)(N + 1));
    t.scan_off = off; t.scan_bytes = scan_tmp; off = up(off + scan_tmp);
    // tiles: with documents exactly length-ordered, the sum over tiles of the longest row
    // is at most nnz / 8 plus the spread of lengths (< 65536)
    const size_t n_tiles = ((size_t)N + 7) / 8;
    t.tilelen_off = off; off = up(off + (n_tiles + 1) * 4);
    t.tilerows_off = off; off = up(off + (n_tiles + 1) * 4);
    t.tileoff_off = off; off = up(off + (n_tiles + 1) * 4);
    t.tilehead_off = off; off = up(off + n_tiles * 8 * 4 * (size_t)(head > 32 ? head / 32 : 1));
    t.tile_rows_cap = (size_t)nnz / 8 + 65536 + n_tiles;
    t.tileids_off = off; off = up(off + t.tile_rows_cap * 16);
    // frequency ranks of the features (dense head only): counts, sort buffers, the two tables
    t.rank_off = t.feat_off = t.fsort_off = t.fsort_tmp_off = off;
    t.fsort_tmp_bytes = 0;
    if (head > 0 && D > 0 && D <= 65535) {
        const size_t d4 = up((size_t)D * 4), d2 = up((size_t)D * 2);
        t.rank_off = off; off += d2;
        t.feat_off = off; off += d2;
        t.fsort_off = off; off += 4 * d4;            // counts, sorted counts, ids, sorted ids
        size_t tmp = 0;
        cub::DeviceRadixSort::SortPairsDescending(nullptr, tmp, (uint32_t *)nullptr, (uint32_t *)nullptr,
                                                  (uint32_t *)nullptr, (uint32_t *)nullptr, (int)D);
        t.fsort_tmp_off = off; t.fsort_tmp_bytes = tmp; off = up(off + tmp);
    }
    // ordering by content: 64-bit keys and document numbers, in and out, and the sort's scratch
    t.cluster_off = t.cluster_tmp_off = off;
    t.cluster_tmp_bytes = 0;
    if (cluster >= 3 && N > 0) {
        t.cluster_off = off; off = up(off + (size_t)N * 8 * 2 + (size_t)N * 4);
        size_t tmp = 0;
        cub::DeviceRadixSort::SortPairs(nullptr, tmp, (u64 *)nullptr, (u64 *)nullptr,
                                        (uint32_t *)nullptr, (uint32_t *)nullptr, (int)N);
        t.cluster_tmp_off = off; t.cluster_tmp_bytes = tmp; off = up(off + tmp);
    }
    t.total = off;
    if (l) *l = t;
    return off;
}

int launch_plan(const int32_t *rowptr, const int32_t *colidx, int64_t N, int64_t nnz,
                int order_by_length, int head, int relabel, int64_t D, char *ws, const PlanLayout &l,
                uint32_t *status, cudaStream_t s)
{
    // dense head: rank the features by how many documents list them, so that the head is the
    // `head` most frequent features whatever their ids
    const uint16_t *rank = nullptr;
    if (head > 0 && relabel != 2 && l.fsort_tmp_bytes > 0) {
        const size_t d4 = ((size_t)D * 4 + 255) / 256 * 256;
        uint32_t *count = reinterpret_cast<uint32_t *>(ws + l.fsort_off);
        uint32_t *count_sorted = reinterpret_cast<uint32_t *>(ws + l.fsort_off + d4);
        uint32_t *ids = reinterpret_cast<uint32_t *>(ws + l.fsort_off + 2 * d4);
        uint32_t *ids_sorted = reinterpret_cast<uint32_t *>(ws + l.fsort_off + 3 * d4);
        uint16_t *rank_of_feat = reinterpret_cast<uint16_t *>(ws + l.rank_off);
        uint16_t *feat_of_rank = reinterpret_cast<uint16_t *>(ws + l.feat_off);
        BMU_CUDA(cudaMemsetAsync(count, 0, (size_t)D * 4, s));
        if (nnz > 0) {
            const int32_t span = 32768;                   // 128 KB of shared-memory counters
            static bool configured[64];
            int dev = 0;
            BMU_CUDA(cudaGetDevice(&dev));
            if (dev >= 0 && dev < 64 && !configured[dev]) {
                BMU_CUDA(cudaFuncSetAttribute(plan_feat_hist_kernel,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, span * 4));
                configured[dev] = true;
            }
            for (int32_t lo = 0; lo < (int32_t)D; lo += span) {
                const int32_t hi = lo + span < (int32_t)D ? lo + span : (int32_t)D;
                { plan_feat_hist_kernel<<<148, 1024, (size_t)(hi - lo) * 4, s>>>(colidx, nnz, lo, hi, count); BMU_LAUNCHED(); }
            }
        }
        { plan_iota_kernel<<<(unsigned)((D + 255) / 256), 256, 0, s>>>((int32_t)D, ids); BMU_LAUNCHED(); }
        size_t tmp = l.fsort_tmp_bytes;
        BMU_CUDA(cub::DeviceRadixSort::SortPairsDescending(ws + l.fsort_tmp_off, tmp, count, count_sorted,
                                                           ids, ids_sorted, (int)D, 0, 32, s));
        // the decision word borrows the first counter of the length histogram (cleared below)
        uint32_t *keep_ids = reinterpret_cast<uint32_t *>(ws + l.bins_off);
        { plan_rank_decide_kernel<<<1, 1024, 0, s>>>(count, count_sorted, (int32_t)D, head, relabel == 1,
                                                   keep_ids); BMU_LAUNCHED(); }
        { plan_rank_tables_kernel<<<(unsigned)((D + 255) / 256), 256, 0, s>>>(ids_sorted, (int32_t)D,
                                                                            keep_ids, rank_of_feat,
                                                                            feat_of_rank); BMU_LAUNCHED(); }
        rank = rank_of_feat;
    }
    int32_t *perm = reinterpret_cast<int32_t *>(ws + l.perm_off);
    uint32_t *doc_off = reinterpret_cast<uint32_t *>(ws + l.docoff_off);
    uint32_t *ngroups = reinterpret_cast<uint32_t *>(ws + l.ngroups_off);
    uint32_t *hist = reinterpret_cast<uint32_t *>(ws + l.bins_off);
    uint32_t *cursor = hist + PLAN_BINS;
    uint32_t *aux = cursor + PLAN_BINS;              // [0] the largest sorting key
    uint16_t *ids16 = reinterpret_cast<uint16_t *>(ws + l.ids_off);
    const unsigned blocks = (unsigned)((N + 255) / 256);
    if (order_by_length) {
        // with a dense head the documents are ordered by what is left for the gather, so that
        // the documents of a tile finish their lists together (the key borrows the doc_off
        // array, which is written only by the scan after the scatter)
        const uint32_t *key = nullptr;
        const bool by_content = order_by_length >= 3 && l.cluster_tmp_bytes > 0;
        u64 *keys_in = reinterpret_cast<u64 *>(ws + l.cluster_off);
        u64 *keys_out = keys_in + N;
        uint32_t *vals_in = reinterpret_cast<uint32_t *>(keys_out + N);
        if (head > 0) {
            // length key and, if wanted, the content key in one pass over the rows
            { plan_key_kernel<<<(unsigned)((N * 32 + 255) / 256), 256, 0, s>>>(
                rowptr, colidx, rank, N, head, doc_off, D, status, order_by_length,
                by_content ? keys_in : nullptr, vals_in); BMU_LAUNCHED(); }
            key = doc_off;
        }
        // counters and the largest key in one clearing (the cursors in between are all written
        // or never read)
        BMU_CUDA(cudaMemsetAsync(hist, 0, (size_t)PLAN_BINS * 4 * 2 + 256, s));
        if (by_content) {
            // by length, then by the rarest features: one radix sort of (key, document) pairs
            if (head == 0)
                { plan_cluster_key_kernel<<<(unsigned)((N * 32 + 255) / 256), 256, 0, s>>>(
                    rowptr, colidx, rank, key, N, head, order_by_length, D, status, keys_in, vals_in); BMU_LAUNCHED(); }
            size_t ctmp = l.cluster_tmp_bytes;
            BMU_CUDA(cub::DeviceRadixSort::SortPairs(ws + l.cluster_tmp_off, ctmp, keys_in, keys_out,
                                                     vals_in, reinterpret_cast<uint32_t *>(perm),
                                                     (int)N, 0, 64, s));
            { plan_groups_kernel<<<blocks, 256, 0, s>>>(rowptr, perm, N, ngroups); BMU_LAUNCHED(); }
        } else {
            { plan_hist_kernel<<<blocks, 256, 0, s>>>(rowptr, key, N, hist, aux); BMU_LAUNCHED(); }
            { plan_scan_bins_kernel<<<1, 1024, 0, s>>>(hist, aux, cursor); BMU_LAUNCHED(); }
            { plan_scatter_kernel<<<blocks, 256, 0, s>>>(rowptr, key, N, cursor, perm, ngroups); BMU_LAUNCHED(); }
        }
    } else {
        { plan_identity_kernel<<<blocks, 256, 0, s>>>(rowptr, N, perm, ngroups); BMU_LAUNCHED(); }
    }
    size_t tmp = l.scan_bytes;
    BMU_CUDA(cub::DeviceScan::ExclusiveSum(ws + l.scan_off, tmp, ngroups, doc_off, (int)(N + 1), s));
    // group 0 is the global sentinel and two groups of slack close the lists
    { plan_check_kernel<<<1, 1, 0, s>>>(doc_off + N, (uint64_t)l.id_groups_cap - 3, status); BMU_LAUNCHED(); }
    { plan_fill_kernel<<<(unsigned)((N * 32 + 255) / 256), 256, 0, s>>>(rowptr, colidx, rank, perm,
                                                                       doc_off, N, ids16, status, D); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

int launch_plan_tiles(const int32_t *rowptr, int64_t N, int interleave, int head, int relabel,
                      int64_t D, char *ws, const PlanLayout &l, uint32_t *status, cudaStream_t s)
{
    const uint16_t *feat_of_rank = (head > 0 && relabel != 2 && l.fsort_tmp_bytes > 0)
                                       ? reinterpret_cast<const uint16_t *>(ws + l.feat_off) : nullptr;
    const int64_t n_tiles = (N + 7) / 8;
    const int32_t *perm = reinterpret_cast<const int32_t *>(ws + l.perm_off);
    const uint32_t *doc_off = reinterpret_cast<const uint32_t *>(ws + l.docoff_off);
    const uint16_t *ids16 = reinterpret_cast<const uint16_t *>(ws + l.ids_off);
    uint32_t *tile_len = reinterpret_cast<uint32_t *>(ws + l.tilelen_off);
    uint32_t *tile_rows = reinterpret_cast<uint32_t *>(ws + l.tilerows_off);
    uint32_t *tile_off = reinterpret_cast<uint32_t *>(ws + l.tileoff_off);
    uint4 *tile_ids = reinterpret_cast<uint4 *>(ws + l.tileids_off);
    uint32_t *tile_head = reinterpret_cast<uint32_t *>(ws + l.tilehead_off);
    { plan_tile_len_kernel<<<(unsigned)n_tiles, 256, 0, s>>>(
        rowptr, perm, doc_off, ids16, N, n_tiles, (uint32_t)head, tile_rows, tile_len, tile_head); BMU_LAUNCHED(); }
    BMU_CUDA(cudaMemsetAsync(tile_rows + n_tiles, 0, 4, s));
    size_t tmp = l.scan_bytes;
    BMU_CUDA(cub::DeviceScan::ExclusiveSum(ws + l.scan_off, tmp, tile_rows, tile_off,
                                           (int)(n_tiles + 1), s));
    // the sweeps read one row past a tile's last (the next row is fetched ahead)
    { plan_check_kernel<<<1, 1, 0, s>>>(tile_off + n_tiles, (uint64_t)l.tile_rows_cap - 1, status); BMU_LAUNCHED(); }
    { plan_tile_fill_kernel<<<(unsigned)((n_tiles * 32 + 255) / 256), 256, 0, s>>>(
        rowptr, perm, doc_off, ids16, tile_len, tile_off, tile_head,
        (uint32_t)(head ? head / 32 : 1), feat_of_rank, N, n_tiles, interleave, tile_ids, status, D); BMU_LAUNCHED(); }
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

}  // namespace bmu
