// Staged gather-accumulate sweep, one document per lane (Section 3 and the
// levers of Section 4, re-cut for B200).
//
// A thread block owns a tile of 992 documents: each of the 31 x 32 consumer
// lanes carries ONE document and keeps its 32 partial sums for the current
// slab of 32 neurons in registers.  The 32nd warp is the producer: for every
// slab it streams the slab's 128-byte segment of EVERY codebook row, feature 0
// to D-1, through a ring of shared-memory stages with 2-D tensor (TMA) box
// copies -- 32 floats x R rows per instruction -- so each staged row is shared
// by all 992 documents of the tile and L2 is read once per tile, not once per
// document.  A lane walks its own ascending feature list (16-bit ids, eight per
// 128-bit load, prepared by the tiling pass) and, for every id that lies in the
// stages already landed, adds that row's 128 bytes into its sums with eight
// 128-bit shared-memory loads.  Lane l reads the row's 16-byte pieces in the
// order q ^ (l & 7), q = 0..7, so the eight lanes of a quarter-warp always hit
// eight different bank groups although they read eight different rows.  After
// the last stage of a slab the lane turns sums into distances n_j - 2 s_ij and
// keeps its running (distance, index) minimum -- no shuffle is needed, the
// lane owns the document -- and after the last slab of the chunk it merges
// into the per-document state.  Full/empty mbarriers order producer and
// consumers; every wait is bounded and reports through `status`.
#include "common.cuh"

#include <cuda.h>
#include <math_constants.h>

namespace bmu {

static const int LW = 32;                    // warps per block
static const int LCW = LW - 1;               // consumer warps
static const int GROUP_DOCS = LCW * 32;      // documents per tile
static const int ROW_BYTES = 128;            // 32 neurons of one feature
static const uint32_t WAIT_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// bounded wait for the phase with the given parity; false = gave up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < WAIT_LIMIT; ++spin) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; "
                     "selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap *tm, int x, int y,
                                              uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void lds_2x64(uint32_t addr, u64 &a, u64 &b)
{
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr));
}

template <int R, int NS>
__global__ void __launch_bounds__(LW * 32, 1)
sweep_lanes_kernel(const __grid_constant__ CUtensorMap tm, const LanesArgs a, const int n_groups)
{
    static_assert((NS & (NS - 1)) == 0, "stage count must be a power of two");
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char *ring = smem;
    unsigned long long *full = reinterpret_cast<unsigned long long *>(smem + (size_t)R * NS * ROW_BYTES);
    unsigned long long *empty = full + NS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sps = (a.D + R - 1) / R;                       // stages per slab pass
    const int n_slabs = (a.j_hi - a.j_lo + 31) / 32;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) {
            mbar_init(smem_addr(full + i), 1);
            mbar_init(smem_addr(empty + i), LCW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == LCW) {
        // ---------------- producer: one thread streams every row of every slab
        if (lane != 0) return;
        uint32_t k = 0;
        for (int g = blockIdx.x; g < n_groups; g += gridDim.x)
            for (int sl = 0; sl < n_slabs; ++sl) {
                const int x = a.j_lo + sl * 32;
                for (int s = 0; s < sps; ++s, ++k) {
                    const uint32_t slot = k & (NS - 1);
                    if (k >= NS && !mbar_wait(smem_addr(empty + slot), ((k / NS) - 1) & 1)) {
                        atomicOr(a.status, 1u);
                        return;
                    }
                    mbar_expect_tx(smem_addr(full + slot), R * ROW_BYTES);
                    tma_load_rows(smem_addr(ring + (size_t)slot * R * ROW_BYTES), &tm, x, s * R,
                                  smem_addr(full + slot));
                }
            }
        return;
    }

    // ---------------- consumers: one document per lane
    const uint32_t lanebits = (uint32_t)(lane & 7) << 4;
    const uint32_t ring_u32 = smem_addr(ring);
    uint32_t k = 0;
    for (int g = blockIdx.x; g < n_groups; g += gridDim.x) {
        const int64_t p = (int64_t)g * GROUP_DOCS + warp * 32 + lane;
        const bool valid = p < a.N;
        const int32_t orig = valid ? __ldg(a.perm + p) : 0;
        const uint4 *gp = a.ids + (valid ? (size_t)__ldg(a.doc_off + p) + 1 : 0);
        float best = CUDART_INF_F;
        int bidx = 0x7fffffff;

        for (int sl = 0; sl < n_slabs; ++sl) {
            const int j0 = a.j_lo + sl * 32;
            u64 acc[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = 0ull;
            // this lane's id stream: 8 ids in (x, y), the next 8 prefetched in (nx, ny)
            uint4 t = __ldg(gp);
            u64 x = ((u64)t.y << 32) | t.x, y = ((u64)t.w << 32) | t.z;
            t = __ldg(gp + 1);
            u64 nx = ((u64)t.y << 32) | t.x, ny = ((u64)t.w << 32) | t.z;
            int gnext = 2, cnt = 8;

            for (int s = 0; s < sps; ++s, ++k) {
                const uint32_t slot = k & (NS - 1);
                if (!mbar_wait(smem_addr(full + slot), (k / NS) & 1)) {
                    atomicOr(a.status, 2u);
                    return;
                }
                const uint32_t f_head = (uint32_t)(s + 1) * R;
                // row f of this stage sits at ring + (slot*R + f - s*R) * 128
                const uint32_t stage_addr =
                    ring_u32 + (uint32_t)(((int)slot - s) * R * ROW_BYTES) + lanebits;
                while (true) {
                    const uint32_t cur = (uint32_t)x & 0xffffu;
                    const bool go = cur < f_head;
                    if (!__any_sync(0xffffffffu, go)) break;
                    if (go) {
                        const uint32_t ra = stage_addr + (cur << 7);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            u64 w0, w1;
                            lds_2x64(ra ^ (uint32_t)(q << 4), w0, w1);
                            add2(acc[2 * q], w0);
                            add2(acc[2 * q + 1], w1);
                        }
                        x = (x >> 16) | (y << 48);
                        y >>= 16;
                        if (--cnt == 0) {
                            x = nx; y = ny; cnt = 8;
                            t = __ldg(gp + gnext);
                            nx = ((u64)t.y << 32) | t.x; ny = ((u64)t.w << 32) | t.z;
                            ++gnext;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_addr(empty + slot));
            }

            // distances of this slab; this lane's piece q holds neurons j0 + 4*((lane&7)^q) ..+3
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int j = j0 + 4 * ((lane & 7) ^ q);
                if (j < a.j_hi) {
                    const float4 n = __ldg(reinterpret_cast<const float4 *>(a.norms + j));
                    const float s4[4] = {lo_f(acc[2 * q]), hi_f(acc[2 * q]), lo_f(acc[2 * q + 1]),
                                         hi_f(acc[2 * q + 1])};
                    const float n4[4] = {n.x, n.y, n.z, n.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float d = fmaf(-2.f, s4[e], n4[e]);
                        if (d < best || (d == best && j + e < bidx)) { best = d; bidx = j + e; }
                    }
                }
            }
        }

        if (valid) {
            u64 key = make_key(best, bidx);
            if (!a.first) {
                const u64 old = a.state[orig];
                if (old < key) key = old;
            }
            a.state[orig] = key;
        }
    }
}

// A wait that cannot succeed: one mbarrier that nothing ever arrives on.  It shows
// that a wait which runs out leaves the kernel through the status word and the
// context usable (no trap, no endless loop); the limit here is short on purpose.
__global__ void wait_timeout_selftest_kernel(uint32_t *status)
{
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_addr(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = false;
    for (uint32_t spin = 0; spin < 4096u && !ok; ++spin) {
        uint32_t r;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; "
                     "selp.u32 %0, 1, 0, p; }"
                     : "=r"(r) : "r"(smem_addr(&bar)), "r"(0u) : "memory");
        ok = r != 0;
    }
    if (!ok && threadIdx.x == 0) atomicOr(status, 2u);
}

int launch_wait_timeout_selftest(uint32_t *status, cudaStream_t s)
{
    wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(status);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int make_codebook_tensor_map(const float *W, int64_t D, int64_t M, int rows_per_stage,
                             void *tensor_map_out)
{
    static EncodeTiledFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        BMU_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) {
            set_error("cuTensorMapEncodeTiled is not available in this driver");
            return BMU_ERR_CUDA;
        }
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    const cuuint64_t gdim[2] = {(cuuint64_t)M, (cuuint64_t)D};
    const cuuint64_t gstride[1] = {(cuuint64_t)M * 4};
    const cuuint32_t box[2] = {32, (cuuint32_t)rows_per_stage};
    const cuuint32_t estride[2] = {1, 1};
    const CUresult r = encode(static_cast<CUtensorMap *>(tensor_map_out),
                              CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(W), gdim,
                              gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with %d", (int)r);
        return BMU_ERR_CUDA;
    }
    return BMU_OK;
}

template <int R, int NS>
static int launch_rn(const CUtensorMap &tm, const LanesArgs &a, int n_groups, int sms,
                     cudaStream_t s)
{
    const size_t smem = (size_t)R * NS * ROW_BYTES + 2 * NS * sizeof(unsigned long long);
    static bool configured = false;
    if (!configured) {
        BMU_CUDA(cudaFuncSetAttribute(sweep_lanes_kernel<R, NS>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = true;
    }
    const int grid = n_groups < sms ? n_groups : sms;
    sweep_lanes_kernel<R, NS><<<grid, LW * 32, smem, s>>>(tm, a, n_groups);
    BMU_CUDA(cudaGetLastError());
    return BMU_OK;
}

static int lanes_rows_per_stage(const bmu_opts &o) { return o.stage_rows ? o.stage_rows : 256; }

int launch_sweep_lanes(const void *tensor_map, const LanesArgs &a, const bmu_opts &o,
                       cudaStream_t s)
{
    if (a.N == 0 || a.j_lo >= a.j_hi) return BMU_OK;
    int dev = 0, sms = 0;
    BMU_CUDA(cudaGetDevice(&dev));
    BMU_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int n_groups = (int)((a.N + GROUP_DOCS - 1) / GROUP_DOCS);
    const CUtensorMap &tm = *static_cast<const CUtensorMap *>(tensor_map);
    const int R = lanes_rows_per_stage(o), NS = o.stages ? o.stages : 4;
#define BMU_CASE(r, ns) if (R == r && NS == ns) return launch_rn<r, ns>(tm, a, n_groups, sms, s);
    BMU_CASE(256, 4) BMU_CASE(128, 8) BMU_CASE(256, 2) BMU_CASE(128, 4) BMU_CASE(64, 16)
#undef BMU_CASE
    set_error("staged kernel: (stage_rows, stages) must be one of (256,4) (128,8) (256,2) (128,4) (64,16)");
    return BMU_ERR_INVALID_ARG;
}

}  // namespace bmu
