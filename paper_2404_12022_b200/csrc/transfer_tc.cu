// Hidden-transfer projection for many source rows at once (Section "Hidden Transfer"; the displayed
// equation of Section "Training stage"): out[B, k d] = h[B, d] . W[k d, d]^T on the tcgen05 tensor
// cores.  With a pseudo state per tree node the batch is B x T rows and the projection is a real matrix
// product; with a handful of rows it is a stream over W, and the same kernel serves both.
//
// One CTA per output tile of 128 source rows x bn weight rows (bn a multiple of 16, chosen so that the
// tiles about fill the GPU), features in steps of 64: TMA fills a ring of stages (h tile 16 KiB, W tile
// bn x 128 B, both with the 128-byte swizzle; rows and features past the end arrive as zeros), one thread
// issues the products into a TMEM accumulator (fp32), four warps read it back, round once and store.
// CTAs that share a W tile are neighbours in the grid, so the tile crosses DRAM once.
#include <cuda.h>

#include <cstdlib>

#include "attn_tc.cuh"

namespace ht {
namespace ttc {

using namespace tc;

constexpr int kBM = 128;                   // source rows per tile (UMMA M)
constexpr int kBK = 64;                    // features per stage: one swizzled 128-byte line per row
constexpr int kHBytes = kBM * kBK * 2;     // h tile of a stage
constexpr int kTThreads = 192;             // warps 0-3 read the accumulator, warp 4 TMA, warp 5 MMA
constexpr int kMaxStages = 24;
constexpr uint32_t kAccCols = 256;         // TMEM columns of one accumulator: bn <= 256

struct TParams {
    void *out;
    int B, R, d;            // source rows, weight rows (k d), features
    int bn, n_m, stages;    // weight rows per tile, 128-row tiles of the batch, ring depth
    int h_rows;             // rows of the h box: 128, or fewer when the whole batch is smaller
    int kc;                 // 64-feature chunks per stage (one TMA instruction per operand fetches them all)
    int mt;                 // 128-row tiles of h per CTA: 1, or 2 (two accumulators, one W tile for both)
    uint32_t stage_bytes;
};

struct TBars {
    unsigned long long full[kMaxStages], empty[kMaxStages], acc_full, mma_drain;
    int abort, wait_kcycles;           // the abort flag, and right behind it the limit of a wait (the waits read both as one 8-byte word)
    uint32_t tmem_base;
};

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, void *bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, void *bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// The feature axis is walked in steps of kc chunks of 64.  The matrices are described to the TMA unit as
// [chunk][row][64 features] (the chunk axis has the smallest stride after the features), so that one
// instruction per operand fetches the kc tiles of a step, each in the layout the tensor pipe reads
// (rows 128 bytes apart, 128-byte swizzle): a step costs about 0.3 us whatever its size, so few large
// steps stream faster than many small ones.  That view only has whole chunks; what is left after the
// last whole step goes chunk by chunk through plain [row][feature] maps, whose box may end past d and
// is zero-filled there.  With kc = 1 (large tiles: the ring needs its depth more) every step is such a one.
template <bool kBf16, int kMT>           // kMT = p.mt: 128-row tiles of h per CTA
__global__ void __launch_bounds__(kTThreads, 1)
transfer_tc_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w,
                   const __grid_constant__ CUtensorMap tm_h_tail, const __grid_constant__ CUtensorMap tm_w_tail, const TParams p) {
    // lets a kernel that is serialized programmatically behind this one set itself up while this one runs
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    TBars &bar = *reinterpret_cast<TBars *>(base + (size_t)p.stages * p.stage_bytes + (kBM * kMT - p.h_rows) * kBK * 2);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &bar.abort;
    const int m0 = ((int)blockIdx.x % p.n_m) * kBM * kMT, n0 = ((int)blockIdx.x / p.n_m) * p.bn;
    constexpr uint32_t acc_cols = kAccCols * (uint32_t)kMT;
    const int n_main = p.kc > 1 ? (p.d / kBK) / p.kc : 0;             // steps of kc whole chunks through the chunked view
    const int f_rest = n_main * p.kc * kBK;                           // first feature after them
    const int nk = n_main + (p.d - f_rest + kBK - 1) / kBK;           // + single chunks (the last one may be ragged)
    const uint32_t chunk_h = (uint32_t)p.h_rows * kBK * 2, chunk_w = (uint32_t)p.bn * kBK * 2;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.stages; ++i) { mbar_init(&bar.full[i], 1); mbar_init(&bar.empty[i], 1); }
        mbar_init(&bar.acc_full, 1);
        mbar_init(&bar.mma_drain, 1);
        bar.abort = 0;
        bar.wait_kcycles = tc::kWaitKcycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x == 32) {
        prefetch_tensormap(&tm_h);
        prefetch_tensormap(&tm_w);
        if (nk > n_main) {
            prefetch_tensormap(&tm_h_tail);
            prefetch_tensormap(&tm_w_tail);
        }
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bar.tmem_base)), "r"((uint32_t)acc_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar.tmem_base;

    if (warp == 4) {
        // ------------------------------- TMA producer -------------------------------
        if (lane == 0) {
            int issued = 0, slot = 0, use = 0;         // slot and round of the ring, kept by counting (no division per step)
            for (int ks = 0; ks < nk; ++ks, ++slot) {
                if (slot == p.stages) { slot = 0; ++use; }
                if (use > 0 && !mbar_wait_quick(smem_u32(&bar.empty[slot]), (use - 1) & 1, abort_flag)) break;
                unsigned char *a = base + (size_t)slot * p.stage_bytes;
                if (ks < n_main) {
                    mbar_expect_tx(&bar.full[slot], (chunk_h + chunk_w) * p.kc);
                    tma_load_3d(a, &tm_h, &bar.full[slot], 0, m0, ks * p.kc);
                    tma_load_3d(a + chunk_h * p.kc, &tm_w, &bar.full[slot], 0, n0, ks * p.kc);
                } else {
                    mbar_expect_tx(&bar.full[slot], chunk_h + chunk_w);
                    tma_load_2d(a, &tm_h_tail, &bar.full[slot], f_rest + (ks - n_main) * kBK, m0);
                    tma_load_2d(a + chunk_h * p.kc, &tm_w_tail, &bar.full[slot], f_rest + (ks - n_main) * kBK, n0);
                }
                ++issued;
            }
            if (*abort_flag) {
                // every copy issued here must have landed before the CTA exits
                for (int e = max(0, issued - p.stages); e < issued; ++e)
                    mbar_wait(&bar.full[e % p.stages], (e / p.stages) & 1, abort_flag, false);
            }
        }
    } else if (warp == 5) {
        // ------------------------------- MMA issuer -------------------------------
        if (lane == 0) {
            const uint32_t idesc = instr_desc(kBf16, 0, (uint32_t)p.bn);
            const uint64_t a_desc0 = smem_desc(smem_u32(base), 1, 1024 >> 4), b_desc0 = a_desc0;
            const uint32_t stage16 = p.stage_bytes >> 4, h16 = chunk_h >> 4, w16 = chunk_w >> 4;
            const bool second = kMT > 1 && m0 + kBM < p.B;
            bool all = true;
            int slot = 0, use = 0;
            for (int ks = 0; ks < nk; ++ks, ++slot) {
                if (slot == p.stages) { slot = 0; ++use; }
                if (!mbar_wait_quick(smem_u32(&bar.full[slot]), use & 1, abort_flag)) { all = false; break; }
                tc_fence_after();
                // The descriptors differ in their address field only (16-byte units in the low bits, never
                // carrying out of it inside this CTA's shared memory): one template each, then additions.
                const uint32_t a16 = (uint32_t)slot * stage16, b16 = a16 + h16 * p.kc;
                const int chunks = ks < n_main ? p.kc : 1;
                for (int c = 0; c < chunks; ++c) {
#pragma unroll
                    for (int i = 0; i < kMT; ++i) {            // a second 128-row tile of h, if it has rows at all
                        if (i > 0 && !second) break;
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)  // 16 features = 32 bytes inside the swizzled line
                            mma_ss(tmem + i * kAccCols, a_desc0 + (a16 + c * h16 + i * (kHBytes >> 4) + kk * 2),
                                   b_desc0 + (b16 + c * w16 + kk * 2), idesc, (ks | c | kk) != 0 ? 1u : 0u);
                    }
                }
                tc_commit(&bar.empty[slot]);
            }
            if (all) tc_commit(&bar.acc_full);
            // no tensor-core operation of this CTA may be in flight when its TMEM is freed
            tc_commit(&bar.mma_drain);
            mbar_wait(&bar.mma_drain, 0, abort_flag, false);
        }
    } else {
        // ------------------------------- accumulator -> out -------------------------------
        const bool waited = mbar_wait(&bar.acc_full, 0, abort_flag);
        const bool ok = __all_sync(0xFFFFFFFFu, waited);
        tc_fence_after();
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
#pragma unroll
        for (int i = 0; i < kMT; ++i) {
            const int row = m0 + i * kBM + (int)threadIdx.x;   // TMEM lane = source row of the tile
            if (m0 + i * kBM >= p.B) break;
            unsigned char *dst_row = static_cast<unsigned char *>(p.out) + ((size_t)min(row, p.B - 1) * p.R + n0) * 2;
#pragma unroll 1
            for (int c = 0; c < p.bn; c += 32) {
                float v[32];
                if (ok) {
                    tmem_ld32(tmem + lane_base + i * kAccCols + c, v);
                    tmem_ld_wait();
                } else {
                    // a wait ran out: the tile's results are marked as not-a-number instead of left stale
#pragma unroll
                    for (int x = 0; x < 32; ++x) v[x] = __int_as_float(0x7FC00000);
                }
                if (row < p.B) {
#pragma unroll
                    for (int x = 0; x < 32; x += 8) {
                        if (c + x < p.bn && n0 + c + x < p.R)  // R and n0 are multiples of 8: a group of 8 is in or out as a whole
                            *reinterpret_cast<uint4 *>(dst_row + (c + x) * 2) =
                                make_uint4(pack2<kBf16>(v[x], v[x + 1]), pack2<kBf16>(v[x + 2], v[x + 3]),
                                           pack2<kBf16>(v[x + 4], v[x + 5]), pack2<kBf16>(v[x + 6], v[x + 7]));
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)acc_cols) : "memory");
    }
}

}  // namespace ttc

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn2)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn2 encode_fn2() {
    static EncodeTiledFn2 fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn2>(ptr);
    }
    return fn;
}

// Row-major [rows, d] 16-bit matrix, boxes of 64 features x box_rows rows, 128-byte swizzle.
static int make_map_2d(CUtensorMap *map, const void *base, int dtype, int rows, int d, int box_rows) {
    EncodeTiledFn2 fn = encode_fn2();
    if (!fn) return fail(HT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {(cuuint32_t)ttc::kBK, (cuuint32_t)box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = fn(map, dtype == HT_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
                          const_cast<void *>(base), dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HT_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    return HT_OK;
}

// The same matrix as [chunks of 64 features][rows][64 features]: boxes of 64 x box_rows x kc.
static int make_map_chunked(CUtensorMap *map, const void *base, int dtype, int rows, int d, int box_rows, int kc) {
    EncodeTiledFn2 fn = encode_fn2();
    if (!fn) return fail(HT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint64_t dims[3] = {(cuuint64_t)ttc::kBK, (cuuint64_t)rows, (cuuint64_t)(d / ttc::kBK)};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)ttc::kBK * 2};
    const cuuint32_t box[3] = {(cuuint32_t)ttc::kBK, (cuuint32_t)box_rows, (cuuint32_t)kc};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    const CUresult r = fn(map, dtype == HT_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                          const_cast<void *>(base), dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HT_ERR_CUDA, "cuTensorMapEncodeTiled (chunked view) failed with %d", (int)r);
    return HT_OK;
}

static int device_sms() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Source-row tiles of 128 per CTA: two (two accumulators fed by one W tile) once there are enough rows -- a
// third less traffic from L2 into shared memory per product, which is what bounds the large shapes.
static int transfer_tc_mt(int B) { return B > 3 * ttc::kBM ? 2 : 1; }

// Weight rows per tile.  While one wave of CTAs can hold all tiles, the tiles are made just small enough to
// give every SM one (the stream over W is spread over the whole GPU).  Beyond that the tiles run in waves,
// and a CTA's time follows the bytes it stages per step (source rows + weight rows): among the wave counts
// that a tile of at most 256 rows can meet, the one with the least waves x (source rows + bn) is taken --
// 512 x 20480: 286 tiles of 144 in two full waves instead of 160 tiles of 256 in a full and a thin one.
int transfer_tc_tile(int B, int R, int sms) {
    const int mt = transfer_tc_mt(B);
    const int rows = ttc::kBM * mt;
    const int n_m = (B + rows - 1) / rows;
    int best_bn = 256;
    long long best = ((((long long)(R + 255) / 256) * n_m + sms - 1) / sms) * (rows + 256);
    for (int w = 1; w <= 16; ++w) {
        const int slots = (int)((long long)sms * w / n_m);
        if (slots < 1) continue;
        const int bn = ((R + slots - 1) / slots + 15) / 16 * 16;
        if (bn > 256) continue;
        if (w == 1) return bn;
        const long long cost = (long long)w * (rows + bn);
        if (cost < best) { best = cost; best_bn = bn; }
    }
    return best_bn;
}

bool transfer_tc_applicable(int B, int k, int d, int dtype) {
    return (dtype == HT_F16 || dtype == HT_BF16) && d % 8 == 0 && B > 0 && (long long)k * d > 0;
}

int launch_transfer_tc(const void *h, const void *W, void *out, int B, int k, int d, int dtype, cudaStream_t s) {
    const int R = k * d;
    ttc::TParams p;
    p.out = out;
    p.B = B; p.R = R; p.d = d;
    p.bn = transfer_tc_tile(B, R, device_sms());
    p.mt = transfer_tc_mt(B);
    p.n_m = (B + ttc::kBM * p.mt - 1) / (ttc::kBM * p.mt);
    // Fewer than 128 source rows: only those are fetched and held.  The tensor pipe still reads 128 rows
    // from the h tile's address on, i.e. on into the W tile and the next stage (the ring is followed by that
    // much padding); row m of the product depends on row m of h alone, and rows past B are not stored.
    p.h_rows = p.mt == 2 ? 2 * ttc::kBM : (B >= ttc::kBM ? ttc::kBM : (B + 7) / 8 * 8);
    const int n_full = d / ttc::kBK;
    const size_t pad = (size_t)(ttc::kBM * p.mt - p.h_rows) * ttc::kBK * 2;
    const size_t budget = 227 * 1024 - 1024 - pad - sizeof(ttc::TBars) - 64;
    const size_t chunk_bytes = (size_t)(p.h_rows + p.bn) * ttc::kBK * 2;
    // Chunks per step: as many as leave two stages, for the streaming shapes (one 128-row tile of h, W tiles
    // well below the maximum); one for the others.
    p.kc = 1;
    if (p.mt == 1 && p.n_m == 1 && p.bn < 192)
        for (int kc = 8; kc > 1; kc /= 2)
            if (kc <= n_full && chunk_bytes * kc * 2 <= budget) { p.kc = kc; break; }
    p.stage_bytes = (uint32_t)((p.h_rows + p.bn) * ttc::kBK * 2 * p.kc);
    int stages = (int)(budget / p.stage_bytes);
    stages = stages > ttc::kMaxStages ? ttc::kMaxStages : stages;
    const int n_main = p.kc > 1 ? n_full / p.kc : 0;
    const int nk = n_main + (d - n_main * p.kc * ttc::kBK + ttc::kBK - 1) / ttc::kBK;
    if (stages > nk) stages = nk;
    p.stages = stages;
    const size_t smem = 1024 + (size_t)stages * p.stage_bytes + pad + sizeof(ttc::TBars);

    CUtensorMap tm_h, tm_w, tm_h_tail, tm_w_tail;
    int rc = make_map_2d(&tm_h_tail, h, dtype, B, d, p.h_rows);
    if (rc != HT_OK) return rc;
    rc = make_map_2d(&tm_w_tail, W, dtype, R, d, p.bn);
    if (rc != HT_OK) return rc;
    if (p.kc > 1) {
        rc = make_map_chunked(&tm_h, h, dtype, B, d, p.h_rows, p.kc);
        if (rc != HT_OK) return rc;
        rc = make_map_chunked(&tm_w, W, dtype, R, d, p.bn, p.kc);
        if (rc != HT_OK) return rc;
    } else {
        tm_h = tm_h_tail;      // never used: every step is a single chunk
        tm_w = tm_w_tail;
    }

    typedef void (*Fn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const ttc::TParams);
    const Fn fns[4] = {ttc::transfer_tc_kernel<false, 1>, ttc::transfer_tc_kernel<true, 1>, ttc::transfer_tc_kernel<false, 2>,
                       ttc::transfer_tc_kernel<true, 2>};
    static bool attr_done[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (!(dev >= 0 && dev < 64 && attr_done[dev])) {
        for (int i = 0; i < 4 && e == cudaSuccess; ++i)
            e = cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
    const long long n_n = (R + p.bn - 1) / p.bn;
    const long long grid = n_n * p.n_m;
    if (grid > 0x7FFFFFFFll) return fail(HT_ERR_INVALID_ARG, "ht_transfer: too many tiles");
    fns[(dtype == HT_BF16 ? 1 : 0) + (p.mt == 2 ? 2 : 0)]<<<(unsigned)grid, ttc::kTThreads, smem, s>>>(tm_h, tm_w, tm_h_tail, tm_w_tail, p);
    return check_launch("ht_transfer");
}

}  // namespace ht
