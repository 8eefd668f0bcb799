// Hidden-transfer projection  h~ = W^i . h  (Section "Training stage", displayed equation).
//
// Shape of the work: k*d output rows, each a dot product of one row of W (d elements,
// read exactly once from HBM) with B hidden vectors (tiny, L1/L2 resident).  The kernel
// is a weight stream: arithmetic intensity is B flop per weight byte, far below the
// ridge for the batch sizes of decoding, so the design goal is 16-byte coalesced loads
// with enough of them in flight.  (Up to 16 source rows per pass: this file.  More rows,
// 16-bit types: the tcgen05 kernel of transfer_tc.cu.)
//
// Every warp of a grid that just fills the GPU owns an equal, contiguous share of the k*d rows of
// the flattened [k*d, d] weight and walks it R rows at a time.  Its lanes stride over the input
// features in 16-byte vectors; U such steps (R x U independent 16-byte loads per lane) are issued
// before the first is used, which keeps over 100 KB of weight in flight per SM -- what a stream
// needs to run at memory speed.  R x BT fp32 accumulators per lane, reduced with shuffles at
// the end of a row group.  The R rows share each loaded h vector (h is small and cache resident).
//
// 16-bit inputs take a second kernel: unpacking bf16 / fp16 and multiplying on the fp32 ALUs costs
// about 15 issue slots per weight element, which caps the stream near 3 TB/s.  The warp-level
// tensor-core instruction (m16n8k16, fp32 accumulate) consumes the 16-bit words as loaded.  The
// order of the contraction index is free as long as both operands agree, so each lane loads
// plain 16-byte vectors (8 consecutive features of one weight row, the same 8 features of one
// batch row) and the pairs of those vectors are dealt to the instruction's k slots in place:
// no shuffles, no shared memory.  (tcgen05 would stage both operands through shared memory for
// an M = 128 tile; with 4 to 16 batch columns this skinny product gains nothing from it.)
#include <cstdlib>
#include <cstring>

#include "ht_common.cuh"

namespace ht {

constexpr int kTransferBlocksPerSm = 4;

template <typename T, int R, int BT, int U>
__global__ void __launch_bounds__(128, kTransferBlocksPerSm)
transfer_kernel(const T *__restrict__ h, const T *__restrict__ W, T *__restrict__ out,
                int rows_total, int d, int b0, int nb) {
    // lets a kernel that is serialized programmatically behind this one set itself up while this one runs
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int VE = Vec16<T>::n;
    constexpr int BC = BT < 4 ? BT : 4;              // batch columns handled per pass over the loaded weights
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * 4 + (threadIdx.x >> 5), n_warps = (long long)gridDim.x * 4;
    const int r_begin = (int)(warp * rows_total / n_warps), r_end = (int)((warp + 1) * rows_total / n_warps);

    for (int row0 = r_begin; row0 < r_end; row0 += R) {
        float acc[R][BT];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int b = 0; b < BT; ++b) acc[r][b] = 0.f;

        for (int c0 = lane * VE; c0 < d; c0 += 32 * VE * U) {
            uint4 wraw[U][R];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int c = c0 + u * 32 * VE;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int row = min(row0 + r, r_end - 1);      // a short last group repeats its last row
                    wraw[u][r] = c < d ? ld_nc16(W + (size_t)row * d + c) : make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int c = min(c0 + u * 32 * VE, d - VE);       // past the end the weights above are zero
                float wf[R][VE];
#pragma unroll
                for (int r = 0; r < R; ++r) unpack16<T>(wraw[u][r], wf[r]);
#pragma unroll
                for (int bb = 0; bb < BT; bb += BC) {
                    float hv[BC][VE];
#pragma unroll
                    for (int b = 0; b < BC; ++b) {
                        const int bi = min(bb + b, nb - 1);        // unused batch columns repeat the last one
                        unpack16<T>(*reinterpret_cast<const uint4 *>(h + (size_t)(b0 + bi) * d + c), hv[b]);
                    }
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int b = 0; b < BC; ++b)
#pragma unroll
                            for (int e = 0; e < VE; ++e) acc[r][bb + b] = fmaf(wf[r][e], hv[b][e], acc[r][bb + b]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                float v = acc[r][b];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (lane == 0 && b < nb && row0 + r < r_end)
                    out[(size_t)(b0 + b) * rows_total + row0 + r] = from_float<T>(v);
            }
    }
}

static int transfer_grid(int rows_total, int R) {
    static int sms[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    if (!sms[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        sms[dev] = n;
    }
    const int full = sms[dev] * kTransferBlocksPerSm;              // every CTA resident at once
    const int need = (rows_total + 4 * R - 1) / (4 * R);           // at least one row group per warp
    return need < full ? need : full;
}

template <typename T, int R, int BT, int U>
static int launch_one(const void *h, const void *W, void *out, int rows_total, int d, int b0, int nb,
                      cudaStream_t s) {
    transfer_kernel<T, R, BT, U><<<transfer_grid(rows_total, R), 128, 0, s>>>(
        static_cast<const T *>(h), static_cast<const T *>(W), static_cast<T *>(out), rows_total, d, b0, nb);
    return check_launch("ht_transfer");
}

template <typename T>
static int launch_typed(const void *h, const void *W, void *out, int B, int k, int d, cudaStream_t s) {
    const int rows_total = k * d;
    // out is [B, k*d]: batch b writes at out + b*rows_total, so batch slices are independent.
    for (int b0 = 0; b0 < B; b0 += 16) {
        const int nb = min(16, B - b0);
        int rc;
        if (nb == 1) rc = launch_one<T, 4, 1, 4>(h, W, out, rows_total, d, b0, nb, s);
        else if (nb == 2) rc = launch_one<T, 4, 2, 4>(h, W, out, rows_total, d, b0, nb, s);
        else if (nb <= 4) rc = launch_one<T, 4, 4, 4>(h, W, out, rows_total, d, b0, nb, s);
        else if (nb <= 8) rc = launch_one<T, 2, 8, 4>(h, W, out, rows_total, d, b0, nb, s);
        else rc = launch_one<T, 2, 16, 4>(h, W, out, rows_total, d, b0, nb, s);
        if (rc != HT_OK) return rc;
    }
    return HT_OK;
}


// ---------------------------------------------------------------------------------------
// 16-bit inputs: m16n8k16 tensor-core products on the words as loaded
// ---------------------------------------------------------------------------------------
template <typename T> struct MmaOp;
template <> struct MmaOp<__half> {
    static __device__ __forceinline__ void run(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};
template <> struct MmaOp<__nv_bfloat16> {
    static __device__ __forceinline__ void run(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};

// Work items are (group of 16 weight rows, one of S equal feature ranges); S = 1, 2 or 4 is chosen on
// the host so that the items about fill the GPU's warp slots (with few row groups a warp per group
// would leave most slots, and most of the memory system, idle).  A warp owns an equal, contiguous
// share of the items; the S warps of a group sit in one block and the first of them adds up the
// partial sums through shared memory.  Lane (g, t) = (lane / 4, lane % 4) loads features
// [f + 8 t, f + 8 t + 8) of rows g and g + 8 of the group and of batch row g of each 8-column batch
// tile; words 0 / 1 of those vectors fill k slots (2t, 2t+1) / (2t+8, 2t+9) of one instruction, words
// 2 / 3 those of a second one.  U steps of 32 features are loaded before the first is used.  The
// accumulator fragment holds rows g, g + 8 and batch columns 2t, 2t + 1.
template <typename T, int NB, int U, bool kSplit>
__global__ void __launch_bounds__(128, kTransferBlocksPerSm)
transfer_mma_kernel(const T *__restrict__ h, const T *__restrict__ W, T *__restrict__ out,
                    int rows_total, int d, int b0, int nb, int S) {
    __shared__ float s_part[kSplit ? 4 : 1][NB * 4][32];
    // lets a kernel that is serialized programmatically behind this one set itself up while this one runs
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
    const int groups = (rows_total + 15) / 16;
    const int items = groups * S;
    const int fchunk = ((d + 32 * S - 1) / (32 * S)) * 32;                   // features per range, a multiple of 32
    const uint4 zero = make_uint4(0, 0, 0, 0);
    // With S > 1 every warp has exactly one item (block b holds items 4b .. 4b+3); with S = 1 the warps of a
    // grid that just fills the GPU take equal contiguous shares of the groups (they differ by one at most).
    const long long w = (long long)blockIdx.x * 4 + wib, n_warps = (long long)gridDim.x * 4;
    const long long first = kSplit ? w : w * groups / n_warps;
    const int count = kSplit ? 1 : (int)((w + 1) * groups / n_warps - first);

    for (int k = 0; k < count; ++k) {
        const long long item = first + k;
        const bool live = item < items;
        const int grp = live ? (int)(kSplit ? item / S : item) : 0, part = kSplit ? (int)(item % S) : 0;   // `part` follows the warp's place in its block even past the last item
        const int r0 = grp * 16;
        const int f_lo = part * fchunk, f_hi = live ? min(d, f_lo + fchunk) : 0;
        const T *wa_row = W + (size_t)min(r0 + g, rows_total - 1) * d;        // rows past the end repeat the last one
        const T *wb_row = W + (size_t)min(r0 + g + 8, rows_total - 1) * d;
        float acc[NB][4];
#pragma unroll
        for (int n = 0; n < NB; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;

        for (int fb = f_lo; fb < f_hi; fb += 32 * U) {       // warp-uniform trip count: the products are warp-wide
            uint4 wa[U], wb[U], hb[U][NB];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int f = fb + u * 32 + t * 8;
                const bool in = f < f_hi;                                        // d is a multiple of 8
                wa[u] = in ? ld_nc16(wa_row + f) : zero;
                wb[u] = in ? ld_nc16(wb_row + f) : zero;
#pragma unroll
                for (int n = 0; n < NB; ++n) {
                    const int b = n * 8 + g;
                    hb[u][n] = (in && b < nb) ? *reinterpret_cast<const uint4 *>(h + (size_t)(b0 + b) * d + f) : zero;
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int n = 0; n < NB; ++n) {
                    MmaOp<T>::run(acc[n], wa[u].x, wb[u].x, wa[u].y, wb[u].y, hb[u][n].x, hb[u][n].y);
                    MmaOp<T>::run(acc[n], wa[u].z, wb[u].z, wa[u].w, wb[u].w, hb[u][n].z, hb[u][n].w);
                }
        }
        if (kSplit) {                                        // uniform over the block: one item per warp
#pragma unroll
            for (int n = 0; n < NB; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) s_part[wib][n * 4 + i][lane] = acc[n][i];
            __syncthreads();
            if (live && part == 0) {                     // part 0 sits S - 1 warps below the block's end: wib + o <= 3
                for (int o = 1; o < S; ++o)
#pragma unroll
                    for (int n = 0; n < NB; ++n)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[n][i] += s_part[wib + o][n * 4 + i][lane];
            }
        }
        if (live && part == 0) {
#pragma unroll
            for (int n = 0; n < NB; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = r0 + g + (i >> 1) * 8, b = n * 8 + 2 * t + (i & 1);
                    if (row < rows_total && b < nb) out[(size_t)(b0 + b) * rows_total + row] = from_float<T>(acc[n][i]);
                }
        }
    }
}

template <typename T, int NB, int U>
static int launch_mma(const void *h, const void *W, void *out, int rows_total, int d, int b0, int nb, cudaStream_t s) {
    const int groups = (rows_total + 15) / 16;
    const int full = transfer_grid(1 << 30, 16);               // blocks that fill the GPU once
    int S = 1;
    if (groups * 4ll <= full * 4ll && d >= 4 * 32 * U) S = 4;
    else if (groups * 2ll <= full * 4ll && d >= 2 * 32 * U) S = 2;
    if (S > 1) {
        const int blocks = (groups * S + 3) / 4;                // S divides 4: a group's warps share a block
        transfer_mma_kernel<T, NB, U, true><<<blocks, 128, 0, s>>>(static_cast<const T *>(h), static_cast<const T *>(W),
                                                                   static_cast<T *>(out), rows_total, d, b0, nb, S);
    } else {
        const int blocks = (groups + 3) / 4 < full ? (groups + 3) / 4 : full;
        transfer_mma_kernel<T, NB, U, false><<<blocks, 128, 0, s>>>(static_cast<const T *>(h), static_cast<const T *>(W),
                                                                    static_cast<T *>(out), rows_total, d, b0, nb, 1);
    }
    return check_launch("ht_transfer");
}

template <typename T>
static int launch_typed16(const void *h, const void *W, void *out, int B, int k, int d, cudaStream_t s) {
    const int rows_total = k * d;
    for (int b0 = 0; b0 < B; b0 += 16) {
        const int nb = min(16, B - b0);
        const int rc = nb <= 8 ? launch_mma<T, 1, 8>(h, W, out, rows_total, d, b0, nb, s)
                               : launch_mma<T, 2, 4>(h, W, out, rows_total, d, b0, nb, s);
        if (rc != HT_OK) return rc;
    }
    return HT_OK;
}

// Which kernel takes a 16-bit call: few source rows the warp-level instruction on the words as
// loaded, more the tcgen05 kernel (one pass over W for any number of rows).  HT_TRANSFER_KERNEL =
// "tc" or "mma" in the environment overrides the choice, for cross-checks of one against the other.
static bool use_tc(int B, int k, int d, int dtype) {
    if (!transfer_tc_applicable(B, k, d, dtype)) return false;
    const char *e = getenv("HT_TRANSFER_KERNEL");
    if ((e && !strcmp(e, "tc")) || knobs().path == 3) return true;
    if ((e && !strcmp(e, "mma")) || knobs().path == 2) return false;
    // 9 to 16 rows take the warp-level kernel's two-tile form (24.5 us on config 3's W against 19.3 with up to 8
    // rows); the tcgen05 kernel is ahead of that once W is large enough to amortise its set-up (21.6 us there).
    return B > 16 || (B > 8 && (long long)k * d * d * 2 >= (64ll << 20));
}

int launch_transfer(const void *h, const void *W, void *out, int B, int k, int d, int dtype,
                    cudaStream_t s) {
    if (use_tc(B, k, d, dtype)) {
        trace("ht_transfer -> tcgen05 kernel");
        return launch_transfer_tc(h, W, out, B, k, d, dtype, s);
    }
    trace("ht_transfer -> %s kernel", dtype == HT_F32 ? "fp32-ALU" : "m16n8k16");
    switch (dtype) {
        case HT_F32: return launch_typed<float>(h, W, out, B, k, d, s);
        case HT_F16: return launch_typed16<__half>(h, W, out, B, k, d, s);
        default: return launch_typed16<__nv_bfloat16>(h, W, out, B, k, d, s);
    }
}

}  // namespace ht
