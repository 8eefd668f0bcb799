// Hidden-transfer projection  h~ = W^i . h  (Section "Training stage", displayed equation).
//
// Shape of the work: k*d output rows, each a dot product of one row of W (d elements,
// read exactly once from HBM) with B hidden vectors (tiny, L1/L2 resident).  The kernel
// is a weight stream: arithmetic intensity is B flop per weight byte, far below the
// ridge for the batch sizes of decoding, so tensor cores are not used here and the
// design goal is 16-byte coalesced loads with enough of them in flight.
//
// Every warp of a grid that just fills the GPU owns an equal, contiguous share of the k*d rows of
// the flattened [k*d, d] weight and walks it R rows at a time.  Its lanes stride over the input
// features in 16-byte vectors; U such steps (R x U independent 16-byte loads per lane) are issued
// before the first is used, which keeps over 100 KB of weight in flight per SM -- what a stream
// needs to run at memory speed.  R x BT fp32 accumulators per lane, reduced with shuffles at
// the end of a row group.  The R rows share each loaded h vector (h is small and cache resident).
#include "ht_common.cuh"

namespace ht {

constexpr int kTransferBlocksPerSm = 4;

template <typename T, int R, int BT, int U>
__global__ void __launch_bounds__(128, kTransferBlocksPerSm)
transfer_kernel(const T *__restrict__ h, const T *__restrict__ W, T *__restrict__ out,
                int rows_total, int d, int b0, int nb) {
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

int launch_transfer(const void *h, const void *W, void *out, int B, int k, int d, int dtype,
                    cudaStream_t s) {
    switch (dtype) {
        case HT_F32: return launch_typed<float>(h, W, out, B, k, d, s);
        case HT_F16: return launch_typed<__half>(h, W, out, B, k, d, s);
        default: return launch_typed<__nv_bfloat16>(h, W, out, B, k, d, s);
    }
}

}  // namespace ht
