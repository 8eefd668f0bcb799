// Hidden-transfer projection  h~ = W^i . h  (Section "Training stage", displayed equation).
//
// Shape of the work: k*d output rows, each a dot product of one row of W (d elements,
// read exactly once from HBM) with B hidden vectors (tiny, L1/L2 resident).  The kernel
// is a weight stream: arithmetic intensity is B flop per weight byte, far below the
// ridge for the batch sizes of decoding, so tensor cores are not used here and the
// design goal is 16-byte coalesced loads with enough of them in flight.
//
// One warp owns R consecutive rows of the flattened [k*d, d] weight; its lanes stride
// over the input features in 16-byte vectors, keep R x BT fp32 accumulators and reduce
// them with shuffles at the end.  The R rows share each loaded h vector, which cuts the
// L1 traffic for h by R.
#include "ht_common.cuh"

namespace ht {

template <typename T, int R, int BT>
__global__ void __launch_bounds__(128)
transfer_kernel(const T *__restrict__ h, const T *__restrict__ W, T *__restrict__ out,
                int B, int rows_total, int d, int b0) {
    constexpr int VE = Vec16<T>::n;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int row0 = warp * R;
    if (row0 >= rows_total) return;

    float acc[R][BT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int b = 0; b < BT; ++b) acc[r][b] = 0.f;

    const int nb = min(BT, B - b0);
    for (int c = lane * VE; c < d; c += 32 * VE) {
        uint4 wraw[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int row = min(row0 + r, rows_total - 1);
            wraw[r] = ld_nc16(W + (size_t)row * d + c);
        }
        float hv[BT][VE];
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            if (b < nb) {
                const uint4 raw = *reinterpret_cast<const uint4 *>(h + (size_t)(b0 + b) * d + c);
                unpack16<T>(raw, hv[b]);
            } else {
#pragma unroll
                for (int e = 0; e < VE; ++e) hv[b][e] = 0.f;
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float wf[VE];
            unpack16<T>(wraw[r], wf);
#pragma unroll
            for (int b = 0; b < BT; ++b)
#pragma unroll
                for (int e = 0; e < VE; ++e) acc[r][b] = fmaf(wf[e], hv[b][e], acc[r][b]);
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int b = 0; b < BT; ++b) {
            float v = acc[r][b];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lane == 0 && b < nb && row0 + r < rows_total)
                out[(size_t)(b0 + b) * rows_total + row0 + r] = from_float<T>(v);
        }
}

template <typename T, int R, int BT>
static int launch_one(const void *h, const void *W, void *out, int B, int rows_total, int d, int b0,
                      cudaStream_t s) {
    const int warps = (rows_total + R - 1) / R;
    const int blocks = (warps + 3) / 4;
    transfer_kernel<T, R, BT><<<blocks, 128, 0, s>>>(static_cast<const T *>(h), static_cast<const T *>(W),
                                                     static_cast<T *>(out), B, rows_total, d, b0);
    return check_launch("ht_transfer");
}

template <typename T>
static int launch_typed(const void *h, const void *W, void *out, int B, int k, int d, cudaStream_t s) {
    const int rows_total = k * d;
    // out is [B, k*d]: batch b writes at out + b*rows_total, so batch slices are independent.
    for (int b0 = 0; b0 < B; b0 += 8) {
        const int nb = min(8, B - b0);
        int rc;
        if (nb == 1) rc = launch_one<T, 4, 1>(h, W, out, B, rows_total, d, b0, s);
        else if (nb == 2) rc = launch_one<T, 4, 2>(h, W, out, B, rows_total, d, b0, s);
        else if (nb <= 4) rc = launch_one<T, 4, 4>(h, W, out, B, rows_total, d, b0, s);
        else rc = launch_one<T, 2, 8>(h, W, out, B, rows_total, d, b0, s);
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
