// KV compaction: the accepted path's K/V rows are moved directly behind the context, in
// place, for every layer and KV head in one launch (Fig. 1 caption and Section "Inference
// stage" imply it: verification runs against a KV cache, and only accepted tokens may
// stay in it).
//
// One block per (layer, sequence, KV head, K-or-V).  A destination row can be another
// step's source: with path [0, 2, 5] row L+2 is overwritten by j = 2 and read by j = 1.
// The block therefore gathers every source row into registers with 16-byte loads,
// synchronises, and only then scatters.  A (layer, sequence, head, tensor) is handled by
// exactly one block, so no other block can observe the intermediate state.
#include "ht_common.cuh"

namespace ht {

constexpr int kCompactThreads = 256;
constexpr int kCompactMaxPath = 64;

__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(unsigned char *__restrict__ k_cache, unsigned char *__restrict__ v_cache,
               int layers, int B, int Hkv, int cap, int N, int row_bytes, long long stride_layer_b,
               long long stride_b_b, long long stride_h_b, const int32_t *__restrict__ kv_len,
               const int32_t *__restrict__ accept_len, const int32_t *__restrict__ accept_path,
               int max_path, int32_t *__restrict__ new_kv_len, int32_t *__restrict__ status) {
    int idx = blockIdx.x;
    const int which = idx & 1;
    idx >>= 1;
    const int h = idx % Hkv;
    idx /= Hkv;
    const int b = idx % B;
    const int layer = idx / B;

    const int L = kv_len[b];
    const int a = accept_len[b];
    const int32_t *path = accept_path + (size_t)b * max_path;

    // Validation is repeated by every block of the sequence (a few integer loads) so that
    // all of them agree on whether to skip it; one block reports.
    int code = HT_STATUS_OK;
    if (L < 0 || (long long)L + N > cap) {
        code = HT_STATUS_BAD_LEN;
    } else if (a < 0 || a > max_path || a > N) {
        code = HT_STATUS_BAD_PATH;
    } else {
        for (int j = 0; j < a; ++j) {
            const int p = path[j];
            if (p < j || p >= N || (j > 0 && p <= path[j - 1])) code = HT_STATUS_BAD_PATH;
        }
    }
    if (layer == 0 && h == 0 && which == 0 && threadIdx.x == 0) {
        status[b] = code;
        new_kv_len[b] = code == HT_STATUS_OK ? L + a : L;
    }
    if (code != HT_STATUS_OK || a == 0) return;

    unsigned char *base = (which ? v_cache : k_cache) + (long long)layer * stride_layer_b +
                          (long long)b * stride_b_b + (long long)h * stride_h_b;
    const int vec_per_row = row_bytes / 16;
    const int total = a * vec_per_row;
    constexpr int kMaxPerThread = 16;   // 64 rows x 1 KiB rows / 256 threads at most
    uint4 regs[kMaxPerThread];
#pragma unroll
    for (int i = 0; i < kMaxPerThread; ++i) {
        const int t = threadIdx.x + i * kCompactThreads;
        if (t < total) {
            const int j = t / vec_per_row, v = t - j * vec_per_row;
            const int src = path[j];
            if (src != j)
                regs[i] = *reinterpret_cast<const uint4 *>(base + (size_t)(L + src) * row_bytes + (size_t)v * 16);
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kMaxPerThread; ++i) {
        const int t = threadIdx.x + i * kCompactThreads;
        if (t < total) {
            const int j = t / vec_per_row, v = t - j * vec_per_row;
            if (path[j] != j)
                *reinterpret_cast<uint4 *>(base + (size_t)(L + j) * row_bytes + (size_t)v * 16) = regs[i];
        }
    }
}

int launch_compact(void *kc, void *vc, const ht_cache_desc &d, const int32_t *kv_len,
                   const int32_t *accept_len, const int32_t *accept_path, int max_path,
                   int32_t *new_kv_len, int32_t *status, cudaStream_t s) {
    const long long e = elem_bytes(d.dtype);
    const long long stride_h = (d.stride_h ? d.stride_h : (long long)d.cap * d.D) * e;
    const long long stride_b = (d.stride_b ? d.stride_b : (long long)d.Hkv * d.cap * d.D) * e;
    const long long stride_l = (d.stride_layer ? d.stride_layer : (long long)d.B * d.Hkv * d.cap * d.D) * e;
    const int row_bytes = d.D * (int)e;
    const long long blocks = 2ll * d.layers * d.B * d.Hkv;
    compact_kernel<<<(unsigned)blocks, kCompactThreads, 0, s>>>(
        static_cast<unsigned char *>(kc), static_cast<unsigned char *>(vc), d.layers, d.B, d.Hkv, d.cap,
        d.N, row_bytes, stride_l, stride_b, stride_h, kv_len, accept_len, accept_path, max_path,
        new_kv_len, status);
    return check_launch("ht_kv_compact");
}

}  // namespace ht
