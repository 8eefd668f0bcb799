// Greedy verification (Fig. 2 caption; Sections "Inference stage" and "Setup"):
// row argmax of the logits, then the longest root path of the draft tree whose tokens
// are the ones greedy decoding would emit.
//
// Kernel 1 streams the logits once (HBM-bound scan, 16-byte loads, shuffle reductions);
// kernel 2 is a few hundred integer operations per sequence.
#include <limits.h>

#include "ht_common.cuh"

namespace ht {

struct Best {
    float v;
    int i;
};

// Total order used at every reduction stage: larger value first, lower index on ties.
__device__ __forceinline__ Best better(Best a, Best b) {
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

template <typename T>
__global__ void __launch_bounds__(256)
row_argmax_kernel(const T *__restrict__ logits, int V, int32_t *__restrict__ pred) {
    constexpr int VE = Vec16<T>::n;
    const T *row = logits + (size_t)blockIdx.x * V;
    Best best{-INFINITY, INT_MAX};
    const bool vec_ok = ((size_t)V * sizeof(T)) % 16 == 0;
    if (vec_ok) {
        const int nvec = V / VE;
        constexpr int U = 8;                       // independent 16-byte loads in flight per thread
        for (int j0 = threadIdx.x; j0 < nvec; j0 += U * blockDim.x) {
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int j = j0 + u * blockDim.x;
                raw[u] = ld_nc16(row + (size_t)min(j, nvec - 1) * VE);   // past the end: the last vector again
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int j = min(j0 + u * (int)blockDim.x, nvec - 1);
                float f[VE];
                unpack16<T>(raw[u], f);
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    // NaN compares false both ways and is skipped; -inf at a lower index than
                    // the current -inf candidate is taken through the equality branch.
                    if (f[e] > best.v || (f[e] == best.v && j * VE + e < best.i)) best = Best{f[e], j * VE + e};
                }
            }
        }
    } else {
        for (int j = threadIdx.x; j < V; j += blockDim.x) {
            const float x = to_float<T>(row[j]);
            if (x > best.v || (x == best.v && j < best.i)) best = Best{x, j};
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Best o{__shfl_xor_sync(0xffffffffu, best.v, off), __shfl_xor_sync(0xffffffffu, best.i, off)};
        best = better(best, o);
    }
    __shared__ Best warp_best[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) warp_best[warp] = best;
    __syncthreads();
    if (warp == 0) {
        best = lane < (int)(blockDim.x >> 5) ? warp_best[lane] : Best{-INFINITY, INT_MAX};
#pragma unroll
        for (int off = 4; off > 0; off >>= 1) {
            Best o{__shfl_xor_sync(0xffffffffu, best.v, off), __shfl_xor_sync(0xffffffffu, best.i, off)};
            best = better(best, o);
        }
        if (lane == 0) pred[blockIdx.x] = best.i == INT_MAX ? 0 : best.i;
    }
}

// One block per sequence.  Every thread walks the root path of its nodes (parent[c] < c
// makes the walk finite), checks the match rule on the way and proposes (depth, node);
// the block keeps the deepest valid node, lowest index on ties.
__global__ void __launch_bounds__(128)
accept_kernel(const int32_t *__restrict__ tokens, const int32_t *__restrict__ parent,
              const int32_t *__restrict__ root_pred, const int32_t *__restrict__ pred, int N, int T,
              int max_path, int32_t *__restrict__ accept_len, int32_t *__restrict__ accept_path,
              int32_t *__restrict__ next_token, int32_t *__restrict__ status) {
    const int b = blockIdx.x;
    const int32_t *par = parent + (size_t)b * N;
    const int32_t *tok = tokens + (size_t)b * T;
    const int32_t *prd = pred + (size_t)b * N;
    int32_t *path = accept_path + (size_t)b * max_path;
    __shared__ int s_bad;
    __shared__ unsigned long long s_key[4];
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    for (int c = threadIdx.x; c < N; c += blockDim.x)
        if (par[c] < -1 || par[c] >= c) s_bad = 1;
    for (int j = threadIdx.x; j < max_path; j += blockDim.x) path[j] = -1;
    __syncthreads();
    if (s_bad) {
        if (threadIdx.x == 0) {
            status[b] = HT_STATUS_BAD_TREE;
            accept_len[b] = 0;
            next_token[b] = -1;
        }
        return;
    }
    const bool has_root = root_pred != nullptr;
    const int rp = has_root ? root_pred[b] : -1;
    // key = depth << 32 | (0xFFFFFFFF - node): max picks the deepest, then the lowest node
    unsigned long long key = 0;
    for (int n = threadIdx.x; n < T; n += blockDim.x) {
        int depth = 0;
        bool ok = true;
        for (int c = n; c >= 0; c = par[c]) {
            const int p = par[c];
            const bool m = p < 0 ? (!has_root || tok[c] == rp) : (tok[c] == prd[p]);
            ok = ok && m;
            ++depth;
        }
        if (ok) {
            const unsigned long long k2 = ((unsigned long long)depth << 32) | (0xFFFFFFFFu - (unsigned)n);
            key = k2 > key ? k2 : key;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, key, off);
        key = o > key ? o : key;
    }
    if ((threadIdx.x & 31) == 0) s_key[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) key = s_key[w] > key ? s_key[w] : key;
        const int len = (int)(key >> 32);
        const int node = (int)(0xFFFFFFFFu - (unsigned)(key & 0xFFFFFFFFu));
        if (len > max_path) {
            status[b] = HT_STATUS_PATH_TOO_LONG;
            accept_len[b] = 0;
            next_token[b] = -1;
        } else {
            status[b] = HT_STATUS_OK;
            accept_len[b] = len;
            if (len == 0) {
                next_token[b] = has_root ? rp : -1;
            } else {
                int j = len - 1;
                for (int c = node; c >= 0; c = par[c]) path[j--] = c;
                next_token[b] = prd[node];
            }
        }
    }
}

int launch_verify(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                  const int32_t *root_pred, int B, int N, int T, int V, int max_path, int32_t *pred,
                  int32_t *accept_len, int32_t *accept_path, int32_t *next_token, int32_t *status,
                  cudaStream_t s) {
    const int rows = B * N;
    switch (dtype) {
        case HT_F32:
            row_argmax_kernel<float><<<rows, 256, 0, s>>>(static_cast<const float *>(logits), V, pred);
            break;
        case HT_F16:
            row_argmax_kernel<__half><<<rows, 256, 0, s>>>(static_cast<const __half *>(logits), V, pred);
            break;
        default:
            row_argmax_kernel<__nv_bfloat16><<<rows, 256, 0, s>>>(
                static_cast<const __nv_bfloat16 *>(logits), V, pred);
            break;
    }
    int rc = check_launch("ht_verify_greedy (row argmax)");
    if (rc != HT_OK) return rc;
    accept_kernel<<<B, 128, 0, s>>>(tokens, parent, root_pred, pred, N, T, max_path, accept_len,
                                    accept_path, next_token, status);
    return check_launch("ht_verify_greedy (acceptance)");
}

}  // namespace ht
