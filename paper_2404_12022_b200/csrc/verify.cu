// Greedy verification (Fig. 2 caption; Sections "Inference stage" and "Setup"):
// row argmax of the logits, then the longest root path of the draft tree whose tokens
// are the ones greedy decoding would emit.
//
// One launch: a block per logits row streams it once (16-byte loads, eight in flight per thread,
// shuffle reductions) and stores the row's argmax; the block that finishes a sequence's last row
// (a ticket per sequence, drawn on the accept_len word, which a memset clears ahead of the launch)
// runs the path search for that sequence -- a few hundred integer operations.  Nobody waits.
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

// pred is written by other blocks of the same launch: read through L2 when it is read from global memory
// (a generic load works for the staged copy in shared memory as well).
__device__ __forceinline__ int ld_pred(const int32_t *p) {
    return __isGlobal(p) ? __ldcg(p) : *p;
}

// Path search of one sequence by one block.  Every thread walks the root path of its nodes (parent[c] < c
// makes the walk finite), checks the match rule on the way and proposes (depth, node);
// the block keeps the deepest valid node, lowest index on ties.
__device__ __forceinline__ void accept_sequence(const int b, const int32_t *__restrict__ tokens, const int32_t *__restrict__ parent,
              const int32_t *__restrict__ root_pred, const int32_t *pred, int N, int T,
              int max_path, int32_t *accept_len, int32_t *__restrict__ accept_path,
              int32_t *__restrict__ next_token, int32_t *__restrict__ status) {
    const int32_t *par = parent + (size_t)b * N;
    const int32_t *tok = tokens + (size_t)b * T;
    const int32_t *prd = pred + (size_t)b * N;
    int32_t *path = accept_path + (size_t)b * max_path;
    __shared__ int s_bad;
    __shared__ unsigned long long s_key[8];
    // The walks below are chains of dependent reads: with the tree's three arrays in shared memory they
    // cost one round trip to L2 in all instead of one per level (trees of up to kStage rows).
    constexpr int kStage = 1024;
    __shared__ int32_t s_par[kStage], s_tok[kStage], s_prd[kStage];
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    if (N <= kStage) {
        for (int c = threadIdx.x; c < N; c += blockDim.x) {
            const int pc = par[c];
            s_par[c] = pc;
            s_prd[c] = __ldcg(prd + c);
            if (c < T) s_tok[c] = tok[c];
            if (pc < -1 || pc >= c) s_bad = 1;
        }
        par = s_par; tok = s_tok; prd = s_prd;
    } else {
        for (int c = threadIdx.x; c < N; c += blockDim.x)
            if (par[c] < -1 || par[c] >= c) s_bad = 1;
    }
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
            const bool m = p < 0 ? (!has_root || tok[c] == rp) : (tok[c] == ld_pred(prd + p));
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
                next_token[b] = ld_pred(prd + node);
            }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
verify_kernel(const T *__restrict__ logits, int V, int32_t *__restrict__ pred, const int32_t *__restrict__ tokens,
              const int32_t *__restrict__ parent, const int32_t *__restrict__ root_pred, int N, int Tn, int max_path,
              int32_t *__restrict__ accept_len, int32_t *__restrict__ accept_path, int32_t *__restrict__ next_token,
              int32_t *__restrict__ status) {
    // The launch is serialized programmatically behind the kernel that zeroes the tickets, which itself waits for the
    // work ahead of it in the stream: from here on everything that work wrote may be read.  A kernel serialized
    // behind this one (the compaction) may set itself up meanwhile.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
                    // A thread meets its elements in increasing index order, so "larger value, lower index
                    // on ties" is "strictly larger than the best so far".  NaN compares false and is
                    // skipped; so is -inf, which a row without anything larger settles below.
                    if (f[e] > best.v) best = Best{f[e], j * VE + e};
                }
            }
        }
    } else {
        for (int j = threadIdx.x; j < V; j += blockDim.x) {
            const float x = to_float<T>(row[j]);
            if (x > best.v) best = Best{x, j};
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
        if (lane == 0) warp_best[0] = best;
    }
    __syncthreads();
    best = warp_best[0];
    if (best.i == INT_MAX) {
        // Nothing in the row exceeds -inf: the answer is the first -inf, or 0 in a row of NaNs only.
        int first = INT_MAX;
        for (int j = threadIdx.x; j < V; j += blockDim.x)
            if (to_float<T>(row[j]) == -INFINITY) { first = j; break; }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, off));
        __shared__ int warp_first[8];
        if (lane == 0) warp_first[warp] = first;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < (int)(blockDim.x >> 5); ++w) first = min(first, warp_first[w]);
            best.i = first == INT_MAX ? 0 : first;
        }
    }
    if (threadIdx.x == 0) pred[blockIdx.x] = best.i;
    // The block that stores a sequence's last argmax searches its tree.
    __shared__ int s_last;
    const int b = blockIdx.x / N;
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(reinterpret_cast<unsigned int *>(accept_len + b), 1u) == (unsigned)(N - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    accept_sequence(b, tokens, parent, root_pred, pred, N, Tn, max_path, accept_len, accept_path, next_token, status);
}

// accept_len doubles as the per-sequence ticket until the sequence's last block overwrites it: zero at the start.
// A kernel rather than a memset node, so that the launches chain by programmatic stream serialization: it is in
// place, waiting, before the kernel ahead of it in the stream has finished.
__global__ void verify_prepare_kernel(int32_t *accept_len, int B) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int i = threadIdx.x; i < B; i += blockDim.x) accept_len[i] = 0;
}

template <typename... KArgs, typename... Args>
static cudaError_t launch_chained(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int launch_verify(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                  const int32_t *root_pred, int B, int N, int T, int V, int max_path, int32_t *pred,
                  int32_t *accept_len, int32_t *accept_path, int32_t *next_token, int32_t *status,
                  cudaStream_t s) {
    const unsigned rows = (unsigned)(B * N);
    cudaError_t e = launch_chained(verify_prepare_kernel, 1u, 256u, s, accept_len, B);
    if (e == cudaSuccess) {
        switch (dtype) {
            case HT_F32:
                e = launch_chained(verify_kernel<float>, rows, 256u, s, static_cast<const float *>(logits), V, pred, tokens, parent, root_pred,
                                   N, T, max_path, accept_len, accept_path, next_token, status);
                break;
            case HT_F16:
                e = launch_chained(verify_kernel<__half>, rows, 256u, s, static_cast<const __half *>(logits), V, pred, tokens, parent, root_pred,
                                   N, T, max_path, accept_len, accept_path, next_token, status);
                break;
            default:
                e = launch_chained(verify_kernel<__nv_bfloat16>, rows, 256u, s, static_cast<const __nv_bfloat16 *>(logits), V, pred, tokens, parent,
                                   root_pred, N, T, max_path, accept_len, accept_path, next_token, status);
                break;
        }
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "ht_verify_greedy: %s", cudaGetErrorString(e));
    }
    return HT_OK;
}

}  // namespace ht
