// Draft tree for the next round (Sections "Inference stage" and "Tree attention"): the most
// likely tokens of each pseudo position's distribution are the candidates for the next
// positions; the candidates are merged by common ancestors into a pre-defined tree (template)
// and the tree is laid out flat with position ids = base position + depth.  With a template,
// merging needs no work at run time: node n at level i simply takes the rank[n]-th most likely
// token of pseudo position i.
//
// One block per (sequence, pseudo position).  The logits row is streamed once (16-byte loads,
// eight in flight per thread); every thread keeps its own K best entries as 64-bit keys
// (order-preserving bits of the value, then the inverted index: larger value first, lower index
// first among equals, NaN below everything), and K rounds of a block-wide maximum pick the
// row's K best in order.  The block then fills in the template nodes of its level.
#include "ht_common.cuh"

namespace ht {

constexpr int kDraftThreads = 256;
constexpr int kDraftMaxK = 16;

// Larger key = more likely.  NaN maps below -inf; among equal values the lower index is larger.
__device__ __forceinline__ unsigned long long draft_key(float x, int idx) {
    uint32_t b = __float_as_uint(x);
    uint32_t o = (b & 0x80000000u) ? ~b : (b | 0x80000000u);      // order-preserving for non-NaN; -0 < +0
    if (x == 0.f) o = 0x80000000u;                                   // -0 and +0 are one value
    if (x != x) o = 0u;                                              // below -inf (whose image is 0x007FFFFF)
    return ((unsigned long long)o << 32) | (0xFFFFFFFFu - (uint32_t)idx);
}

template <typename T, int KT>
__global__ void __launch_bounds__(kDraftThreads)
draft_tree_kernel(const T *__restrict__ logits, int rows, int V, int first_row, int P, int K,
                  const int32_t *__restrict__ tmpl_parent, const int32_t *__restrict__ tmpl_rank, int Tn,
                  const int32_t *__restrict__ root_token, const int32_t *__restrict__ base_pos,
                  int32_t *__restrict__ topk, int32_t *__restrict__ tokens, int32_t *__restrict__ pos,
                  int32_t *__restrict__ status) {
    constexpr int VE = Vec16<T>::n;
    __shared__ unsigned long long s_warp[kDraftThreads / 32];
    __shared__ unsigned long long s_win;
    __shared__ int32_t s_top[kDraftMaxK];
    __shared__ int s_bad;
    const int b = blockIdx.x / max(P, 1), lvl_i = blockIdx.x - b * max(P, 1);   // pseudo position lvl_i + 1
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_bad = 0;

    unsigned long long best[KT];
#pragma unroll
    for (int i = 0; i < KT; ++i) best[i] = 0ull;                   // below every real key (index part is never 0)
    if (P > 0) {
        const T *row = logits + ((size_t)b * rows + first_row + lvl_i) * V;
        auto offer = [&](float x, int idx) {
            const unsigned long long key = draft_key(x, idx);
            if (key > best[KT - 1]) {                              // insert, keeping best[] sorted descending
                best[KT - 1] = key;
#pragma unroll
                for (int i = KT - 1; i > 0; --i) {
                    if (best[i] > best[i - 1]) { const unsigned long long t = best[i]; best[i] = best[i - 1]; best[i - 1] = t; }
                }
            }
        };
        if (((size_t)V * sizeof(T)) % 16 == 0) {
            const int nvec = V / VE;
            constexpr int U = 8;
            for (int j0 = threadIdx.x; j0 < nvec; j0 += U * kDraftThreads) {
                uint4 raw[U];
#pragma unroll
                for (int u = 0; u < U; ++u) raw[u] = ld_nc16(row + (size_t)min(j0 + u * kDraftThreads, nvec - 1) * VE);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int j = j0 + u * kDraftThreads;
                    if (j < nvec) {
                        float f[VE];
                        unpack16<T>(raw[u], f);
#pragma unroll
                        for (int e = 0; e < VE; ++e) offer(f[e], j * VE + e);
                    }
                }
            }
        } else {
            for (int j = threadIdx.x; j < V; j += kDraftThreads) offer(to_float<T>(row[j]), j);
        }
    }
    __syncthreads();
    // K rounds: the block's largest head wins, its owner pops it
    for (int r = 0; r < K && P > 0; ++r) {
        unsigned long long m = best[0];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xffffffffu, m, off);
            m = o > m ? o : m;
        }
        if (lane == 0) s_warp[warp] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long w = s_warp[0];
            for (int i = 1; i < kDraftThreads / 32; ++i) w = s_warp[i] > w ? s_warp[i] : w;
            s_win = w;
            s_top[r] = (int32_t)(0xFFFFFFFFu - (uint32_t)(w & 0xFFFFFFFFull));
        }
        __syncthreads();
        if (best[0] == s_win && s_win != 0ull) {                   // keys are unique: exactly one owner
#pragma unroll
            for (int i = 0; i < KT - 1; ++i) best[i] = best[i + 1];
            best[KT - 1] = 0ull;
        }
    }
    __syncthreads();
    if (P > 0)
        for (int r = threadIdx.x; r < K; r += kDraftThreads) topk[((size_t)b * P + lvl_i) * K + r] = s_top[r];

    // Template: depth by walking up (parent[n] < n makes the walk finite); every block checks all of it
    // so that all agree on whether to skip the sequence.
    const bool has_root = root_token != nullptr;
    for (int n = threadIdx.x; n < Tn; n += kDraftThreads) {
        int depth = 0, c = n;
        bool ok = true;
        while (c >= 0 && ok) {
            const int par = tmpl_parent[c];
            if (par < -1 || par >= c) ok = false;
            if (par >= 0) ++depth;
            c = par;
        }
        const int level = depth + (has_root ? 0 : 1);
        if (!ok || level > P || (level >= 1 && (tmpl_rank[n] < 0 || tmpl_rank[n] >= K))) s_bad = 1;
    }
    __syncthreads();
    if (s_bad) {
        if (lvl_i == 0 && threadIdx.x == 0) status[b] = HT_STATUS_BAD_TREE;
        if (lvl_i == 0)
            for (int n = threadIdx.x; n < Tn; n += kDraftThreads) { tokens[(size_t)b * Tn + n] = -1; pos[(size_t)b * Tn + n] = -1; }
        return;
    }
    if (lvl_i == 0 && threadIdx.x == 0) status[b] = HT_STATUS_OK;
    const int bp = base_pos[b];
    for (int n = threadIdx.x; n < Tn; n += kDraftThreads) {
        int depth = 0;
        for (int c = tmpl_parent[n]; c >= 0; c = tmpl_parent[c]) ++depth;
        const int level = depth + (has_root ? 0 : 1);
        if (level == lvl_i + 1) {
            tokens[(size_t)b * Tn + n] = s_top[tmpl_rank[n]];
            pos[(size_t)b * Tn + n] = bp + depth;
        } else if (level == 0 && lvl_i == 0) {
            tokens[(size_t)b * Tn + n] = root_token[b];
            pos[(size_t)b * Tn + n] = bp;
        }
    }
}

template <typename T>
static void launch_k(int K, int blocks, cudaStream_t s, const void *logits, int rows, int V, int first_row, int P,
                     const int32_t *tp, const int32_t *tr, int Tn, const int32_t *root, const int32_t *bp,
                     int32_t *topk, int32_t *tokens, int32_t *pos, int32_t *status) {
    const T *lg = static_cast<const T *>(logits);
    if (K <= 4) draft_tree_kernel<T, 4><<<blocks, kDraftThreads, 0, s>>>(lg, rows, V, first_row, P, K, tp, tr, Tn, root, bp, topk, tokens, pos, status);
    else if (K <= 8) draft_tree_kernel<T, 8><<<blocks, kDraftThreads, 0, s>>>(lg, rows, V, first_row, P, K, tp, tr, Tn, root, bp, topk, tokens, pos, status);
    else draft_tree_kernel<T, 16><<<blocks, kDraftThreads, 0, s>>>(lg, rows, V, first_row, P, K, tp, tr, Tn, root, bp, topk, tokens, pos, status);
}

int launch_draft(const void *logits, int dtype, int B, int rows, int V, int first_row, int P, int K,
                 const int32_t *tmpl_parent, const int32_t *tmpl_rank, int Tn, const int32_t *root_token,
                 const int32_t *base_pos, int32_t *topk, int32_t *tokens, int32_t *pos, int32_t *status, cudaStream_t s) {
    const int blocks = B * (P > 0 ? P : 1);
    switch (dtype) {
        case HT_F32: launch_k<float>(K, blocks, s, logits, rows, V, first_row, P, tmpl_parent, tmpl_rank, Tn, root_token, base_pos, topk, tokens, pos, status); break;
        case HT_F16: launch_k<__half>(K, blocks, s, logits, rows, V, first_row, P, tmpl_parent, tmpl_rank, Tn, root_token, base_pos, topk, tokens, pos, status); break;
        default: launch_k<__nv_bfloat16>(K, blocks, s, logits, rows, V, first_row, P, tmpl_parent, tmpl_rank, Tn, root_token, base_pos, topk, tokens, pos, status); break;
    }
    return check_launch("ht_draft_tree");
}

}  // namespace ht
