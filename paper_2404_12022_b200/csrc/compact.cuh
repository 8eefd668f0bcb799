// KV compaction of one (layer, sequence, share of the (KV head, K | V) pairs) by one thread block: the accepted
// path's rows are moved directly behind the context (Fig. 1 caption and Section "Inference stage" imply it:
// verification runs against a KV cache, and only accepted tokens may stay in it).  Used by the compaction kernel
// (one item per block) and by the fused verification kernel (items dealt out to the blocks of its grid).
//
// A destination row can be another step's source: with path [0, 2, 5] row L+2 is overwritten by j = 2 and read by
// j = 1.  A block therefore gathers every source row of the pairs it is working on into registers with 16-byte
// loads, synchronises, and only then scatters.  Each (layer, sequence, head, tensor) is handled by exactly one
// block, so no other block can observe the intermediate state.
#pragma once
#include "ht_common.cuh"

namespace ht {

constexpr int kCompactThreads = 256;
constexpr int kCompactMaxPath = 64;

struct CompactArgs {
    unsigned char *k_cache, *v_cache;
    int layers, B, Hkv, cap, N, row_bytes;
    long long stride_layer_b, stride_b_b, stride_h_b;      // bytes
    const int32_t *kv_len, *accept_len, *accept_path;
    int max_path, groups;                                  // groups: shares of the 2 * Hkv pairs of a (layer, sequence)
    int32_t *new_kv_len, *status;
    PageMap pm;                                            // strides in bytes here
};

struct CompactSmem {
    int32_t path[kCompactMaxPath];
    long long src[kCompactMaxPath], dst[kCompactMaxPath];  // byte offsets of the rows within (layer, tensor), short of the head's
    int bad_page;
};

// Called by all kThreads threads of a block; `a` = accept_len[b] and `L` = kv_len[b] as the caller read them
// (the fused kernel reads the former with acquire semantics, and the latter while it waits for the former).  Ends with a barrier, so that the shared arrays may be reused at once.
template <int kPerThread, int kThreads = kCompactThreads>   // 16-byte vectors a thread holds between gather and scatter; threads of the block
__device__ __forceinline__ void compact_item(const CompactArgs &c, CompactSmem &sm, int layer, int b, int grp, int a, int L) {
    if ((int)threadIdx.x < c.max_path) sm.path[threadIdx.x] = c.accept_path[(size_t)b * c.max_path + threadIdx.x];
    if (threadIdx.x == 0) sm.bad_page = 0;
    __syncthreads();

    // Validation is repeated by every block of the sequence (a few integers) so that all of
    // them agree on whether to skip it; one block reports.
    int code = HT_STATUS_OK;
    if (L < 0 || (long long)L + c.N > c.cap) {
        code = HT_STATUS_BAD_LEN;
    } else if (a < 0 || a > c.max_path || a > c.N) {
        code = HT_STATUS_BAD_PATH;
    } else {
        for (int j = 0; j < a; ++j) {
            const int p = sm.path[j];
            if (p < j || p >= c.N || (j > 0 && p <= sm.path[j - 1])) code = HT_STATUS_BAD_PATH;
        }
    }
    // Where the path's source and destination rows lie.  Paged cache: through the block table; an entry
    // outside the pool leaves the sequence untouched, and every block of the sequence sees the same entries.
    if (c.pm.table && code == HT_STATUS_OK && (int)threadIdx.x < a) {
        const int j = threadIdx.x, rows[2] = {L + sm.path[j], L + j};
        long long off[2];
        for (int x = 0; x < 2; ++x) {
            if (c.pm.table) {
                const int page = c.pm.table[(size_t)b * c.pm.max_pages + (rows[x] >> c.pm.shift)];
                if ((unsigned)page >= (unsigned)c.pm.n_pages) sm.bad_page = 1;
                off[x] = (long long)page * c.pm.page_stride + (long long)(rows[x] & ((1 << c.pm.shift) - 1)) * c.row_bytes;
            } else {
                off[x] = 0;
            }
        }
        sm.src[j] = off[0];
        sm.dst[j] = off[1];
    }
    if (c.pm.table) __syncthreads();               // (contiguous cache: the offsets are formed where they are used)
    if (code == HT_STATUS_OK && sm.bad_page) code = HT_STATUS_BAD_PAGE;
    if (layer == 0 && grp == 0 && threadIdx.x == 0) {
        c.status[b] = code;
        c.new_kv_len[b] = code == HT_STATUS_OK ? L + a : L;
    }
    if (code != HT_STATUS_OK || a == 0) {
        __syncthreads();
        return;
    }

    const int pairs = 2 * c.Hkv;                                 // pair = (KV head, K-or-V)
    const int pair_lo = (int)((long long)pairs * grp / c.groups), pair_hi = (int)((long long)pairs * (grp + 1) / c.groups);
    const int vec_per_row = c.row_bytes / 16;
    const int per_pair = a * vec_per_row;                        // <= 4096 (checked by the caller)
    const int pairs_per_pass = max(1, kPerThread * kThreads / per_pair);
    unsigned char *const base_k = c.k_cache + (long long)layer * c.stride_layer_b;
    unsigned char *const base_v = c.v_cache + (long long)layer * c.stride_layer_b;
    const long long seq_off = (long long)b * c.stride_b_b;

    for (int p0 = pair_lo; p0 < pair_hi; p0 += pairs_per_pass) {
        const int total = min(pairs_per_pass, pair_hi - p0) * per_pair;
        uint4 regs[kPerThread];
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int t = threadIdx.x + i * kThreads;
            if (t < total) {
                const int pr = t / per_pair, rem = t - pr * per_pair;
                const int j = rem / vec_per_row, v = rem - j * vec_per_row;
                const int pair = p0 + pr, src = sm.path[j];
                const unsigned char *base = ((pair & 1) ? base_v : base_k) + (long long)(pair >> 1) * c.stride_h_b;
                const long long off = c.pm.table ? sm.src[j] : seq_off + (long long)(L + src) * c.row_bytes;
                if (src != j)
                    regs[i] = *reinterpret_cast<const uint4 *>(base + off + (size_t)v * 16);
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int t = threadIdx.x + i * kThreads;
            if (t < total) {
                const int pr = t / per_pair, rem = t - pr * per_pair;
                const int j = rem / vec_per_row, v = rem - j * vec_per_row;
                const int pair = p0 + pr;
                unsigned char *base = ((pair & 1) ? base_v : base_k) + (long long)(pair >> 1) * c.stride_h_b;
                const long long off = c.pm.table ? sm.dst[j] : seq_off + (long long)(L + j) * c.row_bytes;
                if (sm.path[j] != j)
                    *reinterpret_cast<uint4 *>(base + off + (size_t)v * 16) = regs[i];
            }
        }
        __syncthreads();     // the next pass of this block may touch rows this pass has written only after all of it has
    }
}

// Fills the arguments from the descriptor (host).  `blocks`: how many thread blocks the items should about come to
// (at most one per (head, tensor) pair of a (layer, sequence), at least one per (layer, sequence)).
CompactArgs make_compact_args(void *kc, void *vc, const ht_cache_desc &d, const int32_t *kv_len, const int32_t *accept_len,
                              const int32_t *accept_path, int max_path, int32_t *new_kv_len, int32_t *status,
                              const PageMap &pm_elems, int blocks);

}  // namespace ht
