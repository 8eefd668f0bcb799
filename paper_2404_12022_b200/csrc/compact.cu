// KV compaction: the accepted path's K/V rows are moved directly behind the context, in
// place, for every layer and KV head in one launch (Fig. 1 caption and Section "Inference
// stage" imply it: verification runs against a KV cache, and only accepted tokens may
// stay in it).
//
// A destination row can be another step's source: with path [0, 2, 5] row L+2 is overwritten
// by j = 2 and read by j = 1.  A block therefore gathers every source row of the (KV head,
// K-or-V) pairs it is working on into registers with 16-byte loads, synchronises, and only
// then scatters.  Each (layer, sequence, head, tensor) is handled by exactly one block, so no
// other block can observe the intermediate state.
//
// The data are tiny (a few rows per head), so the kernel is a chain of dependent round trips
// to memory: lengths -> path -> rows -> stores.  A block takes one (layer, sequence) and a
// contiguous share of its 2*Hkv pairs, and moves as many pairs per pass as its registers hold
// (16 vectors per thread), all loads of a pass in flight together.
#include "ht_common.cuh"

namespace ht {

constexpr int kCompactThreads = 256;
constexpr int kCompactMaxPath = 64;
constexpr int kCompactPerThread = 16;   // 16-byte vectors a thread holds between gather and scatter

__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(unsigned char *__restrict__ k_cache, unsigned char *__restrict__ v_cache,
               int layers, int B, int Hkv, int cap, int N, int row_bytes, long long stride_layer_b,
               long long stride_b_b, long long stride_h_b, const int32_t *__restrict__ kv_len,
               const int32_t *__restrict__ accept_len, const int32_t *__restrict__ accept_path,
               int max_path, int groups, int32_t *__restrict__ new_kv_len, int32_t *__restrict__ status, const PageMap pm) {
    __shared__ int32_t s_path[kCompactMaxPath];
    __shared__ long long s_src[kCompactMaxPath], s_dst[kCompactMaxPath];   // byte offsets of the rows within (layer, tensor), short of the head's
    __shared__ int s_bad_page;
    // The launch is serialized programmatically behind the kernel before it in the stream (the verification, as a
    // rule): the blocks are in place while that kernel finishes, and read what it wrote from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int idx = blockIdx.x;
    const int grp = idx % groups;
    idx /= groups;
    const int b = idx % B;
    const int layer = idx / B;

    const int L = kv_len[b];
    const int a = accept_len[b];
    if (threadIdx.x < max_path) s_path[threadIdx.x] = accept_path[(size_t)b * max_path + threadIdx.x];
    __syncthreads();

    // Validation is repeated by every block of the sequence (a few integers) so that all of
    // them agree on whether to skip it; one block reports.
    int code = HT_STATUS_OK;
    if (L < 0 || (long long)L + N > cap) {
        code = HT_STATUS_BAD_LEN;
    } else if (a < 0 || a > max_path || a > N) {
        code = HT_STATUS_BAD_PATH;
    } else {
        for (int j = 0; j < a; ++j) {
            const int p = s_path[j];
            if (p < j || p >= N || (j > 0 && p <= s_path[j - 1])) code = HT_STATUS_BAD_PATH;
        }
    }
    // Where the path's source and destination rows lie.  Paged cache: through the block table; an entry
    // outside the pool leaves the sequence untouched, and every block of the sequence sees the same entries.
    if (threadIdx.x == 0) s_bad_page = 0;
    __syncthreads();
    if (code == HT_STATUS_OK && threadIdx.x < a) {
        const int j = threadIdx.x, rows[2] = {L + s_path[j], L + j};
        long long off[2];
        for (int x = 0; x < 2; ++x) {
            if (pm.table) {
                const int page = pm.table[(size_t)b * pm.max_pages + (rows[x] >> pm.shift)];
                if ((unsigned)page >= (unsigned)pm.n_pages) s_bad_page = 1;
                off[x] = (long long)page * pm.page_stride + (long long)(rows[x] & ((1 << pm.shift) - 1)) * row_bytes;   // strides of `pm` in bytes here
            } else {
                off[x] = (long long)b * stride_b_b + (long long)rows[x] * row_bytes;
            }
        }
        s_src[j] = off[0];
        s_dst[j] = off[1];
    }
    __syncthreads();
    if (code == HT_STATUS_OK && s_bad_page) code = HT_STATUS_BAD_PAGE;
    if (layer == 0 && grp == 0 && threadIdx.x == 0) {
        status[b] = code;
        new_kv_len[b] = code == HT_STATUS_OK ? L + a : L;
    }
    if (code != HT_STATUS_OK || a == 0) return;

    const int pairs = 2 * Hkv;                                   // pair = (KV head, K-or-V)
    const int pair_lo = (int)((long long)pairs * grp / groups), pair_hi = (int)((long long)pairs * (grp + 1) / groups);
    const int vec_per_row = row_bytes / 16;
    const int per_pair = a * vec_per_row;                        // <= 4096 (checked by the caller)
    const int pairs_per_pass = max(1, kCompactPerThread * kCompactThreads / per_pair);
    unsigned char *const base_k = k_cache + (long long)layer * stride_layer_b;
    unsigned char *const base_v = v_cache + (long long)layer * stride_layer_b;

    for (int p0 = pair_lo; p0 < pair_hi; p0 += pairs_per_pass) {
        const int total = min(pairs_per_pass, pair_hi - p0) * per_pair;
        uint4 regs[kCompactPerThread];
#pragma unroll
        for (int i = 0; i < kCompactPerThread; ++i) {
            const int t = threadIdx.x + i * kCompactThreads;
            if (t < total) {
                const int pr = t / per_pair, rem = t - pr * per_pair;
                const int j = rem / vec_per_row, v = rem - j * vec_per_row;
                const int pair = p0 + pr, src = s_path[j];
                const unsigned char *base = ((pair & 1) ? base_v : base_k) + (long long)(pair >> 1) * stride_h_b;
                if (src != j)
                    regs[i] = *reinterpret_cast<const uint4 *>(base + s_src[j] + (size_t)v * 16);
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kCompactPerThread; ++i) {
            const int t = threadIdx.x + i * kCompactThreads;
            if (t < total) {
                const int pr = t / per_pair, rem = t - pr * per_pair;
                const int j = rem / vec_per_row, v = rem - j * vec_per_row;
                const int pair = p0 + pr;
                unsigned char *base = ((pair & 1) ? base_v : base_k) + (long long)(pair >> 1) * stride_h_b;
                if (s_path[j] != j)
                    *reinterpret_cast<uint4 *>(base + s_dst[j] + (size_t)v * 16) = regs[i];
            }
        }
        __syncthreads();     // the next pass of this block may touch rows this pass has written only after all of it has
    }
}

int launch_compact(void *kc, void *vc, const ht_cache_desc &d, const int32_t *kv_len,
                   const int32_t *accept_len, const int32_t *accept_path, int max_path,
                   int32_t *new_kv_len, int32_t *status, cudaStream_t s, const PageMap &pm_elems) {
    const long long e = elem_bytes(d.dtype);
    PageMap pm = pm_elems;                 // the kernel takes the page strides in bytes
    pm.page_stride *= e;
    pm.head_stride *= e;
    const long long stride_h = pm.table ? pm.head_stride : (d.stride_h ? d.stride_h : (long long)d.cap * d.D) * e;
    const long long stride_b = (d.stride_b ? d.stride_b : (long long)d.Hkv * d.cap * d.D) * e;
    const long long stride_l = (d.stride_layer ? d.stride_layer : (pm.table ? (long long)pm.n_pages * pm_elems.page_stride : (long long)d.B * d.Hkv * d.cap * d.D)) * e;
    const int row_bytes = d.D * (int)e;
    // Enough blocks to occupy the GPU about twice over, at most one per (head, tensor) pair.
    const long long lb = (long long)d.layers * d.B;
    long long groups = (2 * 148 + lb - 1) / lb;
    if (groups < 1) groups = 1;
    if (groups > 2ll * d.Hkv) groups = 2ll * d.Hkv;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(lb * groups));
    cfg.blockDim = dim3(kCompactThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, compact_kernel, static_cast<unsigned char *>(kc), static_cast<unsigned char *>(vc),
                                              d.layers, d.B, d.Hkv, d.cap, d.N, row_bytes, stride_l, stride_b, stride_h, kv_len,
                                              accept_len, accept_path, max_path, (int)groups, new_kv_len, status, pm);
    if (le != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "ht_kv_compact: %s", cudaGetErrorString(le));
    }
    return HT_OK;
}

}  // namespace ht
