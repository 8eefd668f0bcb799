// Shared host/device helpers of the tree-verify library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ht.h"

namespace ht {

// Records a message for ht_last_error_string() and returns `code`.
int fail(int code, const char *fmt, ...);

// Host-side checks of an attention descriptor (sizes, dtype, strides).
int check_attn_desc(const ht_attn_desc *d);

// Checks the launch status of the kernel just enqueued.
int check_launch(const char *what);

// Knobs read once from the environment, for cross-checks and bug reports (never needed for results):
//   HT_LOG=1                       every entry point prints its arguments and the kernel it chose to stderr
//   HT_FORCE_PATH=simt|mma|tcgen05 attention on the fp32-ALU kernel (simt); the projection of 16-bit inputs on the
//                                  warp-level kernel (mma) or, where its shape allows, on the tcgen05 kernel
//   HT_SPLITS=n                    attention: n KV splits where the descriptor leaves the choice (num_splits == 0),
//                                  which selects the split-KV ALU kernel, as an explicit num_splits does
struct Knobs {
    bool log;
    int splits;           // 0: not set
    int path;             // 0: not set, 1: simt, 2: mma, 3: tcgen05
};
const Knobs &knobs();
void trace(const char *fmt, ...);      // a line on stderr when HT_LOG is set

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int elem_bytes(int dtype) { return dtype == HT_F32 ? 4 : 2; }

inline bool valid_dtype(int dtype) { return dtype == HT_F32 || dtype == HT_F16 || dtype == HT_BF16; }

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_float<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Number of elements of T in one 16-byte vector.
template <typename T> struct Vec16 { static constexpr int n = 16 / sizeof(T); };

// Unpack a 16-byte vector of T into floats.
template <typename T> __device__ __forceinline__ void unpack16(const uint4 &raw, float *f);
template <> __device__ __forceinline__ void unpack16<float>(const uint4 &raw, float *f) {
    f[0] = __uint_as_float(raw.x); f[1] = __uint_as_float(raw.y);
    f[2] = __uint_as_float(raw.z); f[3] = __uint_as_float(raw.w);
}
template <> __device__ __forceinline__ void unpack16<__half>(const uint4 &raw, float *f) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __half2 h2 = *reinterpret_cast<const __half2 *>(&w[i]);
        float2 f2 = __half22float2(h2);
        f[2 * i] = f2.x; f[2 * i + 1] = f2.y;
    }
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4 &raw, float *f) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {           // bf16 is the upper half of an fp32
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ uint4 ld_nc16(const void *p) {   // streaming 16-byte load
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Paged cache as the row-moving kernels see it: cache row r of sequence b is row r & (page_size - 1) of page
// table[b * max_pages + (r >> shift)].  table == nullptr: contiguous cache.  Strides in elements.
struct PageMap {
    const int32_t *table;
    int shift, max_pages, n_pages;
    long long page_stride, head_stride;
};
inline PageMap make_page_map(const ht_paged_desc *pg, const int32_t *table, int Hkv, int D) {
    PageMap m{};
    if (!pg) return m;
    m.table = table;
    while ((1 << m.shift) < pg->page_size) ++m.shift;
    m.max_pages = pg->max_pages;
    m.n_pages = pg->n_pages;
    m.head_stride = pg->head_stride ? pg->head_stride : (long long)pg->page_size * D;
    m.page_stride = pg->page_stride ? pg->page_stride : (long long)Hkv * pg->page_size * D;
    return m;
}

// Entry points of the individual kernels' host launchers (defined in the .cu files).
int launch_transfer(const void *h, const void *W, void *out, int B, int k, int d, int dtype, cudaStream_t s);
bool transfer_tc_applicable(int B, int k, int d, int dtype);
int transfer_tc_tile(int B, int R, int sms);
int launch_transfer_tc(const void *h, const void *W, void *out, int B, int k, int d, int dtype, cudaStream_t s);
size_t attn_simt_workspace(const ht_attn_desc &d, int *splits_out);
int launch_attn_simt(const ht_attn_desc &d, const void *q, const void *kc, const void *vc,
                     const int32_t *kv_len, const int32_t *parent, void *out, void *ws, size_t ws_bytes,
                     int32_t *status, cudaStream_t s);
bool attn_tc_applicable(const ht_attn_desc &d);
size_t attn_tc_workspace(const ht_attn_desc &d);
int attn_tc_launches(const ht_attn_desc &d);      // kernels one call enqueues (contiguous cache)
// `pages` / `block_table` null: contiguous cache (kc, vc as in ht_tree_attention); else the page pools.
int launch_attn_tc(const ht_attn_desc &d, const void *q, const void *kc, const void *vc, const int32_t *kv_len,
                   const int32_t *parent, void *out, void *ws, size_t ws_bytes, int32_t *status, cudaStream_t s,
                   const ht_paged_desc *pages = nullptr, const int32_t *block_table = nullptr);
struct CompactArgs;
// rows: logits rows per sequence whose argmax is taken (T <= rows <= N); compact: the compaction to run in the same
// launch, or null.
int launch_verify(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                  const int32_t *root_pred, int B, int N, int T, int V, int max_path, int rows, int32_t *pred,
                  int32_t *accept_len, int32_t *accept_path, int32_t *next_token, int32_t *status,
                  const CompactArgs *compact, cudaStream_t s);
int launch_draft(const void *logits, int dtype, int B, int rows, int V, int first_row, int P, int K,
                 const int32_t *tmpl_parent, const int32_t *tmpl_rank, int Tn, const int32_t *root_token,
                 const int32_t *base_pos, int32_t *topk, int32_t *tokens, int32_t *pos, int32_t *status, cudaStream_t s);
int launch_rope(const ht_attn_desc &d, const void *q_in, const void *k_in, const void *v_in, const int32_t *pos,
                const int32_t *kv_len, float base, void *q_out, void *kc, void *vc, int32_t *status, cudaStream_t s,
                const PageMap &pm = PageMap{});
int launch_compact(void *kc, void *vc, const ht_cache_desc &d, const int32_t *kv_len,
                   const int32_t *accept_len, const int32_t *accept_path, int max_path,
                   int32_t *new_kv_len, int32_t *status, cudaStream_t s, const PageMap &pm = PageMap{});

}  // namespace ht
