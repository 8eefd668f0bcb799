// C ABI of the tree-verify library: argument checks and dispatch.  Declarations and the
// meaning of every argument are in include/ht.h.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "compact.cuh"

namespace ht {

// A named range around every entry point, for timelines taken with a profiler (a no-op without one attached).
struct Range {
    explicit Range(const char *name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

static thread_local char g_err[512] = "no error";

const Knobs &knobs() {
    static const Knobs k = [] {
        Knobs x{false, 0, 0};
        const char *e = getenv("HT_LOG");
        x.log = e && *e && strcmp(e, "0") != 0;
        e = getenv("HT_SPLITS");
        if (e) {
            const long v = strtol(e, nullptr, 10);
            x.splits = v > 0 && v <= 1024 ? (int)v : 0;
        }
        e = getenv("HT_FORCE_PATH");
        if (e) x.path = !strcmp(e, "simt") ? 1 : (!strcmp(e, "mma") ? 2 : (!strcmp(e, "tcgen05") ? 3 : 0));
        return x;
    }();
    return k;
}

void trace(const char *fmt, ...) {
    if (!knobs().log) return;
    va_list ap;
    va_start(ap, fmt);
    fputs("[ht] ", stderr);
    vfprintf(stderr, fmt, ap);
    fputc('\n', stderr);
    va_end(ap);
}

// The descriptor as the knobs of the environment leave it.
static ht_attn_desc with_knobs(const ht_attn_desc &d) {
    ht_attn_desc x = d;
    if (knobs().path == 1) x.flags |= HT_ATTN_FORCE_SIMT;
    if (knobs().splits > 0 && x.num_splits == 0) x.num_splits = knobs().splits;
    return x;
}

// Do the int32 arrays [a, a + n) and [b, b + n) share an element?
static bool overlap_i32(const int32_t *a, const int32_t *b, long long n) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b), len = (uintptr_t)n * sizeof(int32_t);
    return x < y + len && y < x + len;
}

int fail(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int check_launch(const char *what) {
    const cudaError_t e = cudaPeekAtLastError();
    if (e != cudaSuccess) {
        cudaGetLastError();  // clear the non-sticky launch error so later calls are judged on their own
        return fail(HT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    }
    return HT_OK;
}

int check_attn_desc(const ht_attn_desc *d) {
    if (!d) return fail(HT_ERR_INVALID_ARG, "desc is NULL");
    if (d->B < 0 || d->N < 0) return fail(HT_ERR_INVALID_ARG, "negative B or N");
    if (d->Hq <= 0 || d->Hkv <= 0 || d->Hq % d->Hkv != 0)
        return fail(HT_ERR_INVALID_ARG, "Hq = %d must be a positive multiple of Hkv = %d", d->Hq, d->Hkv);
    if (!valid_dtype(d->dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", d->dtype);
    if (d->D != 64 && d->D != 128) return fail(HT_ERR_UNSUPPORTED, "head size %d (64 and 128 are built)", d->D);
    if (d->cap <= 0) return fail(HT_ERR_INVALID_ARG, "cap must be positive");
    if (d->N > d->cap) return fail(HT_ERR_INVALID_ARG, "N = %d rows cannot fit in cap = %d", d->N, d->cap);
    if (d->num_splits < 0 || d->num_splits > 1024) return fail(HT_ERR_INVALID_ARG, "num_splits out of range");
    const long long sh = d->kv_stride_h ? d->kv_stride_h : (long long)d->cap * d->D;
    const long long sb = d->kv_stride_b ? d->kv_stride_b : (long long)d->Hkv * d->cap * d->D;
    if (sh < (long long)d->cap * d->D || sb < sh * d->Hkv)
        return fail(HT_ERR_INVALID_ARG, "cache strides overlap");
    if ((sh * elem_bytes(d->dtype)) % 16 || (sb * elem_bytes(d->dtype)) % 16)
        return fail(HT_ERR_INVALID_ARG, "cache strides must be multiples of 16 bytes");
    return HT_OK;
}

}  // namespace ht

using namespace ht;

extern "C" {

int ht_version(void) { return 100; }

const char *ht_last_error_string(void) { return g_err; }

int ht_transfer(const void *h_src, const void *W, void *out, int B, int k, int d, int dtype,
                void *stream) {
    Range range("ht_transfer");
    trace("ht_transfer B=%d k=%d d=%d dtype=%d", B, k, d, dtype);
    if (B < 0 || k < 0 || d < 0) return fail(HT_ERR_INVALID_ARG, "negative size");
    if (!valid_dtype(dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if ((long long)B * k * d == 0) return HT_OK;
    if (!h_src || !W || !out) return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(h_src) || !aligned16(W) || !aligned16(out))
        return fail(HT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    const int ve = 16 / elem_bytes(dtype);
    if (d % ve) return fail(HT_ERR_UNSUPPORTED, "d = %d must be a multiple of %d for this dtype", d, ve);
    if ((long long)k * d > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "k*d too large");
    return launch_transfer(h_src, W, out, B, k, d, dtype, static_cast<cudaStream_t>(stream));
}

size_t ht_tree_attention_workspace(const ht_attn_desc *desc) {
    if (check_attn_desc(desc) != HT_OK) return 0;
    if (desc->B == 0 || desc->N == 0) return 0;
    // (the maximum over the kernels the descriptor may get, whatever the environment's knobs say)
    size_t need = attn_simt_workspace(*desc, nullptr);
    const ht_attn_desc k = with_knobs(*desc);
    const size_t need_k = attn_simt_workspace(k, nullptr);
    need = need_k > need ? need_k : need;
    if (attn_tc_applicable(*desc)) need = attn_tc_workspace(*desc) > need ? attn_tc_workspace(*desc) : need;
    return (need + 255) / 256 * 256;
}

int ht_tree_attention_launches(const ht_attn_desc *user_desc) {
    if (check_attn_desc(user_desc) != HT_OK) return 0;
    const ht_attn_desc d = with_knobs(*user_desc), *desc = &d;
    if (desc->B == 0 || desc->N == 0) return 0;
    if (attn_tc_applicable(*desc)) return attn_tc_launches(*desc);
    int splits = 1;
    attn_simt_workspace(*desc, &splits);
    return splits > 1 ? 2 : 1;
}

int ht_tree_attention(const ht_attn_desc *user_desc, const void *q, const void *k_cache, const void *v_cache,
                      const int32_t *kv_len, const int32_t *parent, void *out, void *workspace,
                      size_t workspace_bytes, int32_t *status, void *stream) {
    Range range("ht_tree_attention");
    int rc = check_attn_desc(user_desc);
    if (rc != HT_OK) return rc;
    const ht_attn_desc d = with_knobs(*user_desc), *desc = &d;
    trace("ht_tree_attention B=%d N=%d Hq=%d Hkv=%d D=%d cap=%d dtype=%d splits=%d flags=0x%x -> %s", desc->B, desc->N, desc->Hq,
          desc->Hkv, desc->D, desc->cap, desc->dtype, desc->num_splits, desc->flags,
          attn_tc_applicable(*desc) ? "tcgen05" : "simt");
    if (desc->B == 0 || desc->N == 0) return HT_OK;
    if (!q || !k_cache || !v_cache || !kv_len || !parent || !out || !status)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out) ||
        (workspace && !aligned16(workspace)))
        return fail(HT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    const size_t need = ht_tree_attention_workspace(desc);
    if (need > 0 && (!workspace || workspace_bytes < need))
        return fail(HT_ERR_WORKSPACE, "workspace holds %zu bytes, %zu needed", workspace ? workspace_bytes : 0, need);
    if (attn_tc_applicable(*desc))
        return launch_attn_tc(*desc, q, k_cache, v_cache, kv_len, parent, out, workspace, workspace_bytes, status,
                              static_cast<cudaStream_t>(stream));
    return launch_attn_simt(*desc, q, k_cache, v_cache, kv_len, parent, out, workspace, workspace_bytes,
                            status, static_cast<cudaStream_t>(stream));
}

int ht_tree_attention_paged(const ht_attn_desc *desc, const ht_paged_desc *pages, const void *q, const void *k_pages,
                            const void *v_pages, const int32_t *block_table, const int32_t *kv_len,
                            const int32_t *parent, void *out, void *workspace, size_t workspace_bytes,
                            int32_t *status, void *stream) {
    Range range("ht_tree_attention_paged");
    if (desc && pages) trace("ht_tree_attention_paged B=%d N=%d Hq=%d Hkv=%d D=%d page_size=%d max_pages=%d n_pages=%d dtype=%d flags=0x%x", desc->B, desc->N, desc->Hq, desc->Hkv, desc->D, pages->page_size, pages->max_pages, pages->n_pages, desc->dtype, desc->flags);
    if (!desc || !pages) return fail(HT_ERR_INVALID_ARG, "NULL descriptor");
    const int ps = pages->page_size;
    if (ps < 16 || (ps & (ps - 1)) != 0) return fail(HT_ERR_INVALID_ARG, "page_size must be a power of two >= 16");
    if (pages->max_pages <= 0 || pages->n_pages <= 0) return fail(HT_ERR_INVALID_ARG, "max_pages and n_pages must be positive");
    if ((long long)pages->max_pages * ps > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "max_pages * page_size too large");
    if (pages->page_stride < 0 || pages->head_stride < 0 || pages->page_stride % 8 != 0 || pages->head_stride % 8 != 0)
        return fail(HT_ERR_INVALID_ARG, "page strides must be non-negative multiples of 8 elements");
    ht_attn_desc d = *desc;                      // the capacity of a sequence is what its table can hold
    d.cap = pages->max_pages * ps;
    d.kv_stride_b = 0;
    d.kv_stride_h = 0;
    int rc = check_attn_desc(&d);
    if (rc != HT_OK) return rc;
    if (pages->head_stride && pages->head_stride < (long long)ps * d.D)
        return fail(HT_ERR_INVALID_ARG, "head_stride smaller than a page's rows of one head");
    if (pages->page_stride && pages->page_stride < (long long)d.Hkv * ps * d.D)
        return fail(HT_ERR_INVALID_ARG, "page_stride smaller than a page");
    if (d.B == 0 || d.N == 0) return HT_OK;
    if (!q || !k_pages || !v_pages || !block_table || !kv_len || !parent || !out || !status)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out) || (workspace && !aligned16(workspace)))
        return fail(HT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (!attn_tc_applicable(d))
        return fail(HT_ERR_UNSUPPORTED, "paged cache: fp16 / bf16, D = 128, Hq / Hkv a power of two, N <= 1024, B <= 256, no kernel choice by flag, no splits");
    const size_t need = attn_tc_workspace(d);      // does not depend on the capacity
    if (need > 0 && (!workspace || workspace_bytes < need))
        return fail(HT_ERR_WORKSPACE, "workspace holds %zu bytes, %zu needed", workspace ? workspace_bytes : 0, need);
    return launch_attn_tc(d, q, k_pages, v_pages, kv_len, parent, out, workspace, workspace_bytes, status,
                          static_cast<cudaStream_t>(stream), pages, block_table);
}

int ht_verify_greedy(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                     const int32_t *root_pred, int B, int N, int T, int V, int max_path, int32_t *pred,
                     int32_t *accept_len, int32_t *accept_path, int32_t *next_token, int32_t *status,
                     void *stream) {
    Range range("ht_verify_greedy");
    trace("ht_verify_greedy B=%d N=%d T=%d V=%d max_path=%d dtype=%d root_pred=%s", B, N, T, V, max_path, dtype, root_pred ? "given" : "none");
    if (B < 0 || N < 0 || T < 0 || T > N) return fail(HT_ERR_INVALID_ARG, "need 0 <= T <= N and B >= 0");
    if (!valid_dtype(dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (B == 0) return HT_OK;
    if (N == 0 || V <= 0) return fail(HT_ERR_INVALID_ARG, "N and V must be positive");
    if (max_path <= 0 || max_path > 255) return fail(HT_ERR_INVALID_ARG, "max_path must be in 1..255");
    if (!logits || !parent || !pred || !accept_len || !accept_path || !next_token || !status || (T > 0 && !tokens))
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(logits)) return fail(HT_ERR_INVALID_ARG, "logits must be 16-byte aligned");
    if ((long long)B * N > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "B*N too large");
    return launch_verify(logits, dtype, tokens, parent, root_pred, B, N, T, V, max_path, N, pred, accept_len,
                         accept_path, next_token, status, nullptr, static_cast<cudaStream_t>(stream));
}

static int check_cache_desc(const ht_cache_desc *desc, int max_path) {
    if (!desc) return fail(HT_ERR_INVALID_ARG, "desc is NULL");
    if (desc->layers <= 0 || desc->B < 0 || desc->Hkv <= 0 || desc->cap <= 0 || desc->D <= 0 || desc->N < 0)
        return fail(HT_ERR_INVALID_ARG, "bad cache sizes");
    if (!valid_dtype(desc->dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", desc->dtype);
    if (max_path <= 0 || max_path > 64) return fail(HT_ERR_INVALID_ARG, "max_path must be in 1..64");
    const int row_bytes = desc->D * elem_bytes(desc->dtype);
    if (row_bytes % 16) return fail(HT_ERR_UNSUPPORTED, "a cache row must be a multiple of 16 bytes");
    if ((long long)max_path * (row_bytes / 16) > 4096)
        return fail(HT_ERR_UNSUPPORTED, "max_path * row size too large for one block");
    const long long e = elem_bytes(desc->dtype);
    if ((desc->stride_layer * e) % 16 || (desc->stride_b * e) % 16 || (desc->stride_h * e) % 16)
        return fail(HT_ERR_INVALID_ARG, "cache strides must be multiples of 16 bytes");
    if (2ll * desc->layers * desc->B * desc->Hkv > 0x7fffffffLL)
        return fail(HT_ERR_UNSUPPORTED, "too many (layer, sequence, head) units");
    return HT_OK;
}

int ht_verify_greedy_compact(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                             const int32_t *root_pred, int B, int N, int T, int V, int max_path, int rows,
                             int32_t *pred, int32_t *accept_len, int32_t *accept_path, int32_t *next_token,
                             int32_t *status, void *k_cache, void *v_cache, const ht_cache_desc *desc,
                             const int32_t *kv_len, int32_t *new_kv_len, int32_t *compact_status, void *stream) {
    Range range("ht_verify_greedy_compact");
    trace("ht_verify_greedy_compact B=%d N=%d T=%d V=%d max_path=%d dtype=%d layers=%d", B, N, T, V, max_path, dtype, desc ? desc->layers : -1);
    if (B < 0 || N < 0 || T < 0 || T > N) return fail(HT_ERR_INVALID_ARG, "need 0 <= T <= N and B >= 0");
    if (!valid_dtype(dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    int rc = check_cache_desc(desc, max_path);
    if (rc != HT_OK) return rc;
    if (desc->B != B || desc->N != N) return fail(HT_ERR_INVALID_ARG, "the cache descriptor's B and N must be those of the logits");
    if (B == 0) return HT_OK;
    if (N == 0 || V <= 0) return fail(HT_ERR_INVALID_ARG, "N and V must be positive");
    if (rows == 0) rows = T > 0 ? T : 1;
    if (rows < T || rows < 1 || rows > N) return fail(HT_ERR_INVALID_ARG, "rows = %d must lie in [max(T, 1), N]", rows);
    if (!logits || !parent || !pred || !accept_len || !accept_path || !next_token || !status || (T > 0 && !tokens) ||
        !k_cache || !v_cache || !kv_len || !new_kv_len || !compact_status)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(logits) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(HT_ERR_INVALID_ARG, "logits and caches must be 16-byte aligned");
    if ((long long)B * N > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "B*N too large");
    if (overlap_i32(new_kv_len, kv_len, B) || overlap_i32(new_kv_len, accept_len, B))
        return fail(HT_ERR_INVALID_ARG, "new_kv_len must not overlap kv_len or accept_len: every block of a sequence reads them");
    // about one compaction item per thread block of the verification's grid (it holds B * rows blocks, or as many as
    // the GPU takes at once, whichever is less: four per SM)
    const long long grid_guess = (long long)B * rows < 4 * 148 ? (long long)B * rows : 4 * 148;
    const CompactArgs c = make_compact_args(k_cache, v_cache, *desc, kv_len, accept_len, accept_path, max_path, new_kv_len,
                                            compact_status, PageMap{}, (int)grid_guess);
    return launch_verify(logits, dtype, tokens, parent, root_pred, B, N, T, V, max_path, rows, pred, accept_len,
                         accept_path, next_token, status, &c, static_cast<cudaStream_t>(stream));
}

int ht_kv_compact(void *k_cache, void *v_cache, const ht_cache_desc *desc, const int32_t *kv_len,
                  const int32_t *accept_len, const int32_t *accept_path, int max_path,
                  int32_t *new_kv_len, int32_t *status, void *stream) {
    Range range("ht_kv_compact");
    if (desc) trace("ht_kv_compact layers=%d B=%d Hkv=%d cap=%d D=%d N=%d max_path=%d", desc->layers, desc->B, desc->Hkv, desc->cap, desc->D, desc->N, max_path);
    if (!desc) return fail(HT_ERR_INVALID_ARG, "desc is NULL");
    if (desc->layers <= 0 || desc->B < 0 || desc->Hkv <= 0 || desc->cap <= 0 || desc->D <= 0 || desc->N < 0)
        return fail(HT_ERR_INVALID_ARG, "bad cache sizes");
    if (!valid_dtype(desc->dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", desc->dtype);
    if (max_path <= 0 || max_path > 64) return fail(HT_ERR_INVALID_ARG, "max_path must be in 1..64");
    if (desc->B == 0) return HT_OK;
    const int row_bytes = desc->D * elem_bytes(desc->dtype);
    if (row_bytes % 16) return fail(HT_ERR_UNSUPPORTED, "a cache row must be a multiple of 16 bytes");
    if ((long long)max_path * (row_bytes / 16) > 4096)
        return fail(HT_ERR_UNSUPPORTED, "max_path * row size too large for one block");
    if (!kv_len || !accept_len || !accept_path || !new_kv_len || !status || !k_cache || !v_cache)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(k_cache) || !aligned16(v_cache)) return fail(HT_ERR_INVALID_ARG, "caches must be 16-byte aligned");
    const long long e = elem_bytes(desc->dtype);
    if ((desc->stride_layer * e) % 16 || (desc->stride_b * e) % 16 || (desc->stride_h * e) % 16)
        return fail(HT_ERR_INVALID_ARG, "cache strides must be multiples of 16 bytes");
    if (2ll * desc->layers * desc->B * desc->Hkv > 0x7fffffffLL)
        return fail(HT_ERR_UNSUPPORTED, "too many (layer, sequence, head) units");
    if (overlap_i32(new_kv_len, kv_len, desc->B) || overlap_i32(new_kv_len, accept_len, desc->B))
        return fail(HT_ERR_INVALID_ARG, "new_kv_len must not overlap kv_len or accept_len: every block of a sequence reads them");
    return launch_compact(k_cache, v_cache, *desc, kv_len, accept_len, accept_path, max_path, new_kv_len, status,
                          static_cast<cudaStream_t>(stream));
}

int ht_draft_tree(const void *logits, int dtype, int B, int rows, int V, int first_row, int P, int K,
                  const int32_t *tmpl_parent, const int32_t *tmpl_rank, int T, const int32_t *root_token,
                  const int32_t *base_pos, int32_t *topk, int32_t *tokens, int32_t *pos, int32_t *status,
                  void *stream) {
    Range range("ht_draft_tree");
    trace("ht_draft_tree B=%d rows=%d V=%d first_row=%d P=%d K=%d dtype=%d", B, rows, V, first_row, P, K, dtype);
    if (B < 0 || rows < 0 || P < 0 || first_row < 0) return fail(HT_ERR_INVALID_ARG, "negative size");
    if (!valid_dtype(dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (B == 0) return HT_OK;
    if (T <= 0 || V <= 0) return fail(HT_ERR_INVALID_ARG, "T and V must be positive");
    if (K < 1 || K > 16 || K > V) return fail(HT_ERR_INVALID_ARG, "K = %d must lie in [1, min(16, V)]", K);
    if ((long long)first_row + P > rows) return fail(HT_ERR_INVALID_ARG, "pseudo rows [%d, %d) exceed the %d rows", first_row, first_row + P, rows);
    if (!tmpl_parent || !tmpl_rank || !base_pos || !tokens || !pos || !status || (P > 0 && (!logits || !topk)))
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (P > 0 && !aligned16(logits)) return fail(HT_ERR_INVALID_ARG, "logits must be 16-byte aligned");
    if ((long long)B * (P > 0 ? P : 1) > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "B*P too large");
    return launch_draft(logits, dtype, B, rows, V, first_row, P, K, tmpl_parent, tmpl_rank, T, root_token, base_pos,
                        topk, tokens, pos, status, static_cast<cudaStream_t>(stream));
}

int ht_rope_kv_append(const ht_attn_desc *desc, const void *q_in, const void *k_in, const void *v_in, const int32_t *pos,
                      const int32_t *kv_len, float rope_base, void *q_out, void *k_cache, void *v_cache, int32_t *status,
                      void *stream) {
    Range range("ht_rope_kv_append");
    if (desc) trace("ht_rope_kv_append B=%d N=%d Hq=%d Hkv=%d D=%d dtype=%d", desc->B, desc->N, desc->Hq, desc->Hkv, desc->D, desc->dtype);
    int rc = check_attn_desc(desc);
    if (rc != HT_OK) return rc;
    if (desc->B == 0 || desc->N == 0) return HT_OK;
    if (!(rope_base > 1.f)) return fail(HT_ERR_INVALID_ARG, "rope_base must exceed 1");
    if (!q_in || !k_in || !v_in || !pos || !kv_len || !q_out || !k_cache || !v_cache || !status)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(q_in) || !aligned16(k_in) || !aligned16(v_in) || !aligned16(q_out) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(HT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if ((long long)desc->B * desc->N > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "B*N too large");
    return launch_rope(*desc, q_in, k_in, v_in, pos, kv_len, rope_base, q_out, k_cache, v_cache, status,
                       static_cast<cudaStream_t>(stream));
}

static int check_paged_desc(const ht_paged_desc *pages, int Hkv, int D) {
    if (!pages) return fail(HT_ERR_INVALID_ARG, "NULL descriptor");
    const int ps = pages->page_size;
    if (ps < 16 || (ps & (ps - 1)) != 0) return fail(HT_ERR_INVALID_ARG, "page_size must be a power of two >= 16");
    if (pages->max_pages <= 0 || pages->n_pages <= 0) return fail(HT_ERR_INVALID_ARG, "max_pages and n_pages must be positive");
    if ((long long)pages->max_pages * ps > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "max_pages * page_size too large");
    if (pages->page_stride < 0 || pages->head_stride < 0 || pages->page_stride % 8 != 0 || pages->head_stride % 8 != 0)
        return fail(HT_ERR_INVALID_ARG, "page strides must be non-negative multiples of 8 elements");
    if (pages->head_stride && pages->head_stride < (long long)ps * D)
        return fail(HT_ERR_INVALID_ARG, "head_stride smaller than a page's rows of one head");
    if (pages->page_stride && pages->page_stride < (long long)Hkv * ps * D)
        return fail(HT_ERR_INVALID_ARG, "page_stride smaller than a page");
    return HT_OK;
}

int ht_rope_kv_append_paged(const ht_attn_desc *desc, const ht_paged_desc *pages, const void *q_in, const void *k_in,
                            const void *v_in, const int32_t *pos, const int32_t *kv_len, const int32_t *block_table,
                            float rope_base, void *q_out, void *k_pages, void *v_pages, int32_t *status, void *stream) {
    Range range("ht_rope_kv_append_paged");
    if (desc && pages) trace("ht_rope_kv_append_paged B=%d N=%d Hq=%d Hkv=%d D=%d page_size=%d dtype=%d", desc->B, desc->N, desc->Hq, desc->Hkv, desc->D, pages->page_size, desc->dtype);
    if (!desc) return fail(HT_ERR_INVALID_ARG, "NULL descriptor");
    int rc = check_paged_desc(pages, desc->Hkv, desc->D);
    if (rc != HT_OK) return rc;
    ht_attn_desc d = *desc;
    d.cap = pages->max_pages * pages->page_size;
    d.kv_stride_b = 0;
    d.kv_stride_h = 0;
    rc = check_attn_desc(&d);
    if (rc != HT_OK) return rc;
    if (d.B == 0 || d.N == 0) return HT_OK;
    if (!(rope_base > 1.f)) return fail(HT_ERR_INVALID_ARG, "rope_base must exceed 1");
    if (!q_in || !k_in || !v_in || !pos || !kv_len || !block_table || !q_out || !k_pages || !v_pages || !status)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(q_in) || !aligned16(k_in) || !aligned16(v_in) || !aligned16(q_out) || !aligned16(k_pages) || !aligned16(v_pages))
        return fail(HT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if ((long long)d.B * d.N > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "B*N too large");
    return launch_rope(d, q_in, k_in, v_in, pos, kv_len, rope_base, q_out, k_pages, v_pages, status,
                       static_cast<cudaStream_t>(stream), make_page_map(pages, block_table, d.Hkv, d.D));
}

int ht_kv_compact_paged(void *k_pages, void *v_pages, const ht_cache_desc *desc, const ht_paged_desc *pages,
                        const int32_t *block_table, const int32_t *kv_len, const int32_t *accept_len,
                        const int32_t *accept_path, int max_path, int32_t *new_kv_len, int32_t *status, void *stream) {
    Range range("ht_kv_compact_paged");
    if (desc && pages) trace("ht_kv_compact_paged layers=%d B=%d Hkv=%d D=%d N=%d page_size=%d max_path=%d", desc->layers, desc->B, desc->Hkv, desc->D, desc->N, pages->page_size, max_path);
    if (!desc) return fail(HT_ERR_INVALID_ARG, "desc is NULL");
    if (desc->layers <= 0 || desc->B < 0 || desc->Hkv <= 0 || desc->D <= 0 || desc->N < 0)
        return fail(HT_ERR_INVALID_ARG, "bad cache sizes");
    int rc = check_paged_desc(pages, desc->Hkv, desc->D);
    if (rc != HT_OK) return rc;
    if (!valid_dtype(desc->dtype)) return fail(HT_ERR_INVALID_ARG, "unknown dtype %d", desc->dtype);
    if (max_path <= 0 || max_path > 64) return fail(HT_ERR_INVALID_ARG, "max_path must be in 1..64");
    if (desc->B == 0) return HT_OK;
    const int row_bytes = desc->D * elem_bytes(desc->dtype);
    if (row_bytes % 16) return fail(HT_ERR_UNSUPPORTED, "a cache row must be a multiple of 16 bytes");
    if ((long long)max_path * (row_bytes / 16) > 4096)
        return fail(HT_ERR_UNSUPPORTED, "max_path * row size too large for one block");
    if (!kv_len || !accept_len || !accept_path || !new_kv_len || !status || !k_pages || !v_pages || !block_table)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(k_pages) || !aligned16(v_pages)) return fail(HT_ERR_INVALID_ARG, "pools must be 16-byte aligned");
    const long long e = elem_bytes(desc->dtype);
    if (desc->stride_layer < 0 || (desc->stride_layer * e) % 16) return fail(HT_ERR_INVALID_ARG, "stride_layer must be a multiple of 16 bytes");
    if (2ll * desc->layers * desc->B * desc->Hkv > 0x7fffffffLL)
        return fail(HT_ERR_UNSUPPORTED, "too many (layer, sequence, head) units");
    if (overlap_i32(new_kv_len, kv_len, desc->B) || overlap_i32(new_kv_len, accept_len, desc->B))
        return fail(HT_ERR_INVALID_ARG, "new_kv_len must not overlap kv_len or accept_len: every block of a sequence reads them");
    ht_cache_desc d = *desc;
    d.cap = pages->max_pages * pages->page_size;
    return launch_compact(k_pages, v_pages, d, kv_len, accept_len, accept_path, max_path, new_kv_len, status,
                          static_cast<cudaStream_t>(stream), make_page_map(pages, block_table, d.Hkv, d.D));
}

}  // extern "C"
