/*
 * ht_oracle.c -- CPU oracle for the tree-verify step of Hidden Transfer decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what the
 * GPU library must compute.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may build or call it; the product path never does.  It shares no
 * code, header, table or helper with the CUDA sources.
 *
 * Inputs arrive as float arrays that hold the dtype-rounded values exactly (every
 * fp16 / bf16 / fp32 value is a float); all arithmetic below is double precision.
 * There is no blocking, tiling, online softmax or fusion: each function is the
 * definition written out.
 *
 * Layouts (row-major, last index fastest):
 *   q, out      [B, N, Hq, D]
 *   k/v cache   [B, Hkv, cap, D]; sequence b holds kv_len[b] context rows followed by
 *               the N rows of the flattened tree (tree row c lives at cache row
 *               kv_len[b] + c)
 *   parent      [B, N]  parent[b][r] in [-1, r): -1 attaches the row to the context
 *   logits      [B, N, V]
 *   tokens      [B, T]  (the first T of the N rows are draft-tree nodes, the rest are
 *               pseudo positions created by the hidden-transfer projection)
 *
 * What each function follows in the paper:
 *   transfer         -- Section "Training stage", the displayed equation
 *                       h~ = W^i_{t_i} . h with W in R^{d x d} (plain linear map)
 *   tree attention   -- Section "Tree attention": a token attends only to its
 *                       ancestors in the tree (and the context), positions kept;
 *                       pseudo rows follow the rule of Section "Training stage"
 *                       (a pseudo state sees the context up to its source, earlier
 *                       pseudo states and itself) and the "No masked" setting of the
 *                       ablation study, which are expressed as ordinary parent links.
 *   greedy verify    -- Fig. 2 caption ("find the last accepted token position"),
 *                       Section "Inference stage", Section "Setup" (greedy sampling,
 *                       output identical to auto-regressive decoding)
 *   compaction       -- implied by verifying under a KV cache (Fig. 1 caption,
 *                       Section "Inference stage"): only the accepted path's K/V stay.
 *
 * Pins (tests/test_oracle_*.py): brute-force causal attention on gathered paths,
 * chain == causal multi-token decode via a library SDPA, independent roots ==
 * single-token decodes, closed forms (q = 0, constant V, L = 0), convex-hull bounds,
 * GQA identities, relabelling invariance, numpy mat-vec for the transfer, exhaustive
 * enumeration of small trees for acceptance, aliasing cases for compaction, and a toy
 * lossless decoding loop.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define HT_ORACLE_OK 0
#define HT_ORACLE_BAD_TREE 1
#define HT_ORACLE_BAD_LEN 2
#define HT_ORACLE_BAD_PATH 3
#define HT_ORACLE_PATH_TOO_LONG 4
#define HT_ORACLE_NOMEM 5

/* ------------------------------------------------------------------------------------
 * Hidden-transfer projection: out[b][i][r] = sum_c W[i][r][c] * h[b][c].
 * W[i] is the i-th transfer step's d x d matrix acting on a column vector, so its
 * rows are output features.  No bias, no activation.
 * ---------------------------------------------------------------------------------- */
int ht_oracle_transfer(const float *h, const float *W, double *out, int B, int k, int d)
{
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < k; ++i)
            for (int r = 0; r < d; ++r) {
                double acc = 0.0;
                const float *wrow = W + ((size_t)i * d + r) * d;
                const float *hv = h + (size_t)b * d;
                for (int c = 0; c < d; ++c)
                    acc += (double)wrow[c] * (double)hv[c];
                out[((size_t)b * k + i) * d + r] = acc;
            }
    return HT_ORACLE_OK;
}

/* A flattened tree is legal when every parent index precedes its child. */
static int tree_is_legal(const int32_t *parent, int N)
{
    for (int r = 0; r < N; ++r)
        if (parent[r] < -1 || parent[r] >= r)
            return 0;
    return 1;
}

int ht_oracle_check_tree(const int32_t *parent, int B, int N)
{
    for (int b = 0; b < B; ++b)
        if (!tree_is_legal(parent + (size_t)b * N, N))
            return HT_ORACLE_BAD_TREE;
    return HT_ORACLE_OK;
}

/* Root-to-node path of row r, root first.  Returns its number of nodes. */
static int root_path(const int32_t *parent, int r, int32_t *path)
{
    int n = 0;
    for (int c = r; c >= 0; c = parent[c])
        path[n++] = c;
    for (int i = 0, j = n - 1; i < j; ++i, --j) {
        int32_t t = path[i];
        path[i] = path[j];
        path[j] = t;
    }
    return n;
}

/* Textbook softmax(scale * q.K^T).V over an explicit list of cache rows. */
static void attend_rows(const float *qrow, const float *kbase, const float *vbase,
                        const int32_t *rows, int n_rows, int D, double scale,
                        double *score, double *out)
{
    double smax = -INFINITY;
    for (int j = 0; j < n_rows; ++j) {
        const float *krow = kbase + (size_t)rows[j] * D;
        double s = 0.0;
        for (int x = 0; x < D; ++x)
            s += (double)qrow[x] * (double)krow[x];
        s *= scale;
        score[j] = s;
        if (s > smax)
            smax = s;
    }
    double denom = 0.0;
    for (int j = 0; j < n_rows; ++j) {
        score[j] = exp(score[j] - smax);
        denom += score[j];
    }
    for (int x = 0; x < D; ++x)
        out[x] = 0.0;
    for (int j = 0; j < n_rows; ++j) {
        const float *vrow = vbase + (size_t)rows[j] * D;
        double w = score[j] / denom;
        for (int x = 0; x < D; ++x)
            out[x] += w * (double)vrow[x];
    }
}

/* ------------------------------------------------------------------------------------
 * Tree attention, definition form ("path form"): the keys and values of row r are the
 * context rows 0..L-1 followed by the rows of r's root-to-node path; the output is
 * ordinary attention of q_r over that list.  Computes the selected (b, h, r) triples
 * only, so that full-size workloads can be sampled.  sel == NULL means every triple in
 * [B, N, Hq] order, in which case out is the full [B, N, Hq, D] tensor.
 * ---------------------------------------------------------------------------------- */
int ht_oracle_tree_attention_rows(const float *q, const float *k_cache, const float *v_cache,
                                  const int32_t *kv_len, const int32_t *parent,
                                  int B, int N, int Hq, int Hkv, int D, int cap, double scale,
                                  const int32_t *sel, long n_sel, double *out)
{
    if (Hkv <= 0 || Hq % Hkv != 0)
        return HT_ORACLE_BAD_LEN;
    const int g = Hq / Hkv;
    for (int b = 0; b < B; ++b) {
        if (!tree_is_legal(parent + (size_t)b * N, N))
            return HT_ORACLE_BAD_TREE;
        if (kv_len[b] < 0 || (long)kv_len[b] + N > cap)
            return HT_ORACLE_BAD_LEN;
    }
    const long total = sel ? n_sel : (long)B * N * Hq;
    int status = HT_ORACLE_OK;
#pragma omp parallel for schedule(dynamic, 8)
    for (long i = 0; i < total; ++i) {
        int b, r, h;
        if (sel) {
            b = sel[3 * i + 0];
            h = sel[3 * i + 1];
            r = sel[3 * i + 2];
        } else {
            b = (int)(i / ((long)N * Hq));
            r = (int)((i / Hq) % N);
            h = (int)(i % Hq);
        }
        const int L = kv_len[b];
        const int32_t *par = parent + (size_t)b * N;
        int32_t *rows = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L + N));
        double *score = (double *)malloc(sizeof(double) * (size_t)(L + N));
        if (!rows || !score) {
            status = HT_ORACLE_NOMEM;
            free(rows);
            free(score);
            continue;
        }
        int n_rows = 0;
        for (int j = 0; j < L; ++j)
            rows[n_rows++] = j;
        int32_t *path = rows + n_rows;
        int plen = root_path(par, r, path);
        for (int j = 0; j < plen; ++j)
            path[j] += L;
        n_rows += plen;
        const int hk = h / g;
        const float *qrow = q + (((size_t)b * N + r) * Hq + h) * D;
        const float *kbase = k_cache + ((size_t)b * Hkv + hk) * (size_t)cap * D;
        const float *vbase = v_cache + ((size_t)b * Hkv + hk) * (size_t)cap * D;
        double *o = sel ? out + (size_t)i * D : out + (((size_t)b * N + r) * Hq + h) * D;
        attend_rows(qrow, kbase, vbase, rows, n_rows, D, scale, score, o);
        free(rows);
        free(score);
    }
    return status;
}

/* ------------------------------------------------------------------------------------
 * Tree attention, dense-mask form: build the N x N visibility matrix M[r][c] (c is r
 * or an ancestor of r) by the recurrence M[r] = M[parent[r]] + {r}, then run masked
 * attention over all L + N rows with the masked entries left out of the softmax.
 * An independent second statement of the same definition; the tests require the two
 * forms to agree.
 * ---------------------------------------------------------------------------------- */
int ht_oracle_tree_attention_mask(const float *q, const float *k_cache, const float *v_cache,
                                  const int32_t *kv_len, const int32_t *parent,
                                  int B, int N, int Hq, int Hkv, int D, int cap, double scale,
                                  double *out)
{
    if (Hkv <= 0 || Hq % Hkv != 0)
        return HT_ORACLE_BAD_LEN;
    const int g = Hq / Hkv;
    for (int b = 0; b < B; ++b) {
        const int32_t *par = parent + (size_t)b * N;
        const int L = kv_len[b];
        if (!tree_is_legal(par, N))
            return HT_ORACLE_BAD_TREE;
        if (L < 0 || (long)L + N > cap)
            return HT_ORACLE_BAD_LEN;
        unsigned char *M = (unsigned char *)calloc((size_t)N * N, 1);
        double *s = (double *)malloc(sizeof(double) * (size_t)(L + N));
        if (!M || !s) {
            free(M);
            free(s);
            return HT_ORACLE_NOMEM;
        }
        for (int r = 0; r < N; ++r) {
            if (par[r] >= 0)
                memcpy(M + (size_t)r * N, M + (size_t)par[r] * N, (size_t)N);
            M[(size_t)r * N + r] = 1;
        }
        for (int r = 0; r < N; ++r)
            for (int h = 0; h < Hq; ++h) {
                const int hk = h / g;
                const float *qrow = q + (((size_t)b * N + r) * Hq + h) * D;
                const float *kbase = k_cache + ((size_t)b * Hkv + hk) * (size_t)cap * D;
                const float *vbase = v_cache + ((size_t)b * Hkv + hk) * (size_t)cap * D;
                double smax = -INFINITY;
                for (int j = 0; j < L + N; ++j) {
                    int visible = (j < L) || M[(size_t)r * N + (j - L)];
                    if (!visible) {
                        s[j] = -INFINITY;
                        continue;
                    }
                    double acc = 0.0;
                    for (int x = 0; x < D; ++x)
                        acc += (double)qrow[x] * (double)kbase[(size_t)j * D + x];
                    s[j] = acc * scale;
                    if (s[j] > smax)
                        smax = s[j];
                }
                double denom = 0.0;
                for (int j = 0; j < L + N; ++j) {
                    s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - smax);
                    denom += s[j];
                }
                double *o = out + (((size_t)b * N + r) * Hq + h) * D;
                for (int x = 0; x < D; ++x) {
                    double acc = 0.0;
                    for (int j = 0; j < L + N; ++j)
                        acc += s[j] * (double)vbase[(size_t)j * D + x];
                    o[x] = acc / denom;
                }
            }
        free(M);
        free(s);
    }
    return HT_ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Greedy prediction per row: index of the largest logit; the lowest index wins ties; a
 * NaN never wins; a row of NaNs gives 0.  Comparisons are exact on the stored values.
 * ---------------------------------------------------------------------------------- */
int ht_oracle_row_argmax(const float *logits, long rows, int V, int32_t *pred)
{
    for (long r = 0; r < rows; ++r) {
        const float *row = logits + (size_t)r * V;
        int best = -1;
        float bv = 0.0f;
        for (int v = 0; v < V; ++v) {
            float x = row[v];
            if (x != x)
                continue;
            if (best < 0 || x > bv) {
                best = v;
                bv = x;
            }
        }
        pred[r] = best < 0 ? 0 : best;
    }
    return HT_ORACLE_OK;
}

/* Does draft node c carry the token greedy decoding would have produced after its
 * parent?  A top-level node is checked against root_pred (the argmax carried over from
 * the previous round) when one is given and is taken as known-correct otherwise. */
static int node_matches(const int32_t *tokens, const int32_t *parent, const int32_t *pred,
                        const int32_t *root_pred_b, int c)
{
    if (parent[c] < 0)
        return root_pred_b ? (tokens[c] == *root_pred_b) : 1;
    return tokens[c] == pred[parent[c]];
}

static void write_result(const int32_t *parent, const int32_t *pred, const int32_t *root_pred_b,
                         int best_node, int best_len, int max_path,
                         int32_t *accept_len, int32_t *accept_path, int32_t *next_token,
                         int32_t *status)
{
    for (int j = 0; j < max_path; ++j)
        accept_path[j] = -1;
    if (best_len > max_path) {
        *status = HT_ORACLE_PATH_TOO_LONG;
        *accept_len = 0;
        *next_token = -1;
        return;
    }
    *accept_len = best_len;
    if (best_len == 0) {
        *next_token = root_pred_b ? *root_pred_b : -1;
        return;
    }
    int j = best_len - 1;
    for (int c = best_node; c >= 0; c = parent[c])
        accept_path[j--] = c;
    *next_token = pred[best_node];
}

/* ------------------------------------------------------------------------------------
 * Greedy acceptance, definition form: enumerate the root path of every one of the T
 * draft nodes; a path is valid when every node on it matches; the answer is the valid
 * path with the most nodes, the smallest terminal index breaking ties.  accept_len is
 * the number of nodes on it, accept_path lists them root first (-1 padded), next_token
 * is the model's prediction after its last node (or root_pred when nothing is
 * accepted).  pred is [B, N]; only rows < T are consulted.
 * ---------------------------------------------------------------------------------- */
int ht_oracle_accept_enumerate(const int32_t *tokens, const int32_t *parent, const int32_t *pred,
                               const int32_t *root_pred, int B, int N, int T, int max_path,
                               int32_t *accept_len, int32_t *accept_path, int32_t *next_token,
                               int32_t *status)
{
    int32_t *path = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
    if (!path)
        return HT_ORACLE_NOMEM;
    for (int b = 0; b < B; ++b) {
        const int32_t *par = parent + (size_t)b * N;
        const int32_t *tok = tokens + (size_t)b * T;
        const int32_t *prd = pred + (size_t)b * N;
        const int32_t *rp = root_pred ? root_pred + b : NULL;
        status[b] = HT_ORACLE_OK;
        if (!tree_is_legal(par, N)) {
            status[b] = HT_ORACLE_BAD_TREE;
            accept_len[b] = 0;
            next_token[b] = -1;
            for (int j = 0; j < max_path; ++j)
                accept_path[(size_t)b * max_path + j] = -1;
            continue;
        }
        int best_node = -1, best_len = 0;
        for (int n = 0; n < T; ++n) {
            int len = root_path(par, n, path);
            int valid = 1;
            for (int j = 0; j < len; ++j)
                if (!node_matches(tok, par, prd, rp, path[j]))
                    valid = 0;
            if (valid && len > best_len) {
                best_len = len;
                best_node = n;
            }
        }
        write_result(par, prd, rp, best_node, best_len, max_path, accept_len + b,
                     accept_path + (size_t)b * max_path, next_token + b, status + b);
    }
    free(path);
    return HT_ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Greedy acceptance, scan form: one pass in flattened order,
 *   ok[c] = matches(c) and (parent[c] < 0 or ok[parent[c]]),  depth[c] = depth[parent] + 1,
 * then the first node of greatest depth among the ok ones.  Must agree with the
 * enumeration above.
 * ---------------------------------------------------------------------------------- */
int ht_oracle_accept_scan(const int32_t *tokens, const int32_t *parent, const int32_t *pred,
                          const int32_t *root_pred, int B, int N, int T, int max_path,
                          int32_t *accept_len, int32_t *accept_path, int32_t *next_token,
                          int32_t *status)
{
    int *ok = (int *)malloc(sizeof(int) * (size_t)(T > 0 ? T : 1));
    int *depth = (int *)malloc(sizeof(int) * (size_t)(T > 0 ? T : 1));
    if (!ok || !depth) {
        free(ok);
        free(depth);
        return HT_ORACLE_NOMEM;
    }
    for (int b = 0; b < B; ++b) {
        const int32_t *par = parent + (size_t)b * N;
        const int32_t *tok = tokens + (size_t)b * T;
        const int32_t *prd = pred + (size_t)b * N;
        const int32_t *rp = root_pred ? root_pred + b : NULL;
        status[b] = HT_ORACLE_OK;
        if (!tree_is_legal(par, N)) {
            status[b] = HT_ORACLE_BAD_TREE;
            accept_len[b] = 0;
            next_token[b] = -1;
            for (int j = 0; j < max_path; ++j)
                accept_path[(size_t)b * max_path + j] = -1;
            continue;
        }
        int best_node = -1, best_len = 0;
        for (int c = 0; c < T; ++c) {
            int p = par[c];
            int m = node_matches(tok, par, prd, rp, c);
            ok[c] = m && (p < 0 || ok[p]);
            depth[c] = (p < 0) ? 1 : depth[p] + 1;
            if (ok[c] && depth[c] > best_len) {
                best_len = depth[c];
                best_node = c;
            }
        }
        write_result(par, prd, rp, best_node, best_len, max_path, accept_len + b,
                     accept_path + (size_t)b * max_path, next_token + b, status + b);
    }
    free(ok);
    free(depth);
    return HT_ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * KV compaction: for every layer, sequence, kv head and j < accept_len[b], cache row
 * kv_len[b] + j becomes what row kv_len[b] + accept_path[b][j] held BEFORE the call
 * (K and V alike); new_kv_len[b] = kv_len[b] + accept_len[b].  Done from a snapshot of
 * the old rows so that overlapping source and destination rows cannot interfere.
 * The caches are raw bytes: [layers, B, Hkv, cap, D] elements of elem_bytes each.
 * Rows below kv_len[b] are never written; rows at or beyond new_kv_len[b] are left as
 * they were here (their content is unspecified by the method).
 * ---------------------------------------------------------------------------------- */
int ht_oracle_kv_compact(unsigned char *k_cache, unsigned char *v_cache,
                         int layers, int B, int Hkv, int cap, int D, int elem_bytes, int N,
                         const int32_t *kv_len, const int32_t *accept_len,
                         const int32_t *accept_path, int max_path,
                         int32_t *new_kv_len, int32_t *status)
{
    const size_t row_bytes = (size_t)D * elem_bytes;
    for (int b = 0; b < B; ++b) {
        const int L = kv_len[b];
        const int a = accept_len[b];
        const int32_t *path = accept_path + (size_t)b * max_path;
        status[b] = HT_ORACLE_OK;
        new_kv_len[b] = L;
        if (L < 0 || (long)L + N > cap) {
            status[b] = HT_ORACLE_BAD_LEN;
            continue;
        }
        if (a < 0 || a > max_path || a > N) {
            status[b] = HT_ORACLE_BAD_PATH;
            continue;
        }
        int good = 1;
        for (int j = 0; j < a; ++j) {
            if (path[j] < j || path[j] >= N)
                good = 0;
            if (j > 0 && path[j] <= path[j - 1])
                good = 0;
        }
        if (!good) {
            status[b] = HT_ORACLE_BAD_PATH;
            continue;
        }
        new_kv_len[b] = L + a;
        if (a == 0)
            continue;
        unsigned char *snap = (unsigned char *)malloc(row_bytes * (size_t)a);
        if (!snap)
            return HT_ORACLE_NOMEM;
        for (int t = 0; t < 2; ++t) {
            unsigned char *cache = t ? v_cache : k_cache;
            for (int l = 0; l < layers; ++l)
                for (int h = 0; h < Hkv; ++h) {
                    unsigned char *base =
                        cache + ((((size_t)l * B + b) * Hkv + h) * (size_t)cap) * row_bytes;
                    for (int j = 0; j < a; ++j)
                        memcpy(snap + row_bytes * j, base + row_bytes * (size_t)(L + path[j]),
                               row_bytes);
                    for (int j = 0; j < a; ++j)
                        memcpy(base + row_bytes * (size_t)(L + j), snap + row_bytes * j, row_bytes);
                }
        }
        free(snap);
    }
    return HT_ORACLE_OK;
}

int ht_oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
