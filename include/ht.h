/*
 * ht.h -- C ABI of the B200 tree-verify library for Hidden Transfer decoding
 * (arXiv 2404.12022).  One decoding round verifies a flattened draft tree and the
 * pseudo positions produced by the hidden-transfer projection in a single forward; this
 * library holds the data-parallel operations of that forward that are specific to the
 * method (projection, tree attention, verification, compaction) and the steps around them
 * (rotary embedding + cache append, draft tree, a paged cache).  Everything else of the
 * transformer layer (norms, Q/K/V/O and MLP GEMMs, lm-head) is the caller's.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless a comment says "host".  The caller owns every
 *     buffer, workspace included; the library allocates no device memory.  What it keeps
 *     between calls is per-device set-up only (kernel attributes, SM count, how many of a
 *     kernel's blocks the device holds, the address of the built-in scratch array of
 *     ht_tree_attention_static); a cudaDeviceReset makes that stale.
 *   - Work is enqueued on the caller's stream (`stream` is a cudaStream_t passed as
 *     void*; NULL = the default stream) and the call returns without synchronising.
 *   - The return value is a host-checkable status (HT_OK or HT_ERR_*).  When it is not
 *     HT_OK nothing was launched and ht_last_error_string() describes why.
 *   - Errors only the device can see (an illegal parent array, a cache length that does
 *     not fit, a malformed accepted path) are written to `status` -- one int32 per
 *     sequence, HT_STATUS_* -- and that sequence's work is skipped.  Device code never
 *     traps or asserts.  Every call that takes `status` writes all B entries.
 *   - Tensors are dense row-major with the last index fastest; every base pointer must
 *     be 16-byte aligned.
 *
 * Shapes: B sequences; N query rows per sequence = T draft-tree nodes followed by P
 * pseudo positions; Hq query heads sharing Hkv KV heads (Hq % Hkv == 0); head size D;
 * `cap` rows of cache capacity per (sequence, KV head); vocabulary V; hidden size d;
 * k transfer steps.
 */
#ifndef HT_H_
#define HT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { HT_F32 = 0, HT_F16 = 1, HT_BF16 = 2 } ht_dtype;

enum {
    HT_OK = 0,
    HT_ERR_INVALID_ARG = 1, /* null / misaligned pointer, non-positive or inconsistent size */
    HT_ERR_UNSUPPORTED = 2, /* a legal request this build has no kernel for */
    HT_ERR_BAD_TREE = 3,    /* reserved for host-side tree checks */
    HT_ERR_WORKSPACE = 4,   /* workspace smaller than ht_tree_attention_workspace() */
    HT_ERR_CUDA = 5,        /* the CUDA runtime reported an error at launch */
    HT_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out (reported via status) */
};

enum {
    HT_STATUS_OK = 0,
    HT_STATUS_BAD_TREE = 1,      /* some parent[r] is outside [-1, r) */
    HT_STATUS_BAD_LEN = 2,       /* kv_len[b] < 0 or kv_len[b] + N > cap */
    HT_STATUS_BAD_PATH = 3,      /* accepted path not increasing / out of range */
    HT_STATUS_PATH_TOO_LONG = 4, /* the accepted path has more than max_path nodes */
    HT_STATUS_BAD_PAGE = 5,      /* paged cache: a block-table entry the sequence needs is outside the pool */
    HT_STATUS_TIMEOUT = 6
};

/* ht_attn_desc.flags */
#define HT_ATTN_FORCE_SIMT 1u /* use the fp32-ALU kernel even where a tensor-core kernel applies */
/* The caller vouches that the first 64 KiB of the workspace are as a cudaMemset to zero, or any earlier
 * ht_tree_attention / ht_tree_attention_paged call on this workspace that reported no HT_STATUS_TIMEOUT, left
 * them: the call then leaves out the small kernel that clears the arrival counters kept there (every call
 * leaves the counters it used at zero).  Worth about a microsecond per call in a chain of calls; with the flag
 * set on a workspace that is not in that state, results of sequences whose work was split are undefined
 * (nothing faults, nothing waits). */
#define HT_ATTN_WORKSPACE_CLEAN 2u
/* The caller vouches that kv_len, parent, the cache rows below kv_len[b] of every sequence (and, for a paged
 * cache, the block-table entries of those rows) were final before the two kernels ahead of this call in `stream`
 * began.  (In a decoding step they are: the lengths change at the compaction, the rows below them are earlier
 * steps', and the tree is drafted before the first layer.)  The tensor-core kernels then make their plan and
 * fetch their first context tiles while the kernel ahead is still finishing, and wait for it only before they
 * read q or rows at or beyond kv_len[b] and before they write anything: about 3 us per call in a chain of calls.
 * A broken promise gives wrong results for the call, never a fault or a wait.  The fp32-ALU kernel ignores the
 * flag. */
#define HT_ATTN_CONTEXT_FINAL 4u
/* Test hook, never to be set in production: the tensor-core kernels' device-side waits give up after about a
 * microsecond instead of a second, so that their give-up path can be exercised: the call returns, the sequences'
 * status words read HT_STATUS_TIMEOUT and `out` is meaningless.  Nothing faults and nothing is left in flight:
 * a thread block that has given up still waits, with the full limit, for its own copies and tensor-core
 * operations before it frees what they write to. */
#define HT_ATTN_TEST_SHORT_WAITS 0x80000000u

typedef struct {
    int32_t B, N, Hq, Hkv, D, cap;
    int32_t dtype;        /* ht_dtype of q, caches and out */
    float scale;          /* softmax scale; <= 0 selects 1/sqrt(D) */
    int64_t kv_stride_b;  /* elements between sequences in each cache; 0 = Hkv*cap*D */
    int64_t kv_stride_h;  /* elements between KV heads; 0 = cap*D.  Rows are D apart. */
    int32_t num_splits;   /* KV splits per (sequence, head); 0 = library chooses */
    uint32_t flags;
} ht_attn_desc;

typedef struct {
    int32_t layers, B, Hkv, cap, D;
    int32_t dtype;        /* ht_dtype (only its width matters) */
    int32_t N;            /* tree rows behind each context: accepted indices lie in [0, N) */
    int64_t stride_layer; /* elements; 0 = B*Hkv*cap*D */
    int64_t stride_b;     /* elements; 0 = Hkv*cap*D */
    int64_t stride_h;     /* elements; 0 = cap*D */
} ht_cache_desc;

/* Knobs read once per process from the environment, for cross-checks and bug reports (results never need them):
 *   HT_LOG=1                        every entry point prints its arguments and the kernel it chose to stderr
 *   HT_FORCE_PATH=simt|mma|tcgen05  attention on the fp32-ALU kernel (simt); ht_transfer of 16-bit inputs on the
 *                                   warp-level kernel (mma) or, where the shape allows, on the tcgen05 kernel
 *   HT_SPLITS=n                     attention with n KV splits where the descriptor leaves the choice
 *                                   (num_splits == 0): the split-KV ALU kernel, as an explicit num_splits selects it
 * ht_tree_attention_workspace() and ht_tree_attention_launches() answer for the kernel the knobs select. */

/* Library version (major*10000 + minor*100 + patch). */
int ht_version(void);

/* Host string describing the most recent non-HT_OK return on the calling thread. */
const char *ht_last_error_string(void);

/*
 * Hidden-transfer projection -- Section "Hidden Transfer" and the displayed equation of
 * Section "Training stage":  h~ = W^i_{t_i} . h  with W^i in R^{d x d}, 1 <= i <= k, a
 * plain linear map (no bias, no activation).
 *   h_src [B, d]      hidden state of the source token of each sequence
 *   W     [k, d, d]   W[i][r][c]: output feature r, input feature c (W acts on a column)
 *   out   [B, k, d]   out[b][i][r] = sum_c W[i][r][c] * h_src[b][c]
 * fp32 accumulation, result rounded once to `dtype`.  d must be a multiple of 4 (fp32)
 * or 8 (fp16 / bf16).  B*k*d == 0 is a no-op.
 * B is the number of source rows, whatever they are: one per sequence (pseudo states
 * hanging off one node), or one per tree node of every sequence (the reading in which
 * every token gets its pseudo states), B x T rows, for which the 16-bit types run as a
 * matrix product on the tensor cores in one pass over W.  That kernel's waits are bounded
 * (about a second); should one run out, the outputs of the affected tile are NaN -- the call
 * has no status argument, so a NaN tile is the only signal (NaN inputs give NaN too).
 * All pointers are device pointers, 16-byte aligned; nothing is retained after the call.
 */
int ht_transfer(const void *h_src, const void *W, void *out, int B, int k, int d, int dtype,
                void *stream);

/*
 * Tree attention -- Section "Tree attention": the draft tree is flattened into a
 * sequence and "a token only attends to its ancestors" (and the context); pseudo
 * positions follow Section "Training stage" (a pseudo state sees the context, earlier
 * pseudo states and itself) and are given as ordinary rows of `parent`.
 *   q        [B, N, Hq, D]
 *   k_cache, v_cache  [B, Hkv, cap, D] (strides in desc); sequence b holds kv_len[b]
 *            context rows; the K/V of query row r must already sit at row kv_len[b] + r
 *   kv_len   [B] int32
 *   parent   [B, N] int32, parent[b][r] in [-1, r); -1 attaches r to the context
 *   out      [B, N, Hq, D]:  out[b,r,h] = softmax(scale * q[b,r,h] . K^T) V over cache rows
 *            [0, kv_len[b]) of KV head h / (Hq/Hkv) and rows kv_len[b] + c for c = r and
 *            every ancestor c of r.  fp32 (fp16 / bf16 inputs: tensor-core products with
 *            fp32 accumulation) softmax and accumulation, rounded once to `dtype`.
 *   workspace, workspace_bytes  scratch of at least ht_tree_attention_workspace(desc)
 *            bytes, 16-byte aligned; contents need no initialisation (but see
 *            HT_ATTN_WORKSPACE_CLEAN) and, beyond the first 64 KiB, are undefined afterwards.
 *            Calls that run concurrently need distinct workspaces.
 *   status   [B] int32 out: HT_STATUS_BAD_TREE / HT_STATUS_BAD_LEN sequences are skipped
 *            (their rows of `out` are left untouched).
 * Cache rows at or beyond kv_len[b] + N are never used for a result, whatever they hold.
 * Supported: D in {64, 128}; N <= 1024.  B == 0 or N == 0 is a no-op.
 * Stream behaviour (fp16 / bf16, D = 128): the call's kernels are launched with programmatic
 * stream serialization, i.e. their thread blocks may be set up while the kernel before them in
 * `stream` is still finishing; they read inputs, workspace and outputs only after that kernel
 * has completed, so the results are those of plain stream order.
 */
size_t ht_tree_attention_workspace(const ht_attn_desc *desc /* host */);
/* Number of this library's kernels that one ht_tree_attention call with this descriptor enqueues (1 or 2:
 * a kernel that zeroes arrival counters -- left out under HT_ATTN_WORKSPACE_CLEAN -- or one that merges split
 * partials, may accompany the attention kernel); 0 for a descriptor the call would reject or that has nothing
 * to do. */
int ht_tree_attention_launches(const ht_attn_desc *desc /* host */);
int ht_tree_attention(const ht_attn_desc *desc /* host */, const void *q, const void *k_cache,
                      const void *v_cache, const int32_t *kv_len, const int32_t *parent, void *out,
                      void *workspace, size_t workspace_bytes, int32_t *status, void *stream);

/*
 * Tree attention over a paged cache: the same operation as ht_tree_attention (Section "Tree
 * attention"), with the K / V rows of a sequence scattered over fixed-size pages of a shared pool,
 * the layout serving systems keep their caches in.
 *   pages->page_size   rows per page: a power of two >= 16
 *   pages->max_pages   block-table entries per sequence; the capacity of a sequence is
 *                      max_pages * page_size rows (desc->cap and desc's cache strides are ignored)
 *   pages->n_pages     pages in the pool
 *   pages->page_stride, head_stride   elements between pages / between the KV heads of a page;
 *                      0 = Hkv * page_size * D / page_size * D.  Rows are D apart.
 *   k_pages, v_pages   [n_pages, Hkv, page_size, D]
 *   block_table        [B, max_pages] int32: cache row r of sequence b is row r % page_size of page
 *                      block_table[b][r / page_size].  As in ht_tree_attention the K / V of query
 *                      row r must already sit at cache row kv_len[b] + r.  Entries of pages wholly
 *                      past row kv_len[b] + N are not consulted for a result and may hold anything.
 *   status             as in ht_tree_attention, plus HT_STATUS_BAD_PAGE for a sequence one of whose
 *                      needed entries lies outside [0, n_pages): page 0 is read in its place (no
 *                      access outside the pool) and the sequence's rows of `out` are meaningless.
 * q, kv_len, parent, out, workspace (ht_tree_attention_workspace(desc) bytes) as in
 * ht_tree_attention.  Supported: fp16 / bf16, D = 128, Hq / Hkv a power of two, N <= 1024,
 * B <= 256 (the tensor-core kernels); anything else returns HT_ERR_UNSUPPORTED.
 */
typedef struct {
    int32_t page_size, max_pages, n_pages;
    int64_t page_stride, head_stride;
} ht_paged_desc;
int ht_tree_attention_paged(const ht_attn_desc *desc /* host */, const ht_paged_desc *pages /* host */,
                            const void *q, const void *k_pages, const void *v_pages,
                            const int32_t *block_table, const int32_t *kv_len, const int32_t *parent,
                            void *out, void *workspace, size_t workspace_bytes, int32_t *status,
                            void *stream);

/*
 * The two row-moving steps on a paged cache (same pools, block table and descriptor as
 * ht_tree_attention_paged; one block table serves all layers):
 *   ht_rope_kv_append_paged  as ht_rope_kv_append, the rows of sequence b landing at logical cache rows
 *       kv_len[b] + r through the block table.  A row whose page entry lies outside the pool is
 *       not stored (its q row is still rotated) and marks the sequence HT_STATUS_BAD_PAGE.
 *   ht_kv_compact_paged      as ht_kv_compact on pools [layers, n_pages, Hkv, page_size, D];
 *       desc->cap, stride_b and stride_h are ignored (the capacity is max_pages * page_size, the strides
 *       are those of `pages`), desc->stride_layer is the distance between the layers' pools in
 *       elements (0 = n_pages * page_stride).  Rows move between pages as the table says; a
 *       needed entry outside the pool leaves the sequence unchanged with HT_STATUS_BAD_PAGE.
 */
int ht_rope_kv_append_paged(const ht_attn_desc *desc /* host */, const ht_paged_desc *pages /* host */,
                            const void *q_in, const void *k_in, const void *v_in, const int32_t *pos,
                            const int32_t *kv_len, const int32_t *block_table, float rope_base,
                            void *q_out, void *k_pages, void *v_pages, int32_t *status, void *stream);
int ht_kv_compact_paged(void *k_pages, void *v_pages, const ht_cache_desc *desc /* host */,
                        const ht_paged_desc *pages /* host */, const int32_t *block_table,
                        const int32_t *kv_len, const int32_t *accept_len, const int32_t *accept_path,
                        int max_path, int32_t *new_kv_len, int32_t *status, void *stream);

/*
 * Greedy verification -- Fig. 2 caption ("find the last accepted token position"),
 * Section "Inference stage", Section "Setup" (greedy sampling; output identical to
 * auto-regressive decoding).
 *   logits    [B, N, V] of `dtype`
 *   tokens    [B, T] int32 draft token of each tree node (T <= N)
 *   parent    [B, N] int32 (rows < T are consulted)
 *   root_pred [B] int32 or NULL: the token greedy decoding emits after the context (the
 *             argmax carried over from the previous round).  Top-level nodes (parent -1)
 *             are checked against it; with NULL they are taken as known-correct.
 *   pred      [B, N] int32 out, required: argmax_v logits[b,r,v]; the lowest index wins
 *             ties, NaN never wins, a row of NaNs gives 0
 *   accept_len  [B] out: number of nodes on the longest root path all of whose nodes c
 *             satisfy tokens[c] == pred[parent[c]] (top level: == root_pred); ties between
 *             paths of equal length go to the smallest terminal node index
 *   accept_path [B, max_path] out: that path, root first, padded with -1
 *   next_token  [B] out: pred at the path's last node; root_pred[b] (or -1 without
 *             root_pred) when nothing is accepted
 *   status    [B] out: HT_STATUS_BAD_TREE, HT_STATUS_PATH_TOO_LONG (accept_len 0, next -1)
 * max_path <= 255.
 * accept_len is also where the kernel counts, in the bits above the low eight, the rows of a sequence that are
 * done; the sequence's last thread block replaces the count by the length.  ON ENTRY every accept_len[b] must
 * therefore hold a value in [0, 255]: zero before the first call (the caller clears it once), afterwards what
 * the previous call left there will do.  Anything else (uninitialised memory, a buffer last used by a call that
 * did not finish) makes the count come out wrong and the sequence's outputs are not written.
 * One kernel, launched with programmatic stream serialization and waiting, at its first instruction, for the
 * work ahead of it in the stream: ordering is that of an ordinary launch.
 */
int ht_verify_greedy(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                     const int32_t *root_pred, int B, int N, int T, int V, int max_path,
                     int32_t *pred, int32_t *accept_len, int32_t *accept_path,
                     int32_t *next_token, int32_t *status, void *stream);

/*
 * Greedy verification and KV compaction in one launch -- Fig. 2 caption and Section "Inference stage" (find the
 * last accepted position, then go on from it): ht_verify_greedy followed by ht_kv_compact, with the same
 * arguments, results and restrictions as the two calls (max_path <= 64; new_kv_len must not overlap kv_len or
 * accept_len; accept_len[b] in [0, 255] on entry), and the same results bit for bit.
 *   rows     logits rows per sequence whose argmax is taken, T <= rows <= N; 0 selects T, the rows
 *            acceptance can consult.  pred[b][r] is written for r < rows only.
 *   status, compact_status   [B] out: the status words of the verification and of the compaction.
 *   desc     its B and N must equal B and N.
 * The thread blocks first take the argmax of the rows; the block that completes a sequence searches its
 * tree; then all blocks share out the compaction's (layer, sequence, head group) items, each waiting (bounded:
 * about a second, then HT_STATUS_TIMEOUT in compact_status and the sequence's cache left as it is) until the
 * sequence's accepted length has been stored.  The grid never exceeds what the GPU holds at once.
 */
int ht_verify_greedy_compact(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                             const int32_t *root_pred, int B, int N, int T, int V, int max_path, int rows,
                             int32_t *pred, int32_t *accept_len, int32_t *accept_path, int32_t *next_token,
                             int32_t *status, void *k_cache, void *v_cache, const ht_cache_desc *desc /* host */,
                             const int32_t *kv_len, int32_t *new_kv_len, int32_t *compact_status, void *stream);

/*
 * KV compaction -- implied by verifying under a KV cache (Fig. 1 caption; Section
 * "Inference stage"): after acceptance only the accepted path's K/V may follow the
 * context.  For every layer, sequence b, KV head and j < accept_len[b], cache row
 * kv_len[b] + j receives what row kv_len[b] + accept_path[b][j] held before the call (K and
 * V alike); new_kv_len[b] = kv_len[b] + accept_len[b].  In place and safe when source and
 * destination rows overlap.  Rows below kv_len[b] are untouched; rows at or beyond
 * new_kv_len[b] are unspecified afterwards.
 *   k_cache, v_cache  [layers, B, Hkv, cap, D] (strides in desc)
 *   accept_path [B, max_path], strictly increasing, accept_path[b][j] in [j, N)
 *   status [B] out: HT_STATUS_BAD_LEN / HT_STATUS_BAD_PATH sequences are left unchanged and
 *            new_kv_len[b] = kv_len[b].
 * max_path <= 64.  D * element size must be a multiple of 16 bytes.
 * new_kv_len must not overlap kv_len or accept_len (HT_ERR_INVALID_ARG): the sequence's thread blocks
 * read both throughout the kernel, so an update in place would be seen by some of them and not by
 * others.  Keep two length arrays and swap them between rounds.
 * The kernel is launched with programmatic stream serialization and waits, at its first instruction, for
 * the work ahead of it in the stream: ordering is that of an ordinary launch.
 */
int ht_kv_compact(void *k_cache, void *v_cache, const ht_cache_desc *desc /* host */,
                  const int32_t *kv_len, const int32_t *accept_len, const int32_t *accept_path,
                  int max_path, int32_t *new_kv_len, int32_t *status, void *stream);

/*
 * Draft tree for the next round -- Section "Inference stage" (the candidate sequences are made
 * "into a tree structure by merging their common ancestors" and the tree is flattened) and Section
 * "Tree attention" ("a pre-defined tree structure and parser"; tokens keep their positional indices).
 * The candidates are the most likely tokens of the pseudo positions' distributions (Section "Hidden
 * Transfer": the lm-head decodes the pseudo hidden states).  The pre-defined structure is a template
 * shared by all sequences: node n at level i takes the tmpl_rank[n]-th most likely token (0 = the
 * most likely) of pseudo position i, so merging common ancestors costs nothing at run time.
 *   logits      [B, rows, V] of `dtype`; pseudo position i (1..P) of sequence b is row first_row + i - 1
 *   tmpl_parent [T] int32, tmpl_parent[n] in [-1, n)
 *   tmpl_rank   [T] int32, in [0, K) for nodes of level >= 1
 *   root_token  [B] int32 or NULL.  Given: nodes with parent -1 are the known next token (level 0,
 *               e.g. next_token of ht_verify_greedy) and their children are level 1.  NULL: nodes
 *               with parent -1 are level 1 themselves (a forest of first drafts).
 *   base_pos    [B] int32: position id of the top-level nodes (e.g. new_kv_len of ht_kv_compact)
 *   topk        [B, P, K] out: the K most likely tokens per pseudo position -- larger value first,
 *               lower index first among equal values, NaN below everything
 *   tokens      [B, T] out: draft token of every template node
 *   pos         [B, T] out: base_pos[b] + depth of the node (top-level nodes: depth 0)
 *   status      [B] out: HT_STATUS_BAD_TREE when the template is malformed (a parent that is not an
 *               earlier node, a level beyond P, a rank outside [0, K)); tokens and pos are then -1.
 * 1 <= K <= 16, K <= V, T >= 1.  B == 0 is a no-op.  The parent array of the next round's
 * ht_tree_attention is tmpl_parent followed by the pseudo rows.
 */
int ht_draft_tree(const void *logits, int dtype, int B, int rows, int V, int first_row, int P, int K,
                  const int32_t *tmpl_parent, const int32_t *tmpl_rank, int T, const int32_t *root_token,
                  const int32_t *base_pos, int32_t *topk, int32_t *tokens, int32_t *pos, int32_t *status,
                  void *stream);

/*
 * Rotary position embedding at the tree's position ids, and placement of the rows' K / V behind
 * the context -- the step ahead of ht_tree_attention.  Section "Tree attention": the flattened tree
 * preserves "the original positional indices of each token"; Section "Training stage": a pseudo state
 * of step i has position id j + i; Section "Setup": LLaMA-2 / Vicuna models, i.e. the rotary embedding
 * in the half-split pairing (feature i with feature i + D/2, angle pos * rope_base^(-2i/D)).
 *   desc     B, N, Hq, Hkv, D, cap, dtype and the cache strides are used (scale, num_splits, flags are not)
 *   q_in     [B, N, Hq, D], k_in, v_in [B, N, Hkv, D]: the rows' projections before the rotation
 *   pos      [B, N] int32 position ids (e.g. ht_draft_tree's `pos`, followed by the pseudo rows')
 *   kv_len   [B] int32
 *   q_out    [B, N, Hq, D]: q_in rotated (may alias q_in)
 *   k_cache, v_cache [B, Hkv, cap, D]: row kv_len[b] + r receives k_in[b, r] rotated / v_in[b, r] as is
 *   status   [B] out: HT_STATUS_BAD_LEN sequences are skipped (nothing of theirs is written)
 * Angles are formed in fp64, products in fp32, one rounding to `dtype`.  D in {64, 128}.
 */
int ht_rope_kv_append(const ht_attn_desc *desc /* host */, const void *q_in, const void *k_in, const void *v_in,
                      const int32_t *pos, const int32_t *kv_len, float rope_base, void *q_out, void *k_cache,
                      void *v_cache, int32_t *status, void *stream);

/*
 * Tree attention without a caller-provided workspace.  (The paper has no counterpart: this
 * entry point exists for integration, not for the method.)
 *
 * Same operation, arguments and results as ht_tree_attention, computed by the split-KV
 * fp32-ALU kernel, for callers that cannot give the library scratch memory because they
 * cannot allocate any: code running where cudaMalloc must not be called, plugin
 * interfaces that pass only inputs and outputs, processes whose device memory is fully
 * committed.  The split partials live in a fixed array of HT_STATIC_SCRATCH_BYTES inside
 * the library image; every GPU context that loads the library holds that array until it
 * exits, used or not.  The call allocates and frees nothing.
 *   - A problem whose partials exceed the array is refused with HT_ERR_WORKSPACE and a
 *     message giving both sizes; desc->num_splits = 1 never needs scratch.
 *   - The first call on each device looks up the array's device address (with the caller's
 *     current device, which must be the one the pointers and the stream belong to; a q on
 *     another device is refused with HT_ERR_INVALID_ARG).  Make that first call outside any
 *     stream capture.  The address is kept for the life of the process: after
 *     cudaDeviceReset the library's per-device state is stale and the process must reload it.
 *   - All calls share the array and it keeps the previous call's contents.  Nothing in it
 *     needs clearing, but calls that overlap on the GPU (two streams, two host threads)
 *     race on it: serialise them.
 */
#define HT_STATIC_SCRATCH_BYTES (16u << 20)
int ht_tree_attention_static(const ht_attn_desc *desc /* host */, const void *q, const void *k_cache,
                             const void *v_cache, const int32_t *kv_len, const int32_t *parent,
                             void *out, int32_t *status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* HT_H_ */
