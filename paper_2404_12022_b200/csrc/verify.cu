// Greedy verification (Fig. 2 caption; Sections "Inference stage" and "Setup"):
// row argmax of the logits, then the longest root path of the draft tree whose tokens
// are the ones greedy decoding would emit -- and, in the fused form, the compaction of the
// accepted path's K/V rows (Fig. 1 caption) in the same launch.
//
// One launch, a grid no larger than the GPU holds at once.  A block streams logits rows
// (asynchronous 16-byte copies into shared memory, 64 KB of a row in flight at once whatever the
// compiler makes of the registers; every thread reads back what it copied, shuffle reductions)
// and stores each row's argmax; the block that finishes a sequence's last row runs the path search for that
// sequence -- a few hundred integer operations.  Arrivals are counted in the upper bits of the
// sequence's accept_len word: the caller hands it over holding a small value (zero, or the
// length an earlier call left there), the last block overwrites it with the new length, so
// that no kernel has to clear anything ahead of the launch.  In the fused form the blocks then
// share out the (layer, sequence, head group) items of the compaction; a block waits (bounded)
// for the sequence's length to appear before it moves that sequence's rows.
#include <limits.h>

#include "compact.cuh"

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

__device__ __forceinline__ void st_release(int32_t *p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int32_t *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// The tree of one sequence in shared memory: parents and draft tokens are inputs (staged while the logits stream, by
// every block, for the sequence of the row it works on), the rows' argmax is what the other blocks of the launch wrote
// (staged by the block that searches, once all rows have arrived).
constexpr int kStage = 1024;                 // trees of up to this many rows are staged
struct TreeSmem {
    int32_t par[kStage], tok[kStage], prd[kStage];
    int bad, root, staged_b;
    unsigned long long key[32];
};

__device__ __forceinline__ void stage_tree(TreeSmem &ts, int b, const int32_t *__restrict__ tokens, const int32_t *__restrict__ parent,
                                           const int32_t *__restrict__ root_pred, int N, int T) {
    if (ts.staged_b == b) return;                      // (uniform over the block: written behind a barrier below)
    __syncthreads();
    if (threadIdx.x == 0) {
        ts.bad = 0;
        ts.root = root_pred ? root_pred[b] : -1;
        ts.staged_b = b;
    }
    __syncthreads();
    const int32_t *par = parent + (size_t)b * N;
    for (int c = threadIdx.x; c < N; c += blockDim.x) {
        const int pc = par[c];
        if (N <= kStage) {
            ts.par[c] = pc;
            if (c < T) ts.tok[c] = tokens[(size_t)b * T + c];
        }
        if (pc < -1 || pc >= c) ts.bad = 1;
    }
}

// Path search of one sequence by one block (its tree staged by stage_tree).  Every thread walks the root path of its
// nodes (parent[c] < c makes the walk finite), checks the match rule on the way and proposes (depth, node);
// the block keeps the deepest valid node, lowest index on ties.
__device__ __forceinline__ void accept_sequence(TreeSmem &ts, const int b, const int32_t *__restrict__ tokens, const int32_t *__restrict__ parent,
              const int32_t *__restrict__ root_pred, const int32_t *pred, int N, int T,
              int max_path, int32_t *accept_len, int32_t *__restrict__ accept_path,
              int32_t *__restrict__ next_token, int32_t *__restrict__ status, const int done_mark) {
    const int32_t *par = parent + (size_t)b * N;
    const int32_t *tok = tokens + (size_t)b * T;
    const int32_t *prd = pred + (size_t)b * N;
    int32_t *path = accept_path + (size_t)b * max_path;
    // The walks below are chains of dependent reads: with the tree's three arrays in shared memory they
    // cost one round trip to L2 in all instead of one per level (trees of up to kStage rows).
    if (N <= kStage) {
        for (int c = threadIdx.x; c < N; c += blockDim.x) ts.prd[c] = __ldcg(prd + c);
        par = ts.par; tok = ts.tok; prd = ts.prd;
    }
    for (int j = threadIdx.x; j < max_path; j += blockDim.x) path[j] = -1;
    __syncthreads();
    // the word other blocks wait on (fused form) is stored with release semantics, behind everything else
    auto finish = [&](int word) {
        if (done_mark) st_release(accept_len + b, done_mark | word);
        else accept_len[b] = word;
    };
    if (ts.bad) {
        if (threadIdx.x == 0) {
            status[b] = HT_STATUS_BAD_TREE;
            next_token[b] = -1;
            finish(0);
        }
        return;
    }
    const bool has_root = root_pred != nullptr;
    const int rp = ts.root;
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
    if ((threadIdx.x & 31) == 0) ts.key[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) key = ts.key[w] > key ? ts.key[w] : key;
        const int len = (int)(key >> 32);
        const int node = (int)(0xFFFFFFFFu - (unsigned)(key & 0xFFFFFFFFu));
        if (len > max_path) {
            status[b] = HT_STATUS_PATH_TOO_LONG;
            next_token[b] = -1;
            finish(0);
        } else {
            status[b] = HT_STATUS_OK;
            if (len == 0) {
                next_token[b] = has_root ? rp : -1;
            } else {
                int j = len - 1;
                for (int c = node; c >= 0; c = par[c]) path[j--] = c;
                next_token[b] = ld_pred(prd + node);
            }
            finish(len);
        }
    }
}

// Two shapes of block, 128 KB of logits in flight per SM either way: 512 threads (64 KB of a row at once, two blocks
// per SM) while the rows are few, so that a row is there in one round trip; 256 threads (32 KB at once, four blocks
// per SM) when there are more rows than twice the SMs, so that all of them are under way at once.
constexpr int kVerifyInFlight = 8;           // 16-byte copies per thread in flight
constexpr int verify_smem(int threads) { return threads * kVerifyInFlight * 16; }
constexpr unsigned kTicket = 256u;           // arrivals are counted in units of this on the accept_len word: lengths stay below it
constexpr int kDoneMark = 1 << 30;           // fused form: the length is in the word's low bits, the compaction may begin

// Argmax of one logits row by the block: lowest index on ties, NaN never wins, a row of NaNs gives 0.  All threads
// return the same index.
// This thread's copies of one pass over a row (vectors j0, j0 + kVerifyThreads, ...) into its slots of the staging area.
template <typename T, int kVerifyThreads>
__device__ __forceinline__ void row_issue(const T *__restrict__ row, int nvec, int j0) {
    extern __shared__ uint4 s_stage[];                 // [kVerifyInFlight][kVerifyThreads]: a thread reads back its own copies only
#pragma unroll
    for (int u = 0; u < kVerifyInFlight; ++u) {
        const int j = j0 + u * kVerifyThreads;
        if (j < nvec)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_stage[u * kVerifyThreads + threadIdx.x])),
                         "l"(row + (size_t)j * Vec16<T>::n) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <typename T>
__device__ __forceinline__ bool row_vectorized(int V) { return ((size_t)V * sizeof(T)) % 16 == 0; }

// The caller has issued the row's first pass (row_issue with j0 = threadIdx.x) where the row is vectorized.
template <typename T, int kVerifyThreads>
__device__ __forceinline__ int row_argmax(const T *__restrict__ row, int V) {
    constexpr int VE = Vec16<T>::n;
    Best best{-INFINITY, INT_MAX};
    const bool vec_ok = row_vectorized<T>(V);
    if (vec_ok) {
        const int nvec = V / VE;
        constexpr int U = kVerifyInFlight;
        extern __shared__ uint4 s_stage[];
        for (int j0 = threadIdx.x; j0 < nvec; j0 += U * kVerifyThreads) {
            if (j0 != (int)threadIdx.x) row_issue<T, kVerifyThreads>(row, nvec, j0);
            asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int j = j0 + u * kVerifyThreads;
                if (j < nvec) {
                    float f[VE];
                    unpack16<T>(s_stage[u * kVerifyThreads + threadIdx.x], f);
#pragma unroll
                    for (int e = 0; e < VE; ++e) {
                        // A thread meets its elements in increasing index order, so "larger value, lower index
                        // on ties" is "strictly larger than the best so far".  NaN compares false and is
                        // skipped; so is -inf, which a row without anything larger settles below.
                        if (f[e] > best.v) best = Best{f[e], j * VE + e};
                    }
                }
            }
        }
    } else {
        for (int j = threadIdx.x; j < V; j += kVerifyThreads) {
            const float x = to_float<T>(row[j]);
            if (x > best.v) best = Best{x, j};
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Best o{__shfl_xor_sync(0xffffffffu, best.v, off), __shfl_xor_sync(0xffffffffu, best.i, off)};
        best = better(best, o);
    }
    __shared__ Best warp_best[kVerifyThreads / 32];
    __shared__ int warp_first[kVerifyThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();                               // the previous row's readers of these arrays are done
    if (lane == 0) warp_best[warp] = best;
    __syncthreads();
    best = warp_best[0];
#pragma unroll
    for (int w = 1; w < kVerifyThreads / 32; ++w) best = better(best, warp_best[w]);
    if (best.i == INT_MAX) {
        // Nothing in the row exceeds -inf: the answer is the first -inf, or 0 in a row of NaNs only.
        int first = INT_MAX;
        for (int j = threadIdx.x; j < V; j += kVerifyThreads)
            if (to_float<T>(row[j]) == -INFINITY) { first = j; break; }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, off));
        if (lane == 0) warp_first[warp] = first;
        __syncthreads();
        first = warp_first[0];
        for (int w = 1; w < kVerifyThreads / 32; ++w) first = min(first, warp_first[w]);
        best.i = first == INT_MAX ? 0 : first;
    }
    return best.i;
}

struct VerifyArgs {
    const void *logits;
    const int32_t *tokens, *parent, *root_pred;
    int B, N, T, V, max_path;
    int rows;                 // logits rows per sequence whose argmax is taken: T <= rows <= N
    int32_t *pred, *accept_len, *accept_path, *next_token, *status;
};

// kFused: the blocks go on to the compaction once their rows are done.
template <typename T, bool kFused, int kVerifyThreads>
__global__ void __launch_bounds__(kVerifyThreads, 1024 / kVerifyThreads)
verify_kernel(const VerifyArgs v, const CompactArgs c) {
    // The launch is serialized programmatically behind the kernel ahead of it in the stream: from here on everything
    // that kernel wrote may be read.  A kernel serialized behind this one may set itself up meanwhile.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ int s_last;
    __shared__ TreeSmem ts;
    if (threadIdx.x == 0) ts.staged_b = -1;
    __syncthreads();
    const int n_rows = v.B * v.rows;
    for (int idx = blockIdx.x; idx < n_rows; idx += gridDim.x) {
        const int b = idx / v.rows, r = idx - b * v.rows;
        // the row's first 64 KB are asked for, then the sequence's tree (inputs) goes into shared memory while they stream
        const T *row = static_cast<const T *>(v.logits) + ((size_t)b * v.N + r) * v.V;
        if (row_vectorized<T>(v.V)) row_issue<T, kVerifyThreads>(row, v.V / Vec16<T>::n, threadIdx.x);
        stage_tree(ts, b, v.tokens, v.parent, v.root_pred, v.N, v.T);
        const int best = row_argmax<T, kVerifyThreads>(row, v.V);
        if (threadIdx.x == 0) {
            v.pred[(size_t)b * v.N + r] = best;
            // The block that stores a sequence's last argmax searches its tree: the count is added with release
            // semantics (the store above comes first) and read with acquire semantics (the other rows' stores are
            // visible behind it, to the whole block behind the barrier below).
            unsigned before;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(before) : "l"(v.accept_len + b), "r"(kTicket) : "memory");
            s_last = before / kTicket == (unsigned)(v.rows - 1);
        }
        __syncthreads();
        if (s_last)
            accept_sequence(ts, b, v.tokens, v.parent, v.root_pred, v.pred, v.N, v.T, v.max_path, v.accept_len, v.accept_path,
                            v.next_token, v.status, kFused ? kDoneMark : 0);
        __syncthreads();
    }
    if (!kFused) return;
    // ---- compaction: items (layer, sequence, head group) dealt out to the blocks.  The grid is no larger than the
    // GPU holds at once and every block has finished its rows before it waits here, so the length it waits for is
    // on its way; the wait is bounded all the same.  The sequence's word says "done | length" from the path search
    // on; finished items are counted in it as the rows were, and the last one leaves the plain length there. ----
    __shared__ CompactSmem csm;
    __shared__ int s_len_b;
    const int n_items = c.layers * c.B * c.groups;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        int x = item;
        const int grp = x % c.groups;
        x /= c.groups;
        const int b = x % c.B, layer = x / c.B;
        const int L = c.kv_len[b];                           // on its way while the length is waited for
        if (threadIdx.x == 0) {
            int a = ld_acquire(v.accept_len + b);
            const long long t0 = clock64();
            while (!(a & kDoneMark)) {                       // rows are still arriving, or have not begun to
                if (clock64() - t0 > 2000000000ll) { a = -1; break; }
                __nanosleep(64);
                a = ld_acquire(v.accept_len + b);
            }
            s_len_b = a < 0 ? -1 : (a & (int)(kTicket - 1));
        }
        __syncthreads();
        const int a = s_len_b;
        if (a < 0) {                                         // gave up: the sequence is left as it is
            if (layer == 0 && grp == 0 && threadIdx.x == 0) {
                c.status[b] = HT_STATUS_TIMEOUT;
                c.new_kv_len[b] = L;
            }
            __syncthreads();
            continue;
        }
        compact_item<2048 / kVerifyThreads, kVerifyThreads>(c, csm, layer, b, grp, a, L);
        if (threadIdx.x == 0) {
            const unsigned before = atomicAdd(reinterpret_cast<unsigned int *>(v.accept_len + b), kTicket);
            if ((before & ~(unsigned)kDoneMark) / kTicket == (unsigned)(c.layers * c.groups - 1)) v.accept_len[b] = a;
        }
    }
}

template <typename... KArgs, typename... Args>
static cudaError_t launch_chained(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Blocks of a verification kernel the GPU holds at once (and its shared memory limit raised, once).
template <typename Kernel>
static int resident_blocks(Kernel kernel, int threads) {
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, verify_smem(threads)) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, verify_smem(threads)) != cudaSuccess || sms <= 0 || per_sm <= 0) {
        cudaGetLastError();
        return 148;
    }
    return sms * per_sm;
}

template <typename T, bool kFused, int kThreads>
static cudaError_t launch_verify_shape(const VerifyArgs &v, const CompactArgs &c, cudaStream_t s, int *blocks_out) {
    static int caps[64];                              // per device
    int dev = 0;
    cudaGetDevice(&dev);
    int *slot = (dev >= 0 && dev < 64) ? &caps[dev] : nullptr;
    int cap = slot ? *slot : 0;
    if (cap == 0) {
        cap = resident_blocks(verify_kernel<T, kFused, kThreads>, kThreads);
        if (slot) *slot = cap;
    }
    if (blocks_out) {
        *blocks_out = cap;
        return cudaSuccess;
    }
    const long long want = (long long)v.B * v.rows;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    return launch_chained(verify_kernel<T, kFused, kThreads>, grid, (unsigned)kThreads, (size_t)verify_smem(kThreads), s, v, c);
}

template <typename T>
static cudaError_t launch_verify_t(const VerifyArgs &v, const CompactArgs *compact, cudaStream_t s) {
    int wide = 0;                                     // blocks of the 512-thread shape the GPU holds
    cudaError_t e = compact ? launch_verify_shape<T, true, 512>(v, *compact, s, &wide) : launch_verify_shape<T, false, 512>(v, CompactArgs{}, s, &wide);
    if (e != cudaSuccess) return e;
    const bool few = (long long)v.B * v.rows <= wide;
    if (compact) return few ? launch_verify_shape<T, true, 512>(v, *compact, s, nullptr) : launch_verify_shape<T, true, 256>(v, *compact, s, nullptr);
    return few ? launch_verify_shape<T, false, 512>(v, CompactArgs{}, s, nullptr) : launch_verify_shape<T, false, 256>(v, CompactArgs{}, s, nullptr);
}

int launch_verify(const void *logits, int dtype, const int32_t *tokens, const int32_t *parent,
                  const int32_t *root_pred, int B, int N, int T, int V, int max_path, int rows, int32_t *pred,
                  int32_t *accept_len, int32_t *accept_path, int32_t *next_token, int32_t *status,
                  const CompactArgs *compact, cudaStream_t s) {
    VerifyArgs v{};
    v.logits = logits; v.tokens = tokens; v.parent = parent; v.root_pred = root_pred;
    v.B = B; v.N = N; v.T = T; v.V = V; v.max_path = max_path; v.rows = rows;
    v.pred = pred; v.accept_len = accept_len; v.accept_path = accept_path; v.next_token = next_token; v.status = status;
    cudaError_t e;
    switch (dtype) {
        case HT_F32: e = launch_verify_t<float>(v, compact, s); break;
        case HT_F16: e = launch_verify_t<__half>(v, compact, s); break;
        default: e = launch_verify_t<__nv_bfloat16>(v, compact, s); break;
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "ht_verify_greedy: %s", cudaGetErrorString(e));
    }
    return HT_OK;
}

}  // namespace ht
