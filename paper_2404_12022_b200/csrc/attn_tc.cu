// Tree attention on the 5th-generation tensor cores (Section "Tree attention"; pseudo rows:
// Section "Training stage").  fp16 / bf16 inputs, head size 128.
//
// Why tensor cores here: all N query rows of the g = Hq/Hkv heads that share a KV head form
// one [N*g, 128] operand that meets every K/V row exactly once, so the cache prefix is a
// real dense contraction with N*g flop per K/V byte (about 90 in the 7B configs) -- far
// beyond what the fp32 ALUs sustain at HBM speed, and below the tensor ridge, i.e. the
// kernel is meant to be HBM-bound with the tensor pipe roughly half busy.
//
// Design (one persistent CTA per SM, 320 threads, warp-specialised):
//   warp 8, one thread : TMA producer.  Q tile [128 rows x 128] once per work segment and a
//                        ring of 32 KiB K / V tiles (128 keys x 128, 128-byte swizzle), each
//                        fetched by this CTA itself (no multicast).
//   warp 9, one thread : issues tcgen05.mma.  S = Q K^T (SS form) into one of two TMEM
//                        score buffers, O += P V (TS form: P is read from TMEM, V from
//                        shared memory in MN-major layout) into one of two TMEM output
//                        accumulators.  Order QK(j), PV(j-1), QK(j+1), ... so the tensor
//                        pipe computes the next scores while the softmax of the current
//                        tile runs.
//   warps 0-3, 4-7     : two softmax groups of 128 threads; thread i owns query row i
//                        (TMEM lane i), so row max and row sum need no shuffles.  Group s
//                        handles tiles j with j % 2 == s and keeps its own running max,
//                        sum and output accumulator; the two are merged by log-sum-exp at
//                        the end of a segment.  The running max is only raised when it
//                        would grow by more than 2^8 (the accumulator is then rescaled in
//                        TMEM), so the common case touches O not at all.
//   tree mask          : bit c of row r's ancestor word (built in shared memory from
//                        parent[] per segment) decides visibility of tree key c; only tiles
//                        that reach past the context length are masked.
//   work split         : all (sequence, KV head, row tile) units are laid end to end as
//                        a list of 128-key tiles; CTA i takes tiles [i*per, (i+1)*per).  A
//                        unit that is cut writes (m, l, O) partials to the workspace and
//                        takes a ticket; the CTA that delivers the last part of a unit
//                        merges all parts -- nobody waits on another CTA.
//
// Every wait on an mbarrier is bounded; when one runs out the CTA raises an abort flag,
// reports HT_STATUS_TIMEOUT, runs to the end of its control flow without further waiting,
// drains its own copies, frees its TMEM and returns.
#include <cuda.h>

#include "ht_common.cuh"

namespace ht {
namespace tc {

constexpr int kTile = 128;                 // keys per tile
constexpr int kRows = 128;                 // query rows per tile (UMMA M)
constexpr int kD = 128;
constexpr int kStages = 5;                 // ring entries (each one K or one V tile)
constexpr int kEntryBytes = kTile * kD * 2;
constexpr int kSlabBytes = kEntryBytes / 2;   // [128 rows][64 elements] = 16 KiB
constexpr int kThreads = 320;
constexpr int kMaxB = 256;
constexpr int kMaxWords = 16;              // ancestor words per row -> N <= 512
constexpr int kSlotFloats = kRows * kD + 2 * kRows;   // one partial result: O as [32 feature groups][128 rows][4], m[128], l[128]
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;  // log2 domain

struct Params {
    const int32_t *kv_len, *parent;
    int32_t *status;
    void *out;
    float *part;           // partial results of cut units: [grid][2][kSlotFloats]
    unsigned int *tickets; // one arrival counter per unit, zero on entry
    int B, N, Hq, Hkv, g, cap, n_rt, rows_per_tile_nodes;   // rows_per_tile_nodes = 128 / g
    float scale_log2;
    int is_bf16;
    int grid;
#ifdef HT_TC_TRACE
    long long *trace;
#endif
};

// Optional timeline of one CTA (clock64 stamps per role / tile / event) for tuning builds.
#ifdef HT_TC_TRACE
#define HT_TR(role, j, ev) do { if (p.trace && blockIdx.x == HT_TC_TRACE && (threadIdx.x & 31) == 0 && ((role) < 2 || (threadIdx.x & 127) == 0) && (j) < 40) p.trace[((role) * 40 + (j)) * 4 + (ev)] = clock64(); } while (0)
#define HT_TR_CTA(ev) do { if (p.trace && (threadIdx.x & 31) == 0) { unsigned long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); p.trace[1000 + blockIdx.x * 4 + (ev)] = (long long)gt; } } while (0)
#else
#define HT_TR(role, j, ev) do { } while (0)
#define HT_TR_CTA(ev) do { } while (0)
#endif

struct __align__(1024) Smem {
    unsigned char q[kEntryBytes];
    unsigned char ring[kStages][kEntryBytes];
    uint32_t anc[kMaxWords][kRows];
    int32_t parent[kMaxWords * 32];
    float ml[2][kRows][2];
    int32_t len[kMaxB];
    int32_t nkt[kMaxB];
    int32_t pre[kMaxB + 1];
    unsigned long long kv_full[kStages], kv_empty[kStages], q_full, q_empty, s_full[2], p_ready[2], o_done[2], mma_drain;
    uint32_t tmem_base;
    int abort;
    int merge_here[2];
    int direct;
};

// ---------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait for the completion of the phase with the given parity.  Returns false (and
// raises the CTA's abort flag) when about a second passes without it.
__device__ __forceinline__ bool mbar_wait(void *bar, uint32_t parity, volatile int *abort_flag,
                                          bool honor_abort = true) {
    if (honor_abort && *abort_flag) return false;
    const uint32_t addr = smem_u32(bar);
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u) {
            if (honor_abort && *abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > 2000000000ll) { *abort_flag = 1; return false; }
        }
    }
}

__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, void *bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(void *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 consecutive TMEM columns of this thread's lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t *r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t *r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {             // 2^x, -inf -> 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}


__device__ __forceinline__ unsigned int ld_relaxed_gpu(const unsigned int *ptr) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// Two fp32 values in one 64-bit register, for the paired fp32 instructions.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ void softmax_groups_sync() {   // the 256 softmax threads
    asm volatile("bar.sync 1, 256;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  Offsets are in 16-byte units.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo16, uint32_t sbo16) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)lbo16 << 16) | ((uint64_t)sbo16 << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulate, M = N = 128.
__device__ __forceinline__ uint32_t instr_desc(int is_bf16, int b_mn_major) {
    const uint32_t fmt = is_bf16 ? 1u : 0u;
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)b_mn_major << 16) | ((128u >> 3) << 17) |
           ((128u >> 4) << 24);
}

// ---------------------------------------------------------------------------------------
// Work partition, evaluated identically by every role and by the merge kernel.
// ---------------------------------------------------------------------------------------
struct Segment {
    int b, hk, rt, kt0, len, nkt;
};

__device__ __forceinline__ Segment locate(const int32_t *pre, const int32_t *nkt, int B, int n_rt, int t, int t_end, int &b_hint) {
    int b = b_hint;
    while (b < B - 1 && t >= pre[b + 1]) ++b;
    b_hint = b;
    Segment s;
    s.b = b;
    s.nkt = nkt[b];
    const int local = t - pre[b];
    const int unit = local / s.nkt;
    s.kt0 = local - unit * s.nkt;
    s.hk = unit / n_rt;
    s.rt = unit - s.hk * n_rt;
    s.len = min(s.nkt - s.kt0, t_end - t);
    return s;
}

__device__ __forceinline__ int tiles_per_cta(int total, int grid) { return (total + grid - 1) / grid; }

// Tiles per CTA.  An even share cuts nearly every unit in two, and every cut costs a partial
// result in the workspace and a merge at the end.  While the cache is streamed at memory speed a
// few idle SMs cost less than that, so when all sequences are equally long and some whole
// multiple or whole fraction of a unit lies within 20 % above the even share, ranges of that
// length are used and cuts fall on unit boundaries (or, for fractions, near them).
__device__ __forceinline__ int choose_per(int total, int grid, const int32_t *nkt, int B) {
    const int even = tiles_per_cta(total, grid);
    int n = 0;
    for (int b = 0; b < B; ++b) {
        if (nkt[b] == 0) continue;
        if (n != 0 && nkt[b] != n) return even;
        n = nkt[b];
    }
    if (n == 0 || even == 0) return even;
    int cand;
    if (n >= even) {
        const int k = n / even;                       // largest count of parts whose length is >= even
        cand = (n + k - 1) / k;
    } else {
        cand = (even + n - 1) / n * n;                // whole units
    }
    return (cand * 5 <= even * 6) ? cand : even;
}

// Validates every sequence and fills len / nkt / pre.  Called by all threads of a block.
template <int NT>
__device__ __forceinline__ void plan_sequences(const Params &p, int32_t *s_len, int32_t *s_nkt, int32_t *s_pre,
                                               bool write_status) {
    for (int b = threadIdx.x; b < p.B; b += NT) s_nkt[b] = 0;       // 0 = legal so far
    __syncthreads();
    for (int i = threadIdx.x; i < p.B * p.N; i += NT) {
        const int b = i / p.N, c = i - b * p.N;
        const int par = p.parent[i];
        if (par < -1 || par >= c) s_nkt[b] = -1;                     // benign race: all writers store -1
    }
    __syncthreads();
    for (int b = threadIdx.x; b < p.B; b += NT) {
        const int L = p.kv_len[b];
        int code = HT_STATUS_OK;
        if (s_nkt[b] < 0) code = HT_STATUS_BAD_TREE;
        if (L < 0 || (long long)L + p.N > p.cap) code = HT_STATUS_BAD_LEN;
        s_len[b] = L;
        s_nkt[b] = code == HT_STATUS_OK ? (L + p.N + kTile - 1) / kTile : 0;
        if (write_status) p.status[b] = code;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int b = 0; b < p.B; ++b) {
            s_pre[b] = acc;
            acc += s_nkt[b] * p.Hkv * p.n_rt;
        }
        s_pre[p.B] = acc;
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------
// Main kernel
// ---------------------------------------------------------------------------------------
template <bool kBf16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    if (kBf16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&v);
    } else {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&v);
    }
}

// A unit that was cut between CTAs: which one, and which CTAs hold its parts.
struct CutUnit {
    int valid, unit, b, hk, rt, t0, c_lo, c_hi;
};

// Merge of the parts of a cut unit by the 256 softmax threads of the CTA that delivered the
// last part.  Threads r and r + 128 own query row r, 64 features each; a warp reads 32
// consecutive rows of one feature group at a time (contiguous in the part's layout), and the
// loads of a part are independent of one another so that one round trip to L2 fetches it.
template <bool kBf16>
__device__ __noinline__ void merge_parts(const Params &p, const CutUnit &cu, int per, int tid256) {
    const int row = tid256 & 127, half = tid256 >> 7;
    const int node = cu.rt * p.rows_per_tile_nodes + row / p.g;
    if (node >= p.N) return;
    const int head = cu.hk * p.g + row % p.g;
    float M = -INFINITY, l = 0.f;
    float acc[64];
#pragma unroll
    for (int x = 0; x < 64; ++x) acc[x] = 0.f;
#pragma unroll 1
    for (int c = cu.c_lo; c <= cu.c_hi; ++c) {
        const int slot = 2 * c + ((max(cu.t0, c * per) == c * per) ? 0 : 1);
        const float *pslot = p.part + (size_t)slot * kSlotFloats;
        const float m = __ldcg(pslot + kRows * kD + row), lp = __ldcg(pslot + kRows * kD + kRows + row);
        float4 v[16];
#pragma unroll
        for (int x = 0; x < 16; ++x) v[x] = __ldcg(reinterpret_cast<const float4 *>(pslot) + (half * 16 + x) * kRows + row);
        const float Mn = fmaxf(M, m);
        const float fa = (M == -INFINITY) ? 0.f : exp2f(M - Mn);
        const float fb = (m == -INFINITY) ? 0.f : exp2f(m - Mn);
        l = l * fa + lp * fb;
#pragma unroll
        for (int x = 0; x < 16; ++x) {
            acc[4 * x] = acc[4 * x] * fa + v[x].x * fb;
            acc[4 * x + 1] = acc[4 * x + 1] * fa + v[x].y * fb;
            acc[4 * x + 2] = acc[4 * x + 2] * fa + v[x].z * fb;
            acc[4 * x + 3] = acc[4 * x + 3] * fa + v[x].w * fb;
        }
        M = Mn;
    }
    const float inv = 1.f / l;
    unsigned char *dst = static_cast<unsigned char *>(p.out) +
                         ((((size_t)cu.b * p.N + node) * p.Hq + head) * kD + half * 64) * 2;
#pragma unroll
    for (int x = 0; x < 8; ++x)
        *reinterpret_cast<uint4 *>(dst + x * 16) =
            make_uint4(pack2<kBf16>(acc[8 * x] * inv, acc[8 * x + 1] * inv), pack2<kBf16>(acc[8 * x + 2] * inv, acc[8 * x + 3] * inv),
                       pack2<kBf16>(acc[8 * x + 4] * inv, acc[8 * x + 5] * inv), pack2<kBf16>(acc[8 * x + 6] * inv, acc[8 * x + 7] * inv));
}

template <bool kBf16>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const Params p) {
    extern __shared__ unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sm.abort;
    if (threadIdx.x == 0) HT_TR_CTA(0);

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&sm.kv_full[i], 1); mbar_init(&sm.kv_empty[i], 1); }
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_empty, 1);
        mbar_init(&sm.mma_drain, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&sm.s_full[i], 1); mbar_init(&sm.p_ready[i], 128); mbar_init(&sm.o_done[i], 1); }
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    plan_sequences<kThreads>(p, sm.len, sm.nkt, sm.pre, blockIdx.x == 0);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    const int total = sm.pre[p.B];
    const int per = choose_per(total, p.grid, sm.nkt, p.B);
    const int t_begin = min((int)blockIdx.x * per, total);
    const int t_end = min(t_begin + per, total);

    if (warp == 8) {
        // ------------------------------- TMA producer -------------------------------
        if (lane == 0) {
            int b_hint = 0, ring_i = 0, seg_i = 0;
            HT_TR_CTA(1);
            for (int t = t_begin; t < t_end && !*abort_flag;) {
                const Segment s = locate(sm.pre, sm.nkt, p.B, p.n_rt, t, t_end, b_hint);
                if (seg_i > 0 && !mbar_wait(&sm.q_empty, (seg_i - 1) & 1, abort_flag)) break;
                mbar_expect_tx(&sm.q_full, kEntryBytes);
                tma_load_4d(sm.q, &tm_q, &sm.q_full, 0, s.hk * p.g, s.rt * p.rows_per_tile_nodes, s.b);
                tma_load_4d(sm.q + kSlabBytes, &tm_q, &sm.q_full, 64, s.hk * p.g, s.rt * p.rows_per_tile_nodes, s.b);
                ++seg_i;
                for (int i = 0; i < 2 * s.len; ++i) {
                    const int kt = s.kt0 + (i >> 1);
                    const int slot = ring_i % kStages, use = ring_i / kStages;
                    if (use > 0 && !mbar_wait(&sm.kv_empty[slot], (use - 1) & 1, abort_flag)) break;
                    HT_TR(0, ring_i >> 1, ring_i & 1);
                    const CUtensorMap *tm = (i & 1) ? &tm_v : &tm_k;
                    mbar_expect_tx(&sm.kv_full[slot], kEntryBytes);
                    tma_load_4d(sm.ring[slot], tm, &sm.kv_full[slot], 0, kt * kTile, s.hk, s.b);
                    tma_load_4d(sm.ring[slot] + kSlabBytes, tm, &sm.kv_full[slot], 64, kt * kTile, s.hk, s.b);
                    ++ring_i;
                }
                t += s.len;
            }
            if (*abort_flag) {
                // Every copy this thread issued must have landed before the CTA exits: wait, with the
                // usual bound, for the latest armed phase of each ring slot and of the Q buffer.
                for (int e = max(0, ring_i - kStages); e < ring_i; ++e)
                    mbar_wait(&sm.kv_full[e % kStages], (e / kStages) & 1, abort_flag, false);
                if (seg_i > 0) mbar_wait(&sm.q_full, (seg_i - 1) & 1, abort_flag, false);
            }
        }
    } else if (warp == 9) {
        // ------------------------------- MMA issuer -------------------------------
        if (lane == 0) {
            const uint32_t idesc_qk = instr_desc(kBf16, 0), idesc_pv = instr_desc(kBf16, 1);
            const uint32_t q_addr = smem_u32(sm.q);
            int b_hint = 0, j = 0, seg_i = 0;
            int prev_first = 0;          // is tile j-1 the first of its stream within its segment?
            auto issue_pv = [&](int jj, int first) {
                const int s = jj & 1;
                mbar_wait(&sm.p_ready[s], (jj >> 1) & 1, abort_flag);
                HT_TR(1, jj, 2);
                const int e = 2 * jj + 1, slot = e % kStages;
                mbar_wait(&sm.kv_full[slot], (e / kStages) & 1, abort_flag);
                tc_fence_after();
                if (!*abort_flag) {
                    const uint32_t v_addr = smem_u32(sm.ring[slot]);
#pragma unroll
                    for (int kk = 0; kk < kTile / 16; ++kk) {
                        // V tile as B operand, MN-major: 64 features contiguous (one swizzled 128-byte
                        // line per key), the second 64-feature slab one slab further (LBO), groups of
                        // 8 keys 1 KiB apart (SBO); 16 keys per instruction = 2 KiB.
                        const uint64_t b_desc = smem_desc(v_addr + kk * 2048, kSlabBytes >> 4, 1024 >> 4);
                        mma_ts(tmem + 256 + s * 128, tmem + s * 128 + kk * 8, b_desc, idesc_pv, (kk > 0 || !first) ? 1u : 0u);
                    }
                }
                tc_commit(&sm.kv_empty[slot]);
                tc_commit(&sm.o_done[s]);
            };
            for (int t = t_begin; t < t_end;) {
                const Segment sg = locate(sm.pre, sm.nkt, p.B, p.n_rt, t, t_end, b_hint);
                mbar_wait(&sm.q_full, seg_i & 1, abort_flag);
                for (int i = 0; i < sg.len; ++i) {
                    const int s = j & 1;
                    const int e = 2 * j, slot = e % kStages;
                    mbar_wait(&sm.kv_full[slot], (e / kStages) & 1, abort_flag);
                    tc_fence_after();
                    HT_TR(1, j, 0);
                    if (!*abort_flag) {
                        const uint32_t k_addr = smem_u32(sm.ring[slot]);
#pragma unroll
                        for (int kk = 0; kk < kD / 16; ++kk) {
                            // K-major operands: 16 features = 32 bytes inside the 128-byte swizzled
                            // line; the second 64-feature slab lies one slab further.
                            const uint32_t off = (kk >> 2) * kSlabBytes + (kk & 3) * 32;
                            mma_ss(tmem + s * 128, smem_desc(q_addr + off, 1, 1024 >> 4),
                                   smem_desc(k_addr + off, 1, 1024 >> 4), idesc_qk, kk > 0 ? 1u : 0u);
                        }
                    }
                    tc_commit(&sm.s_full[s]);
                    tc_commit(&sm.kv_empty[slot]);
                    if (i == sg.len - 1) tc_commit(&sm.q_empty);
                    if (j > 0) issue_pv(j - 1, prev_first);
                    prev_first = i < 2;
                    ++j;
                }
                t += sg.len;
                ++seg_i;
            }
            if (j > 0) issue_pv(j - 1, prev_first);
            // No tensor-core operation of this CTA may be in flight when its TMEM is freed.
            tc_commit(&sm.mma_drain);
            mbar_wait(&sm.mma_drain, 0, abort_flag, false);
        }
    } else {
        // ------------------------------- softmax groups -------------------------------
        const int s = warp >> 2;                       // stream of this group
        const int row = threadIdx.x & 127;             // query row within the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int tid256 = threadIdx.x;                // 0..255 among the softmax threads
        const int words = (p.N + 31) >> 5;
        const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
        int b_hint = 0, J = 0;
        float xa_e[32], xb_e[32];
        CutUnit cut[2];
        unsigned int ticket[2] = {0u, 0u};
        cut[0].valid = cut[1].valid = 0;
        int anc_b = -1, anc_rt = -1;           // sequence / row tile the ancestor words were built for
        for (int t = t_begin; t < t_end;) {
            const Segment sg = locate(sm.pre, sm.nkt, p.B, p.n_rt, t, t_end, b_hint);
            const int L = sm.len[sg.b];
            // --- ancestor masks of this tile's rows (kept while sequence and row tile stay the same) ---
            const int node = sg.rt * p.rows_per_tile_nodes + row / p.g;
            const bool real = node < p.N;
            if (sg.b != anc_b || sg.rt != anc_rt) {
                softmax_groups_sync();                 // previous segment no longer reads parent / anc
                for (int c = tid256; c < p.N; c += 256) sm.parent[c] = p.parent[(size_t)sg.b * p.N + c];
                softmax_groups_sync();
                if (s == 0) {
                    for (int w = 0; w < words; ++w) sm.anc[w][row] = 0u;   // padding rows see the context only; their results are dropped
                    if (real)
                        for (int c = node; c >= 0; c = sm.parent[c]) sm.anc[c >> 5][row] |= 1u << (c & 31);
                }
                softmax_groups_sync();
                anc_b = sg.b;
                anc_rt = sg.rt;
            }

            // A segment that is only part of its unit: which CTAs hold the other parts.  How many of
            // them have been delivered is asked anew at every tile and looked at in the epilogue, so
            // that the answer never has to be waited for.
            const bool complete = sg.kt0 == 0 && sg.len == sg.nkt;
            const int cut_k = (t == t_begin) ? 0 : 1;
            unsigned int delivered = 0, delivered_old = 0;   // newest answer, and the one before it
            if (!complete) {
                CutUnit &cu = cut[cut_k];
                cu.unit = (sg.b * p.Hkv + sg.hk) * p.n_rt + sg.rt;
                cu.b = sg.b; cu.hk = sg.hk; cu.rt = sg.rt;
                cu.t0 = sm.pre[sg.b] + (sg.hk * p.n_rt + sg.rt) * sg.nkt;
                cu.c_lo = cu.t0 / per;
                cu.c_hi = (cu.t0 + sg.nkt - 1) / per;
            }

            float m_ref = -INFINITY, l_sum = 0.f;
            int n_mine = 0, last_jj = 0;
#pragma unroll 1
            for (int i = 0; i < sg.len; ++i) {
                const int jj = J + i;
                if ((jj & 1) != s) continue;
                const int kt = sg.kt0 + i;
                if (!complete && tid256 == 0) {
                    delivered_old = delivered;
                    delivered = ld_relaxed_gpu(&p.tickets[cut[cut_k].unit]);
                }
                HT_TR(2 + s, jj, 0);
                mbar_wait(&sm.s_full[s], (jj >> 1) & 1, abort_flag);
                tc_fence_after();
                HT_TR(2 + s, jj, 1);
                const uint32_t s_addr = tmem + lane_base + s * 128;
                const int tile_lo = kt * kTile;
                float *const xa = xa_e, *const xb = xb_e;
                if (tile_lo + kTile > L) {
                    // The tile reaches into the tree rows / the tail: overwrite the scores of keys this
                    // row must not see with -inf, in place, so that the two passes below need no mask.
                    // Context keys are visible, tree key c iff bit c of the row's ancestor words, the
                    // tail never (whatever those cache rows hold, NaN included).
#pragma unroll 1
                    for (int w = 0; w < 4; ++w) {
                        const int cc0 = tile_lo + 32 * w - L;           // tree index of the word's first key
                        if (cc0 <= -32) continue;
                        const int wi = cc0 >> 5, sh = cc0 & 31;         // arithmetic shift: -1 for cc0 in (-32, 0)
                        const uint32_t lo = wi < 0 ? 0xFFFFFFFFu : (wi < words ? sm.anc[wi][row] : 0u);
                        const uint32_t hi = (wi + 1 >= 0 && wi + 1 < words) ? sm.anc[wi + 1][row] : 0u;
                        const uint32_t vis = __funnelshift_r(lo, hi, sh);
                        tmem_ld32(s_addr + w * 32, xa);
                        tmem_ld_wait();
                        uint32_t r[32];
#pragma unroll
                        for (int c = 0; c < 32; ++c) r[c] = ((vis >> c) & 1u) ? __float_as_uint(xa[c]) : 0xFF800000u;
                        tmem_st32(s_addr + w * 32, r);
                    }
                    tmem_st_wait();
                }
                // --- pass 1: row maximum, 32 scores at a time, the next chunk in flight meanwhile ---
                float mx0 = -INFINITY, mx1 = -INFINITY;
                tmem_ld32(s_addr, xa);
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    tmem_ld_wait();
                    tmem_ld32(s_addr + (2 * h + 1) * 32, xb);
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        mx0 = max3(mx0, xa[c], xa[c + 1]);
                        mx1 = max3(mx1, xa[c + 2], xa[c + 3]);
                    }
                    tmem_ld_wait();
                    tmem_ld32(s_addr + ((2 * h + 2) & 3) * 32, xa);   // after the last chunk: chunk 0 again, for pass 2
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        mx0 = max3(mx0, xb[c], xb[c + 1]);
                        mx1 = max3(mx1, xb[c + 2], xb[c + 3]);
                    }
                }
                const float mx = fmaxf(mx0, mx1) * p.scale_log2;   // scale > 0: max commutes with scaling
                HT_TR(2 + s, jj, 2);
                // --- running maximum, raised lazily ---
                const float m_new = fmaxf(m_ref, mx);
                const bool grow = (m_ref != -INFINITY) && (m_new > m_ref + kRescaleThreshold);
                if (m_ref == -INFINITY) m_ref = m_new;  // nothing accumulated yet for this row
                if (__any_sync(0xffffffffu, grow)) {
                    // Scores of this tile being ready implies this stream's previous P.V has completed
                    // (the tensor pipe runs in issue order), so its accumulator may be rescaled here.
                    const float f = grow ? exp2f(m_ref - m_new) : 1.f;
                    const uint32_t o_addr = tmem + lane_base + 256 + s * 128;
                    tmem_ld_wait();                    // the prefetched chunk has landed in xa before xb is reused
#pragma unroll 1
                    for (int c4 = 0; c4 < 4; ++c4) {
                        uint32_t r[32];
                        tmem_ld32(o_addr + c4 * 32, xb);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(xb[c] * f);
                        tmem_st32(o_addr + c4 * 32, r);
                    }
                    tmem_st_wait();
                    l_sum *= f;
                    if (grow) m_ref = m_new;
                }
                const float base = (m_ref == -INFINITY) ? 0.f : m_ref;
                // --- pass 2: exponentials, row sum, P to TMEM as packed 16-bit pairs.  P chunk c lands
                // in columns [16 c, 16 c + 16), which hold scores already consumed. ---
                const unsigned long long nbase2 = pack_f32x2(-base, -base);
                unsigned long long acc2 = pack_f32x2(0.f, 0.f);
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    uint32_t r[16];
                    tmem_ld_wait();
                    tmem_ld32(s_addr + (2 * h + 1) * 32, xb);
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        float p0, p1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(xa[2 * c], xa[2 * c + 1]), scale2, nbase2), p0, p1);
                        p0 = ex2(p0);
                        p1 = ex2(p1);
                        acc2 = add_f32x2(acc2, pack_f32x2(p0, p1));
                        r[c] = pack2<kBf16>(p0, p1);
                    }
                    tmem_st16(s_addr + (2 * h) * 16, r);
                    tmem_ld_wait();
                    if (h == 0) tmem_ld32(s_addr + 2 * 32, xa);
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        float p0, p1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(xb[2 * c], xb[2 * c + 1]), scale2, nbase2), p0, p1);
                        p0 = ex2(p0);
                        p1 = ex2(p1);
                        acc2 = add_f32x2(acc2, pack_f32x2(p0, p1));
                        r[c] = pack2<kBf16>(p0, p1);
                    }
                    tmem_st16(s_addr + (2 * h + 1) * 16, r);
                }
                {
                    float a0, a1;
                    unpack_f32x2(acc2, a0, a1);
                    l_sum += a0 + a1;
                }
                tmem_st_wait();
                // --- last tile of the unit: rows of V past the tree are not data; make them zero ---
                if (kt == sg.nkt - 1) {
                    const int valid = L + p.N - tile_lo;
                    if (valid < kTile) {
                        const int e = 2 * jj + 1, slot = e % kStages;
                        mbar_wait(&sm.kv_full[slot], (e / kStages) & 1, abort_flag);
                        const int vecs = (kTile - valid) * 8;               // 16-byte vectors per slab
                        for (int v = row; v < vecs; v += 128) {
                            *reinterpret_cast<uint4 *>(sm.ring[slot] + valid * 128 + v * 16) = make_uint4(0, 0, 0, 0);
                            *reinterpret_cast<uint4 *>(sm.ring[slot] + kSlabBytes + valid * 128 + v * 16) = make_uint4(0, 0, 0, 0);
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    }
                }
                tc_fence_before();
                HT_TR(2 + s, jj, 3);
                mbar_arrive(&sm.p_ready[s]);
                ++n_mine;
                last_jj = jj;
            }
            // --- segment epilogue: merge the two streams, write the result or a partial ---
            if (n_mine > 0) {
                mbar_wait(&sm.o_done[s], (last_jj >> 1) & 1, abort_flag);
                tc_fence_after();
            }
            HT_TR(4, J, 0);
            sm.ml[s][row][0] = m_ref;
            sm.ml[s][row][1] = l_sum;
            // With one other part and that part already in the workspace, this CTA finishes the unit
            // from its registers; otherwise it leaves its own part there.
            if (tid256 == 0) sm.direct = !complete && cut[cut_k].c_hi - cut[cut_k].c_lo == 1 && delivered_old == 1u;
            tc_fence_before();
            softmax_groups_sync();
            tc_fence_after();
            const float m0 = sm.ml[0][row][0], l0 = sm.ml[0][row][1];
            const float m1 = sm.ml[1][row][0], l1 = sm.ml[1][row][1];
            const bool direct = sm.direct;
            const float M = fmaxf(m0, m1);
            const float f0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - M);
            const float f1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - M);
            const float l_tot = f0 * l0 + f1 * l1;
            // which streams own tiles of this segment (uniform over the CTA)
            const bool has0 = sg.len >= 2 || (J & 1) == 0;
            const bool has1 = sg.len >= 2 || (J & 1) == 1;
            const int head = sg.hk * p.g + row % p.g;
            float *pslot = p.part + (size_t)(2 * (int)blockIdx.x + cut_k) * kSlotFloats;
            const float *oslot = pslot;                // the other part, when finishing the unit here
            float g0, g1, gb = 0.f;
            if (direct) {
                const CutUnit &cu = cut[cut_k];
                const int oc = (cu.c_lo == (int)blockIdx.x) ? cu.c_hi : cu.c_lo;
                oslot = p.part + (size_t)(2 * oc + ((max(cu.t0, oc * per) == oc * per) ? 0 : 1)) * kSlotFloats;
                __threadfence();
                const float m_o = __ldcg(oslot + kRows * kD + row), l_o = __ldcg(oslot + kRows * kD + kRows + row);
                const float Mn = fmaxf(M, m_o);
                const float fa = (M == -INFINITY) ? 0.f : exp2f(M - Mn);
                const float fb = (m_o == -INFINITY) ? 0.f : exp2f(m_o - Mn);
                const float inv = 1.f / (l_tot * fa + l_o * fb);
                g0 = f0 * fa * inv;
                g1 = f1 * fa * inv;
                gb = fb * inv;
            } else {
                const float inv = complete ? 1.f / l_tot : 1.f;
                g0 = f0 * inv;
                g1 = f1 * inv;
            }
            const bool final = complete || direct;
#pragma unroll 1
            for (int c2 = 0; c2 < 2; ++c2) {
                const int col0 = s * 64 + c2 * 32;
                tmem_ld32(tmem + lane_base + 256 + col0, xa_e);
                tmem_ld32(tmem + lane_base + 384 + col0, xb_e);
                tmem_ld_wait();
                // an accumulator no tile of this segment wrote holds stale numbers (possibly NaN)
#pragma unroll
                for (int c = 0; c < 32; ++c) xa_e[c] = (has0 ? g0 * xa_e[c] : 0.f) + (has1 ? g1 * xb_e[c] : 0.f);
                if (!real) continue;
                if (direct) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float4 v = __ldcg(reinterpret_cast<const float4 *>(oslot) + (col0 / 4 + c) * kRows + row);
                        xa_e[4 * c] = fmaf(gb, v.x, xa_e[4 * c]);
                        xa_e[4 * c + 1] = fmaf(gb, v.y, xa_e[4 * c + 1]);
                        xa_e[4 * c + 2] = fmaf(gb, v.z, xa_e[4 * c + 2]);
                        xa_e[4 * c + 3] = fmaf(gb, v.w, xa_e[4 * c + 3]);
                    }
                }
                if (final) {
                    uint32_t w[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) w[c] = pack2<kBf16>(xa_e[2 * c], xa_e[2 * c + 1]);
                    unsigned char *dst = static_cast<unsigned char *>(p.out) +
                                         ((((size_t)sg.b * p.N + node) * p.Hq + head) * kD + col0) * 2;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        *reinterpret_cast<uint4 *>(dst + c * 16) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c)      // 32 consecutive rows of one feature group: 512 contiguous bytes per warp
                        reinterpret_cast<float4 *>(pslot)[(col0 / 4 + c) * kRows + row] = make_float4(xa_e[4 * c], xa_e[4 * c + 1], xa_e[4 * c + 2], xa_e[4 * c + 3]);
                }
            }
            if (!final && s == 0 && real) {
                pslot[kRows * kD + row] = M;
                pslot[kRows * kD + kRows + row] = l_tot;
            }
            tc_fence_before();
            softmax_groups_sync();                     // both accumulators are free for the next segment
            if (!final) {
                // This CTA's part is in the workspace: take the unit's ticket.  One thread orders the
                // CTA's stores (the barrier above collected them) and draws; the answer is looked at
                // after the CTA's last segment.
                cut[cut_k].valid = 1;
                if (tid256 == 0) {
                    __threadfence();
                    ticket[cut_k] = atomicAdd(&p.tickets[cut[cut_k].unit], 1u);
                }
            }
            HT_TR(4, J, 1);
            J += sg.len;
            t += sg.len;
        }
        if (tid256 == 0) HT_TR_CTA(2);
        // --- cut units: the CTA that delivers the last part of a unit merges all parts; nobody waits ---
        if (cut[0].valid || cut[1].valid) {
            if (tid256 == 0)
                for (int k = 0; k < 2; ++k)
                    sm.merge_here[k] = cut[k].valid && ticket[k] == (unsigned)(cut[k].c_hi - cut[k].c_lo);
            softmax_groups_sync();
            for (int k = 0; k < 2; ++k)
                if (sm.merge_here[k]) {
                    __threadfence();
                    merge_parts<kBf16>(p, cut[k], per, tid256);
                }
        }
        HT_TR(4, 39, 0);
    }

    // ------------------------------- teardown -------------------------------
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) HT_TR_CTA(3);
    if (sm.abort && threadIdx.x == 0) {
        for (int b = 0; b < p.B; ++b)
            if (sm.nkt[b] > 0) p.status[b] = HT_STATUS_TIMEOUT;
    }
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace tc

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

static int sm_count() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

bool attn_tc_applicable(const ht_attn_desc &d) {
    if (d.flags & HT_ATTN_FORCE_SIMT) return false;
    if (d.dtype != HT_F16 && d.dtype != HT_BF16) return false;
    if (d.D != tc::kD) return false;
    const int g = d.Hq / d.Hkv;
    if (g > tc::kRows || (g & (g - 1)) != 0) return false;
    if (d.N > tc::kMaxWords * 32 || d.B > tc::kMaxB) return false;
    if (d.num_splits != 0) return false;              // an explicit split count asks for the split-KV ALU kernel
    return true;
}

static size_t ticket_bytes(const ht_attn_desc &d) {
    const int g = d.Hq / d.Hkv;
    const size_t units = (size_t)d.B * d.Hkv * ((d.N * g + tc::kRows - 1) / tc::kRows);
    return (units * sizeof(unsigned int) + 255) / 256 * 256;
}

// Arrival counters of the units, then two partial-result slots per CTA.
size_t attn_tc_workspace(const ht_attn_desc &d) {
    return ticket_bytes(d) + (size_t)2 * sm_count() * tc::kSlotFloats * sizeof(float);
}

// The kernels' dynamic shared memory limit is raised once per device.
static cudaError_t ensure_smem_attr(size_t smem) {
    static bool done[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(tc::attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tc::attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) done[dev] = true;
    return cudaSuccess;
}

static int make_map(CUtensorMap *map, const void *base, int dtype, const cuuint64_t dims[4], const cuuint64_t strides_b[3],
                    const cuuint32_t box[4]) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(HT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint32_t elem_strides[4] = {1, 1, 1, 1};
    const CUresult r = fn(map, dtype == HT_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                          const_cast<void *>(base), dims, strides_b, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HT_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    return HT_OK;
}

#ifdef HT_TC_TRACE
static long long *g_trace = nullptr;
extern "C" void ht_set_trace(void *ptr) { g_trace = static_cast<long long *>(ptr); }
#endif

int launch_attn_tc(const ht_attn_desc &d, const void *q, const void *kc, const void *vc, const int32_t *kv_len,
                   const int32_t *parent, void *out, void *ws, size_t ws_bytes, int32_t *status, cudaStream_t s) {
    if (ws_bytes < attn_tc_workspace(d) || !ws)
        return fail(HT_ERR_WORKSPACE, "workspace holds %zu bytes, %zu needed", ws ? ws_bytes : 0, attn_tc_workspace(d));
    const int g = d.Hq / d.Hkv;
    const long long sh = d.kv_stride_h ? d.kv_stride_h : (long long)d.cap * d.D;
    const long long sb = d.kv_stride_b ? d.kv_stride_b : (long long)d.Hkv * d.cap * d.D;
    CUtensorMap tm_q, tm_k, tm_v;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)d.D, (cuuint64_t)d.Hq, (cuuint64_t)d.N, (cuuint64_t)d.B};
        const cuuint64_t strides[3] = {(cuuint64_t)d.D * 2, (cuuint64_t)d.Hq * d.D * 2, (cuuint64_t)d.N * d.Hq * d.D * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)g, (cuuint32_t)(tc::kRows / g), 1};
        int rc = make_map(&tm_q, q, d.dtype, dims, strides, box);
        if (rc != HT_OK) return rc;
    }
    {
        const cuuint64_t dims[4] = {(cuuint64_t)d.D, (cuuint64_t)d.cap, (cuuint64_t)d.Hkv, (cuuint64_t)d.B};
        const cuuint64_t strides[3] = {(cuuint64_t)d.D * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)tc::kTile, 1, 1};
        int rc = make_map(&tm_k, kc, d.dtype, dims, strides, box);
        if (rc != HT_OK) return rc;
        rc = make_map(&tm_v, vc, d.dtype, dims, strides, box);
        if (rc != HT_OK) return rc;
    }
    tc::Params p;
    p.kv_len = kv_len; p.parent = parent; p.status = status; p.out = out; p.tickets = static_cast<unsigned int *>(ws);
    p.part = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + ticket_bytes(d));
    p.B = d.B; p.N = d.N; p.Hq = d.Hq; p.Hkv = d.Hkv; p.g = g; p.cap = d.cap;
    p.rows_per_tile_nodes = tc::kRows / g;
    p.n_rt = (d.N * g + tc::kRows - 1) / tc::kRows;
    const float scale = d.scale > 0.f ? d.scale : 1.f / sqrtf((float)d.D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.is_bf16 = d.dtype == HT_BF16;
    p.grid = sm_count();
#ifdef HT_TC_TRACE
    p.trace = g_trace;
#endif
    const size_t smem = sizeof(tc::Smem) + 1024;
    const long long units = (long long)d.B * d.Hkv * p.n_rt;
    if (units > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "too many (sequence, head, row tile) units");
    cudaError_t e = ensure_smem_attr(smem);
    if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    e = cudaMemsetAsync(p.tickets, 0, (size_t)units * sizeof(unsigned int), s);
    if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    if (d.dtype == HT_BF16) tc::attn_tc_kernel<true><<<p.grid, tc::kThreads, smem, s>>>(tm_q, tm_k, tm_v, p);
    else tc::attn_tc_kernel<false><<<p.grid, tc::kThreads, smem, s>>>(tm_q, tm_k, tm_v, p);
    return check_launch("ht_tree_attention (tcgen05)");
}

}  // namespace ht
