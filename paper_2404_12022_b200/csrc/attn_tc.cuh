// Building blocks shared by the tensor-core tree-attention kernels: PTX wrappers (mbarrier, TMA,
// tcgen05), the work plan every role evaluates identically, and the merge of cut units.
#pragma once
#include <cuda.h>

#include "ht_common.cuh"

namespace ht {
namespace tc {

constexpr int kTile = 128;                 // keys per tile
constexpr int kRows = 128;                 // query rows per tile (UMMA M)
constexpr int kD = 128;
constexpr int kStages = 4;                 // ring entries (each one K or one V tile)
constexpr int kEntryBytes = kTile * kD * 2;
constexpr int kSlabBytes = kEntryBytes / 2;   // [128 rows][64 elements] = 16 KiB
constexpr int kThreads = 320;
constexpr int kMaxB = 256;
constexpr int kPlanWords = 12;         // per, t_begin, t_end, first segment (b, hk, rt, kt0, len, nkt)
constexpr int kMaxWords = 32;              // ancestor words per row -> N <= 1024
constexpr int kSlotFloats = kRows * kD + 2 * kRows;   // one partial result: O as [32 feature groups][128 rows][4], m[128], l[128]
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;  // log2 domain
constexpr int kPgTiles = 8;                // paged cache: tiles whose page ids are held (4 in use or on their way + 4 being fetched)
constexpr int kPgAhead = 4;                // ... and how many tiles ahead of the fetch the ids are asked for
constexpr int kPgSub = 8;                  // pages per tile at the smallest page size (16 rows)

struct Params {
    const int32_t *kv_len, *parent;
    int32_t *status;
    void *out;
    float *part;           // partial results of cut units: [grid][2][kSlotFloats]
    unsigned int *tickets; // one arrival counter per unit, zero on entry
    int B, N, Hq, Hkv, g, cap, n_rt, rows_per_tile_nodes;   // n_rt: units per (sequence, KV head); rows_per_tile_nodes = 128 / g
    int n_row_tiles;       // 128-row tiles of the N*g query rows (= n_rt, or 2 n_rt - 1 / 2 n_rt when units are tile pairs)
    float scale_log2;
    int is_bf16;
    int grid;
    int cluster_k;         // > 1: launched as clusters of this many CTAs, one cluster per (sequence, KV head)
    int cluster_split;     // clusters per unit: 1, or 2 (each reduces its half of the keys; the two results meet in the workspace)
    int wait_kcycles;      // how long a wait on an mbarrier may last, in units of 1024 clock cycles
    int early;             // HT_ATTN_CONTEXT_FINAL: lengths, trees and context rows may be read while the kernel ahead still runs
};
// The launch is serialized programmatically behind the kernel before it in the stream: a thread passes this point once
// that kernel has completed and what it wrote is visible, and only then lets this kernel's own dependents be set up.
__device__ __forceinline__ void wait_for_kernel_ahead() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
enum : int {
    kWaitKcycles = 2000000,            // about a second
    kWaitKcyclesTest = 0               // HT_ATTN_TEST_SHORT_WAITS: a wait for anything not yet there runs out at once
};

// Paged cache: cache row r of sequence b is row r % page_size of page block_table[b * max_pages + r / page_size];
// the K / V maps then describe [page][head][row][D].  A kernel parameter of its own, read by the paged
// instantiations only.
struct PagedParams {
    const int32_t *block_table;
    int page_size, page_shift, max_pages, n_pages;      // page_size = 1 << page_shift
};

struct __align__(1024) Smem {
    unsigned char q[kEntryBytes];
    unsigned char ring[kStages][kEntryBytes];
    int32_t parent[kMaxWords * 32];
    float ml[2][kRows][2];
    int32_t len[kMaxB];
    int32_t nkt[kMaxB];
    int32_t pre[kMaxB + 1];
    int32_t plan[kPlanWords];          // the CTA's share of the tiles and its first segment (plan_sequences)
    unsigned char bad_page[kMaxB];     // paged cache, early start: sequences whose bad page entry is reported behind the wait
    unsigned long long kv_full[kStages], kv_empty[kStages], q_full, q_empty, s_full[2], p_ready[2], o_done[2], mma_drain;
    int abort, wait_kcycles;           // the abort flag, and right behind it the limit of a wait (the waits read both as one 8-byte word)
    uint32_t tmem_base;
    int merge_here[2];
    int direct;
    int32_t pg[kPgTiles][kPgSub];      // paged cache: page ids of the tiles about to be fetched
    uint32_t anc[kMaxWords][kRows];    // ancestor words of the tile's rows; last member: only ceil(N / 32) words are allocated
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
// raises the CTA's abort flag) when the limit kept behind the abort flag (about a second) passes without it.
// honor_abort = false is for the waits that must not be cut short once the CTA has given up: those for its
// own copies in flight and for its own tensor-core operations, ahead of freeing what they write to; they
// always get the full second.
__device__ __forceinline__ bool mbar_wait(void *bar, uint32_t parity, volatile int *abort_flag,
                                          bool honor_abort = true) {
    // one load for the flag and the limit behind it
    const long long ctl = *reinterpret_cast<volatile long long *>(abort_flag);
    const int limit_k = (int)(ctl >> 32);
    if (honor_abort && (int)ctl) return false;
    // limit 0 (the test hook): polls that do not suspend, and the clock looked at after every one of them, so that
    // a wait for anything not yet there runs out at once
    const bool instant = honor_abort && limit_k == 0;
    const uint32_t addr = smem_u32(bar);
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        if (instant)
            asm volatile(
                "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        else
            asm volatile(
                "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u || instant) {
            if (honor_abort && *abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > ((long long)(honor_abort ? limit_k : kWaitKcycles) << 10)) { *abort_flag = 1; return false; }
        }
    }
}

// The same wait for the roles that are one thread's chain of dependent instructions (the MMA issuers): the
// common case -- the phase has completed or completes within the instruction's own suspension -- costs one
// try_wait and a branch; the abort flag is looked at only once the wait has to spin (out of line).  The caller
// remembers a false result and stops waiting and issuing from then on.
static __device__ __noinline__ bool mbar_wait_spin(uint32_t addr, uint32_t parity, volatile int *abort_flag) {
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > ((long long)abort_flag[1] << 10)) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ bool mbar_wait_quick(uint32_t addr, uint32_t parity, volatile int *abort_flag) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
    return mbar_wait_spin(addr, parity, abort_flag);
}

__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, void *bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// Asynchronous 4-byte copy global -> shared by the calling thread, and the group bookkeeping around it.
__device__ __forceinline__ void cp_async4(void *dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
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
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t *r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0, %1, %2, %3, %4, %5, %6, %7};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(taddr) : "memory");
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

// ---- thread-block cluster: rank, stores to a peer's shared memory, barrier of the whole cluster ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_peer(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_smem_addr), "r"(rank));
    return ra;
}
__device__ __forceinline__ void st_peer_f4(uint32_t peer_addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(peer_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_peer_f1(uint32_t peer_addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_addr), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {   // every thread of every CTA of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
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
// Instruction descriptor of kind::f16: fp32 accumulate, M = 128, N = n (a multiple of 16).
__device__ __forceinline__ uint32_t instr_desc(int is_bf16, int b_mn_major, uint32_t n = 128u) {
    const uint32_t fmt = is_bf16 ? 1u : 0u;
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)b_mn_major << 16) | ((n >> 3) << 17) |
           ((128u >> 4) << 24);
}

// ---------------------------------------------------------------------------------------
// Whole products as one instruction sequence.  The MMA-issuing threads are chains of dependent instructions that
// share their schedulers with the softmax warps, so every instruction between "operands landed" and "products
// issued" shows in the tile time; here a descriptor costs one 32-bit addition (all descriptors of an operand
// share their upper word, and the lower word is linear in the shared-memory address).
// ---------------------------------------------------------------------------------------
// Lower / upper word of the descriptor smem_desc(addr, lbo16, sbo16).
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr) { return (addr >> 4) & 0x3FFFu; }
__device__ __forceinline__ uint32_t desc_hi(uint32_t lbo16, uint32_t sbo16) {
    return (uint32_t)(smem_desc(0, lbo16, sbo16) >> 32);
}
// lbo16 sits in the lower word
__device__ __forceinline__ uint32_t desc_lo_with_lbo(uint32_t addr, uint32_t lbo16) { return desc_lo(addr) | (lbo16 << 16); }

#define HT_MMA_SS_STEP(off, pred) \
    "add.u32 al, %1, " #off ";\nadd.u32 bl, %2, " #off ";\nmov.b64 a, {al, %3};\nmov.b64 b, {bl, %3};\n" \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %4, " #pred ";\n"
// S[tmem] = Q K^T over the 128 features: both operands K-major in shared memory (a_lo / b_lo: lower descriptor
// words of feature 0, lbo included; hi: the shared upper word); 16 features = 2 descriptor units inside a
// 64-feature slab, the second slab kSlabBytes further.
__device__ __forceinline__ void mma_block_qk(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
    asm volatile(
        "{\n.reg .pred pf, pt;\n.reg .b32 al, bl;\n.reg .b64 a, b;\n"
        "setp.ne.b32 pf, %0, %0;\nsetp.eq.b32 pt, %0, %0;\n"
        HT_MMA_SS_STEP(0, pf) HT_MMA_SS_STEP(2, pt) HT_MMA_SS_STEP(4, pt) HT_MMA_SS_STEP(6, pt)
        HT_MMA_SS_STEP(1024, pt) HT_MMA_SS_STEP(1026, pt) HT_MMA_SS_STEP(1028, pt) HT_MMA_SS_STEP(1030, pt)
        "}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
}
static_assert(kSlabBytes / 16 == 1024, "slab offset in descriptor units");

#define HT_MMA_TS_STEP(acol, boff, pred) \
    "add.u32 at, %1, " #acol ";\nadd.u32 bl, %2, " #boff ";\nmov.b64 b, {bl, %3};\n" \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [at], b, %4, " #pred ";\n"
// O[tmem] (+)= P V over 64 keys: P from TMEM (16 keys = 8 columns), V MN-major in shared memory (16 keys = 2 KiB
// = 128 descriptor units).  accumulate = 0 starts the accumulator afresh.
__device__ __forceinline__ void mma_block_pv64(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p0, pt;\n.reg .b32 at, bl;\n.reg .b64 b;\n"
        "setp.ne.b32 p0, %5, 0;\nsetp.eq.b32 pt, %0, %0;\n"
        HT_MMA_TS_STEP(0, 0, p0) HT_MMA_TS_STEP(8, 128, pt) HT_MMA_TS_STEP(16, 256, pt) HT_MMA_TS_STEP(24, 384, pt)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
}
// ... over 128 keys, P in columns [0, 64) of its buffer.
__device__ __forceinline__ void mma_block_pv128(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p0, pt;\n.reg .b32 at, bl;\n.reg .b64 b;\n"
        "setp.ne.b32 p0, %5, 0;\nsetp.eq.b32 pt, %0, %0;\n"
        HT_MMA_TS_STEP(0, 0, p0) HT_MMA_TS_STEP(8, 128, pt) HT_MMA_TS_STEP(16, 256, pt) HT_MMA_TS_STEP(24, 384, pt)
        HT_MMA_TS_STEP(32, 512, pt) HT_MMA_TS_STEP(40, 640, pt) HT_MMA_TS_STEP(48, 768, pt) HT_MMA_TS_STEP(56, 896, pt)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
}
// ... over 128 keys with P as a hi + lo pair: the 16 keys of step kk are the half (kk & 1) of score chunk kk / 2,
// hi in the chunk's columns [0, 16), lo in [16, 32); both products are issued.
__device__ __forceinline__ void mma_block_pv128_hilo(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p0, pt;\n.reg .b32 at, bl;\n.reg .b64 b;\n"
        "setp.ne.b32 p0, %5, 0;\nsetp.eq.b32 pt, %0, %0;\n"
        HT_MMA_TS_STEP(0, 0, p0) HT_MMA_TS_STEP(16, 0, pt) HT_MMA_TS_STEP(8, 128, pt) HT_MMA_TS_STEP(24, 128, pt)
        HT_MMA_TS_STEP(32, 256, pt) HT_MMA_TS_STEP(48, 256, pt) HT_MMA_TS_STEP(40, 384, pt) HT_MMA_TS_STEP(56, 384, pt)
        HT_MMA_TS_STEP(64, 512, pt) HT_MMA_TS_STEP(80, 512, pt) HT_MMA_TS_STEP(72, 640, pt) HT_MMA_TS_STEP(88, 640, pt)
        HT_MMA_TS_STEP(96, 768, pt) HT_MMA_TS_STEP(112, 768, pt) HT_MMA_TS_STEP(104, 896, pt) HT_MMA_TS_STEP(120, 896, pt)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
}
// ... over 64 keys with P as a hi + lo pair: hi in columns [0, 32) of the half's buffer, lo in [32, 64).
__device__ __forceinline__ void mma_block_pv64_hilo(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p0, pt;\n.reg .b32 at, bl;\n.reg .b64 b;\n"
        "setp.ne.b32 p0, %5, 0;\nsetp.eq.b32 pt, %0, %0;\n"
        HT_MMA_TS_STEP(0, 0, p0) HT_MMA_TS_STEP(32, 0, pt) HT_MMA_TS_STEP(8, 128, pt) HT_MMA_TS_STEP(40, 128, pt)
        HT_MMA_TS_STEP(16, 256, pt) HT_MMA_TS_STEP(48, 256, pt) HT_MMA_TS_STEP(24, 384, pt) HT_MMA_TS_STEP(56, 384, pt)
        "}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit_addr(uint32_t bar_addr) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_addr) : "memory");
}

// ---------------------------------------------------------------------------------------
// Work partition, evaluated identically by every role and by the merge kernel.
// ---------------------------------------------------------------------------------------
struct Segment {
    int b, hk, rt, kt0, len, nkt;
};

// a / b for 0 <= a, 0 < b.  The plan is a chain of dependent instructions that every launch runs through before its
// first fetch, and the compiler's 32-bit division is some 35 of them: below 2^22 the quotient comes from the
// reciprocal in single precision (within one of the truth: both operands are exact, the product is off by a few
// units in its last place) and is put right by the remainder.
__device__ __forceinline__ int fast_div(int a, int b) {
    if ((a | b) >> 22) return a / b;
    int q = __float2int_rz(__fdividef((float)a, (float)b));
    const int r = a - q * b;
    q += r >= b ? 1 : (r < 0 ? -1 : 0);
    return q;
}

__device__ __forceinline__ Segment locate(const int32_t *pre, const int32_t *nkt, int B, int n_rt, int t, int t_end, int &b_hint) {
    int b = b_hint;
    while (b < B - 1 && t >= pre[b + 1]) ++b;
    b_hint = b;
    Segment s;
    s.b = b;
    s.nkt = nkt[b];
    const int local = t - pre[b];
    const int unit = fast_div(local, s.nkt);
    s.kt0 = local - unit * s.nkt;
    s.hk = n_rt == 1 ? unit : fast_div(unit, n_rt);
    s.rt = unit - s.hk * n_rt;
    s.len = min(s.nkt - s.kt0, t_end - t);
    return s;
}

// Walks the tiles of a CTA's range one by one; `locate` (two divisions) runs once per segment only.
struct TileCursor {
    Segment s;       // segment of the tile last returned
    int i;           // tiles of it returned so far
    int t, t_end, b_hint;
    __device__ __forceinline__ void init(int t_begin, int t_end_) {
        t = t_begin; t_end = t_end_; b_hint = 0; i = 0; s.len = 0; s.kt0 = 0;
    }
    // ... with the range's first segment already known (an empty range: first.len == 0)
    __device__ __forceinline__ void init(int t_begin, int t_end_, const Segment &first) {
        t = t_begin; t_end = t_end_; b_hint = first.b; i = 0; s = first;
        if (s.len == 0) s.kt0 = 0;
    }
    // Moves to the next tile; false past the end of the range.  Afterwards s.b / s.hk / s.rt are the tile's
    // unit, kt() its index within the unit's tiles and first() tells whether it opens a segment.
    __device__ __forceinline__ bool next(const int32_t *pre, const int32_t *nkt, int B, int n_rt) {
        if (i == s.len) {
            if (t >= t_end) return false;
            s = locate(pre, nkt, B, n_rt, t, t_end, b_hint);
            i = 0;
        }
        ++i;
        ++t;
        return true;
    }
    __device__ __forceinline__ int kt() const { return s.kt0 + i - 1; }
    __device__ __forceinline__ bool first() const { return i == 1; }
};

__device__ __forceinline__ int tiles_per_cta(int total, int grid) { return fast_div(total + grid - 1, grid); }

// Shares of a unit's nkt tiles among the k CTAs of a cluster.  A tile with tree keys costs about two context tiles
// (mask, P as a hi + lo pair, twice the P V products), so the shares are equal in cost rather than in tiles: with
// 8 context tiles and the tree tile over 4 CTAs, 3 + 3 + 2 + 1 instead of 3 + 3 + 3 + 0.
__device__ __forceinline__ void cluster_share(int nkt, int L, int k, int rank, int &lo, int &hi) {
    const int n_ctx = max(0, min(L / kTile, nkt));         // tiles of context keys only (a refused length: none)
    const int cost = n_ctx + 2 * (nkt - n_ctx), share = (cost + k - 1) >> (__ffs(k) - 1);     // k is a power of two
    auto tile_at = [&](int c) { return min(c <= n_ctx ? c : n_ctx + (c - n_ctx) / 2, nkt); };
    lo = tile_at(rank * share);
    hi = rank == k - 1 ? nkt : tile_at((rank + 1) * share);
}

// Tiles per CTA.  An even share cuts nearly every unit in two, and every cut costs a partial
// result in the workspace and a merge at the end: about as much as half a dozen tiles, whatever the
// unit's length.  So when all sequences are equally long and some whole multiple or whole fraction of a
// unit lies at most eight tiles above the even share, ranges of that length are used and cuts fall on unit
// boundaries (config 3: 33 tiles against 29, one unit per CTA on 128 of the SMs); beyond that the idle SMs
// cost more than the cuts (16 sequences of 32768 keys, one unit each: 257 tiles against 223, 566 -> 509 us
// with the even share).  Where several units share a KV head (n_rt > 1: row-tile pairs of grouped-query
// attention) aligned ranges also keep the CTAs of a head in step, so that its tiles cross DRAM once and
// reach the other CTAs from L2; there alignment is kept up to 5 % above the even share (4 x 32768 keys,
// 259 rows: 1.31 ms aligned, 1.42 ms even).
__device__ __forceinline__ int choose_per(int total, int grid, const int32_t *nkt, int B, int n_rt) {
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
        const int k = fast_div(n, even);              // largest count of parts whose length is >= even
        cand = fast_div(n + k - 1, k);
    } else {
        cand = fast_div(even + n - 1, n) * n;         // whole units
    }
    return (cand - even <= 8 || (n_rt > 1 && cand * 20 <= even * 21)) ? cand : even;
}

// Which share of the tile list a CTA takes.  Persistent form: place `my_pos` of `n_pos` ranges of `per` tiles
// (choose_per).  Cluster form (cluster_k > 1): the CTA's cost-equal share of the one unit its cluster (or set of
// clusters) works on.
struct RangeAsk {
    int n_pos, my_pos;
    int cluster_k, cl_rank;                     // cluster form: CTAs that share a unit (side by side in the grid), this CTA's place among them
    int cl_b, cl_unit;                          // ... their sequence, and which of its units
};
struct Range {
    int per, t_begin, t_end;
    Segment first;                 // the segment that holds tile t_begin (len == 0: the range is empty)
};
__device__ __forceinline__ Range read_range(const int32_t *w) {
    Range r;
    r.per = w[0]; r.t_begin = w[1]; r.t_end = w[2];
    r.first.b = w[3]; r.first.hk = w[4]; r.first.rt = w[5]; r.first.kt0 = w[6]; r.first.len = w[7]; r.first.nkt = w[8];
    return r;
}

// The CTA's range and first segment from the finished len / nkt / pre arrays: one thread's work (a chain of
// dependent integer instructions with half a dozen divisions; run by every thread it would also queue up at the
// conversion units), left in shared memory for everybody.
__device__ __forceinline__ void plan_range(const int32_t *s_len, const int32_t *s_nkt, const int32_t *s_pre, int B, int Hkv,
                                           int units_per_head, const RangeAsk &ask, int32_t *w) {
    const int total = s_pre[B];
    Range r;
    r.first.b = 0; r.first.hk = 0; r.first.rt = 0; r.first.kt0 = 0; r.first.len = 0; r.first.nkt = 0;
    if (ask.cluster_k > 1) {
        r.per = 0;
        // ask.cluster_k CTAs share the unit (one cluster, or several clusters side by side in the grid); ask.cl_rank
        // is this CTA's place among them
        const int cl_b = ask.cl_b, cl_unit = ask.cl_unit;
        const int nk = s_nkt[cl_b];
        int lo, hi;
        cluster_share(nk, s_len[cl_b], ask.cluster_k, ask.cl_rank, lo, hi);
        const int t0 = s_pre[cl_b] + cl_unit * nk;
        r.t_begin = t0 + lo;
        r.t_end = t0 + hi;
        r.first.b = cl_b;
        r.first.hk = units_per_head == 1 ? cl_unit : fast_div(cl_unit, units_per_head);
        r.first.rt = cl_unit - r.first.hk * units_per_head;
        r.first.kt0 = lo; r.first.len = hi - lo; r.first.nkt = nk;
    } else {
        r.per = choose_per(total, ask.n_pos, s_nkt, B, units_per_head);
        r.t_begin = ask.my_pos < ask.n_pos ? min(ask.my_pos * r.per, total) : total;
        r.t_end = min(r.t_begin + r.per, total);
        if (r.t_end > r.t_begin) {
            int hint = 0;
            r.first = locate(s_pre, s_nkt, B, units_per_head, r.t_begin, r.t_end, hint);
        }
    }
    w[0] = r.per; w[1] = r.t_begin; w[2] = r.t_end;
    w[3] = r.first.b; w[4] = r.first.hk; w[5] = r.first.rt; w[6] = r.first.kt0; w[7] = r.first.len; w[8] = r.first.nkt;
    w[9] = 0; w[10] = 0;           // (the producer's tally of what it asked for, read by the teardown of a CTA that gave up)
}

// Validates every sequence and fills len / nkt / pre.  Called by all threads of a block; ends with a barrier.  Every
// launch runs through this before its first fetch, so the common case (no malformed tree) takes two barriers: one
// that also tells whether any thread met a bad parent entry, and the one at the end.
template <int NT>
__device__ __forceinline__ void plan_sequences(const Params &p, int32_t *s_len, int32_t *s_nkt, int32_t *s_pre,
                                               bool write_status, bool errors_only, int units_per_head,
                                               const RangeAsk &ask, int32_t *s_plan) {
    // The lengths are asked for first and used last, so that their round trip to memory overlaps
    // the scan of the parent arrays (B <= kMaxB <= NT: one sequence per thread).
    const int my_b = threadIdx.x;
    const int my_L = my_b < p.B ? p.kv_len[my_b] : 0;
    const int entries = p.B * p.N;
    bool saw_bad = false;
    {
        // entry i = (sequence b, row c); a step of NT entries moves (b, c) by (db, dc) with one carry at most
        const int par0 = (int)threadIdx.x < entries ? p.parent[threadIdx.x] : -1;   // on its way while (b, c) are formed
        int b = fast_div((int)threadIdx.x, p.N), c = (int)threadIdx.x - b * p.N;
        const int db = fast_div(NT, p.N), dc = NT - db * p.N;
        for (int i = threadIdx.x; i < entries; i += NT) {
            const int par = i == (int)threadIdx.x ? par0 : p.parent[i];
            saw_bad = saw_bad || par < -1 || par >= c;
            b += db;
            c += dc;
            if (c >= p.N) { c -= p.N; ++b; }
        }
    }
    if (__syncthreads_or(saw_bad)) {
        // some tree is malformed: which sequences, through shared memory (0 = legal so far)
        for (int b = threadIdx.x; b < p.B; b += NT) s_nkt[b] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < entries; i += NT) {
            const int b = i / p.N, c = i - b * p.N;
            const int par = p.parent[i];
            if (par < -1 || par >= c) s_nkt[b] = -1;                 // benign race: all writers store -1
        }
        __syncthreads();
        saw_bad = my_b < p.B && s_nkt[my_b] < 0;                     // now: is this thread's own sequence malformed
        __syncthreads();
    } else {
        saw_bad = false;
    }
    int my_n = 0;                                                    // this thread's sequence: its tiles per unit
    if (my_b < p.B) {
        const int b = my_b, L = my_L;
        int code = HT_STATUS_OK;
        if (saw_bad) code = HT_STATUS_BAD_TREE;
        if (L < 0 || (long long)L + p.N > p.cap) code = HT_STATUS_BAD_LEN;
        s_len[b] = L;
        my_n = code == HT_STATUS_OK ? (L + p.N + kTile - 1) / kTile : 0;
        s_nkt[b] = my_n;
        // paged cache: the status words were zeroed ahead of the launch, and a fetch may already have
        // reported a bad page for this sequence, so only errors are written
        if (write_status && (code != HT_STATUS_OK || !errors_only)) p.status[b] = code;
    }
    if (p.B <= 32) {
        // prefix sums of the units' tiles by shuffles in the first warp
        if (threadIdx.x < 32) {
            const int mine = my_n * p.Hkv * units_per_head;
            int inc = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xFFFFFFFFu, inc, off);
                if ((int)threadIdx.x >= off) inc += o;
            }
            if (my_b < p.B) s_pre[my_b] = inc - mine;
            if (my_b == p.B - 1) s_pre[p.B] = inc;
            __syncwarp();
            if (threadIdx.x == 0) plan_range(s_len, s_nkt, s_pre, p.B, p.Hkv, units_per_head, ask, s_plan);
        }
    } else {
        __syncthreads();
        if (threadIdx.x == 0) {
            int acc = 0;
            for (int b = 0; b < p.B; ++b) {
                s_pre[b] = acc;
                acc += s_nkt[b] * p.Hkv * units_per_head;
            }
            s_pre[p.B] = acc;
            plan_range(s_len, s_nkt, s_pre, p.B, p.Hkv, units_per_head, ask, s_plan);
        }
    }
    __syncthreads();
}


// ---------------------------------------------------------------------------------------
// Paged cache, producer side (one thread).  The page ids of tile jt of this CTA's range are asked for
// kPgAhead tiles before the tile is fetched, by asynchronous 4-byte copies into a small ring in shared
// memory, one copy group per tile (empty past the end of the range), so that the lookup's round trip
// never stalls the fetches.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void pages_request(const Params &p, const PagedParams &pp, const int32_t *pre, const int32_t *nkt,
                                              int32_t (*pg)[kPgSub], int jt, TileCursor &cur, int lane, int n_rt_list) {
    if (cur.next(pre, nkt, p.B, n_rt_list)) {               // `cur` walks the range one tile per call: this is tile jt
        const int sub = pp.page_size >= kTile ? 1 : kTile >> pp.page_shift;
        const int first = (cur.kt() * kTile) >> pp.page_shift;
        if (lane < sub) {                                // lane x: page x of the tile
            if (first + lane < pp.max_pages)
                cp_async4(&pg[jt % kPgTiles][lane], pp.block_table + (size_t)cur.s.b * pp.max_pages + first + lane);
            else
                pg[jt % kPgTiles][lane] = -1;
        }
    }
    cp_async_commit();
}

// Fetch of one K or V tile (two 64-feature slabs) into a ring entry.  Contiguous cache (one thread): rows
// kt * 128 ... of (sequence b, head hk).
__device__ __forceinline__ void fetch_kv_tile(unsigned char *dst, const CUtensorMap *tm, void *bar, int b, int hk, int kt) {
    tma_load_4d(dst, tm, bar, 0, kt * kTile, hk, b);
    tma_load_4d(dst + kSlabBytes, tm, bar, 64, kt * kTile, hk, b);
}
// Paged cache (the whole producer warp): lane x fetches the rows that page x of the tile holds, whose id
// it asked for itself.  An id outside the pool is replaced by page 0 (no access outside the pool), and
// reported in the sequence's status word if any of the page's rows is a key of the sequence (rows past
// kv_len + N are masked and zeroed anyway).
// `later`: not null while the kernel ahead in the stream may still be running (it is the one that clears the status
// words): the report is left there and written out behind the wait.
__device__ __forceinline__ void fetch_kv_tile_paged(const Params &p, const PagedParams &pp, unsigned char *dst, const CUtensorMap *tm,
                                                    void *bar, int b, int hk, int kt, int keys, const int32_t *pg, int lane,
                                                    unsigned char *later) {
    const int ps = pp.page_size;
    const int sub = ps >= kTile ? 1 : kTile >> pp.page_shift;
    if (lane < sub) {
        const int row0 = ps >= kTile ? (kt * kTile) & (ps - 1) : 0;
        int page = pg[lane];
        if ((unsigned)page >= (unsigned)pp.n_pages) {
            if (kt * kTile + (lane << pp.page_shift) < keys) {
                if (later) later[b] = 1;
                else p.status[b] = HT_STATUS_BAD_PAGE;
            }
            page = 0;
        }
        const int off = (lane << pp.page_shift) * 128;      // rows of a slab are 128 bytes apart
        tma_load_4d(dst + off, tm, bar, 0, row0, hk, page);
        tma_load_4d(dst + kSlabBytes + off, tm, bar, 64, row0, hk, page);
    }
}

// Ring order of the one-tile kernel: the tensor pipe consumes K_0, K_1, V_0, K_2, V_1, ... (the scores of
// tile j+1 are issued before P V of tile j), so the tiles are fetched in that order and the ring is a FIFO:
// a slot is handed back in the order it was filled.  n = tiles of this CTA.
__device__ __forceinline__ int ring_entry_k(int j) { return j == 0 ? 0 : 2 * j - 1; }
__device__ __forceinline__ int ring_entry_v(int j, int n) { return j == n - 1 ? 2 * n - 1 : 2 * j + 2; }

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

// What rounding (lo, hi) to the packed 16-bit word w took away, rounded likewise:
// value = w + rest to about 2^-17 (bf16) / 2^-22 (fp16) of the value.
template <bool kBf16>
__device__ __forceinline__ uint32_t pack2_rest(float lo, float hi, uint32_t w) {
    float wl, wh;
    if (kBf16) {
        wl = __uint_as_float(w << 16);
        wh = __uint_as_float(w & 0xFFFF0000u);
    } else {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w));
        wl = f.x;
        wh = f.y;
    }
    return pack2<kBf16>(lo - wl, hi - wh);
}

// A unit that was cut between CTAs: which one, and which CTAs hold its parts.
struct CutUnit {
    int valid, unit, b, hk, rt, t0, c_lo, c_hi;      // c_lo .. c_hi: places in the list's partition that hold the parts
    int cta_mul, cta_add;                            // the CTA at place c is c * cta_mul + cta_add
};

// Merge of the parts of a cut unit by the 256 softmax threads of the CTA that delivered the
// last part.  Threads r and r + 128 own query row r, 64 features each; a warp reads 32
// consecutive rows of one feature group at a time (contiguous in the part's layout), and the
// loads of a part are independent of one another so that one round trip to L2 fetches it.
// `row_tile` is the 128-row tile the part holds; a workspace slot has `subs` parts, this is `sub`.
template <bool kBf16>
__device__ __noinline__ void merge_parts(const Params &p, const CutUnit &cu, int per, int tid256, int row_tile, int sub, int subs) {
    const int row = tid256 & 127, half = tid256 >> 7;
    const int node = row_tile * p.rows_per_tile_nodes + row / p.g;
    if (node >= p.N) return;
    const int head = cu.hk * p.g + row % p.g;
    float M = -INFINITY, l = 0.f;
    float acc[64];
#pragma unroll
    for (int x = 0; x < 64; ++x) acc[x] = 0.f;
#pragma unroll 1
    for (int c = cu.c_lo; c <= cu.c_hi; ++c) {
        const int slot = 2 * (c * cu.cta_mul + cu.cta_add) + ((max(cu.t0, c * per) == c * per) ? 0 : 1);
        const float *pslot = p.part + ((size_t)slot * subs + sub) * kSlotFloats;
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

// Reduction of a unit's parts inside a thread-block cluster, by the 256 softmax threads of each CTA.  Every CTA
// owns 128 / k of the 128 output features.  Behind a barrier of the whole cluster (all parts complete, no Q
// buffer or ring in use any more) each thread sends its row's feature groups straight from the accumulator
// into the owners' shared memory, `area` + kXchgRecvOffset (Q buffer and ring), through distributed shared
// memory; behind a second barrier each CTA merges the k slices it holds and writes its features of the result.
// No global memory, no atomics, no wait that could run out.  The other warps of every CTA of the cluster execute
// the same two barriers.
constexpr int kXchgRecvOffset = (kSlotFloats * 4 + 1023) / 1024 * 1024;   // bytes from the area's start
constexpr int kXchgBytes = kXchgRecvOffset + kRows * kD * 4 + 16 * 2 * kRows * 4;   // part + received slices + up to 16 senders' m, l
static_assert(kXchgBytes <= (1 + kStages) * kEntryBytes, "the exchange area is the Q buffer and the ring");

// Second half of the reduction: behind the barrier every part has arrived everywhere, and nobody writes into a
// peer's shared memory any more, so a CTA may leave as soon as it has merged what it holds.
//
// The merge of one row's received parts.  It runs once per CTA, so what counts is the length of its chain of
// dependent instructions, not their number: all loads are independent of one another (the k <= 16 parts unrolled
// with predicates), the parts' weights are formed once, and the row's features leave as 16-byte stores.
__device__ __forceinline__ float lds_f32(uint32_t a) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t a) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
    return v;
}
// Weights of the k parts of `row`, 1 / (sum of the weighted row sums) folded in.  recv_ml: [sender][m | l][row] floats.
constexpr int kMaxCluster = 16;        // CTAs per cluster at most (16 is beyond the portable size: asked for per kernel)
// raw != nullptr: the weights stay relative to the maximum, which is returned with the weighted sum (raw[0] = M,
// raw[1] = l): the cluster's result is then a part itself (two clusters share the unit).
template <int KP>                       // KP >= k: how far the loops over the parts are unrolled
__device__ __forceinline__ void merge_weights(uint32_t recv_ml, int k, int row, float (&f)[kMaxCluster], float *raw = nullptr) {
    float m[kMaxCluster], M = -INFINITY;
#pragma unroll
    for (int c = 0; c < KP; ++c) {
        m[c] = c < k ? lds_f32(recv_ml + (uint32_t)(c * 2 * kRows + row) * 4u) : -INFINITY;
        f[c] = c < k ? lds_f32(recv_ml + (uint32_t)(c * 2 * kRows + kRows + row) * 4u) : 0.f;     // the part's row sum, for now
    }
#pragma unroll
    for (int c = 0; c < KP; ++c) M = fmaxf(M, m[c]);
    float l = 0.f;
#pragma unroll
    for (int c = 0; c < KP; ++c) {
        const float w = m[c] == -INFINITY ? 0.f : ex2(m[c] - M);
        l = fmaf(w, f[c], l);
        f[c] = w;
    }
    if (raw) {
        raw[0] = M;
        raw[1] = l;
        return;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int c = 0; c < KP; ++c) f[c] *= inv;
}
// X groups of 4 features from group x0 on, summed over the parts with their weights: recv holds
// [sender][group in slice (cgps of them)][row] float4.
template <int X, int KP>
__device__ __forceinline__ void merge_sums(uint32_t recv, int k, int cgps, int row, int x0, const float (&f)[kMaxCluster], float4 (&o)[X]) {
#pragma unroll
    for (int x = 0; x < X; ++x) {
        o[x] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int c = 0; c < KP; ++c)
            if (c < k && f[c] != 0.f) {            // a part that saw nothing sent no features: what lies there is not data
                const float4 v = lds_f32x4(recv + (uint32_t)((c * cgps + x0 + x) * kRows + row) * 16u);
                o[x].x = fmaf(f[c], v.x, o[x].x); o[x].y = fmaf(f[c], v.y, o[x].y); o[x].z = fmaf(f[c], v.z, o[x].z); o[x].w = fmaf(f[c], v.w, o[x].w);
            }
    }
}
// ... rounded and stored: 8 X bytes at dst (16-byte aligned for even X, 8-byte aligned for X = 1).
template <bool kBf16, int X>
__device__ __forceinline__ void store_groups(const float4 (&o)[X], float scale, unsigned char *dst) {
    uint32_t w[2 * X];
#pragma unroll
    for (int x = 0; x < X; ++x) {
        w[2 * x] = pack2<kBf16>(o[x].x * scale, o[x].y * scale);
        w[2 * x + 1] = pack2<kBf16>(o[x].z * scale, o[x].w * scale);
    }
    if (X == 1) {
        *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1]);
        return;
    }
#pragma unroll
    for (int i = 0; i < X / 2; ++i)
        *reinterpret_cast<uint4 *>(dst + i * 16) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
}
template <bool kBf16, int X, int KP>
__device__ __forceinline__ void merge_groups(uint32_t recv, int k, int cgps, int row, int x0, const float (&f)[kMaxCluster], unsigned char *dst) {
    float4 o[X];
    merge_sums<X, KP>(recv, k, cgps, row, x0, f, o);
    store_groups<kBf16, X>(o, 1.f, dst);
}

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int *ptr) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// Several clusters share a unit (p.cluster_split = 2 or 4): behind its own exchange each CTA holds, for its slice of
// the features, a part of the unit over its cluster's share of the keys -- o (unnormalised sums), M, l per row.  The
// CTAs of the same rank in the sibling clusters hold the other parts.  Whichever comes last finishes the rows: from
// its registers if all the others' parts are in the workspace already, else after leaving its own there and finding,
// by the arrival counter, that it was last after all.  Nobody waits.  Called by all 256 softmax threads (three
// barriers at most); `flag` is a word of shared memory.  mine / theirs[]: [group in slice][row] float4, M and l behind
// kRows * kD floats, as a part of a cut unit.
// The thread's groups of 4 features are worked through in n_chunks chunks of XC groups, formed anew by `sums(chunk, o)`
// from what the CTA received wherever they are needed (few registers: this code runs once, behind a call).
template <bool kBf16, int XC, typename Sums>
__device__ __forceinline__ void finish_with_siblings(float *mine, const float *const (&theirs)[3], int n_others, unsigned int *ticket,
                                                     int *flag, Sums sums, int n_chunks, float M, float l, bool has_row, bool writes_ml,
                                                     int row, int xg0, unsigned char *dst, int tid256, volatile int *abort_flag) {
    if (tid256 == 0) *flag = *abort_flag ? 2 : (ld_acquire_gpu(ticket) == (unsigned)n_others ? 1 : 0);
    softmax_groups_sync();
    int state = *flag;
    if (state == 2) return;                                 // some wait of this CTA ran out: its part is not to be trusted
    float4 o[XC];
    if (state == 0) {
        if (has_row) {
            for (int ch = 0; ch < n_chunks; ++ch) {
                sums(ch, o);
#pragma unroll
                for (int x = 0; x < XC; ++x) reinterpret_cast<float4 *>(mine)[(xg0 + ch * XC + x) * kRows + row] = o[x];
            }
            if (writes_ml) {
                mine[kRows * kD + row] = M;
                mine[kRows * kD + kRows + row] = l;
            }
        }
        softmax_groups_sync();                              // the CTA's part is written, and everybody has read the flag
        if (tid256 == 0) {
            __threadfence();
            *flag = atomicAdd(ticket, 1u) == (unsigned)n_others ? 1 : 0;
        }
        softmax_groups_sync();
        state = *flag;
        if (state == 0) return;                             // not the last: a sibling finishes
    }
    __threadfence();
    if (has_row) {
        float m_o[3], l_o[3], Mn = M;
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            m_o[j] = j < n_others ? __ldcg(theirs[j] + kRows * kD + row) : -INFINITY;
            l_o[j] = j < n_others ? __ldcg(theirs[j] + kRows * kD + kRows + row) : 0.f;
            Mn = fmaxf(Mn, m_o[j]);
        }
        const float fa = M == -INFINITY ? 0.f : ex2(M - Mn);
        float fb[3], sum = l * fa;
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            fb[j] = m_o[j] == -INFINITY ? 0.f : ex2(m_o[j] - Mn);
            sum = fmaf(l_o[j], fb[j], sum);
        }
        const float inv = 1.f / sum;
        for (int ch = 0; ch < n_chunks; ++ch) {
            sums(ch, o);
#pragma unroll
            for (int x = 0; x < XC; ++x) {
                o[x].x *= fa; o[x].y *= fa; o[x].z *= fa; o[x].w *= fa;
#pragma unroll
                for (int j = 0; j < 3; ++j)
                    if (j < n_others && fb[j] != 0.f) {
                        const float4 v = __ldcg(reinterpret_cast<const float4 *>(theirs[j]) + (xg0 + ch * XC + x) * kRows + row);
                        o[x].x = fmaf(fb[j], v.x, o[x].x); o[x].y = fmaf(fb[j], v.y, o[x].y);
                        o[x].z = fmaf(fb[j], v.z, o[x].z); o[x].w = fmaf(fb[j], v.w, o[x].w);
                    }
            }
            store_groups<kBf16, XC>(o, inv, dst + ch * XC * 8);
        }
    }
    if (tid256 == 0) *ticket = 0u;                          // zero again for the next call on this workspace
}
// The workspace slots of the CTAs of this CTA's rank in the sibling clusters (sub: the stream's slot of a tile pair).
__device__ __forceinline__ void sibling_slots(const Params &p, int slots_per_cta, int sub, const float *(&theirs)[3]) {
    const int k = p.cluster_k, S = p.cluster_split;
    const int cluster = (int)blockIdx.x / k, rank = (int)blockIdx.x - cluster * k, first = cluster / S * S;
    int n = 0;
    for (int j = 0; j < S; ++j)
        if (first + j != cluster) theirs[n++] = p.part + ((size_t)(2 * ((first + j) * k + rank)) * slots_per_cta + sub) * kSlotFloats;
    for (; n < 3; ++n) theirs[n] = nullptr;
}

// One-tile kernel: received slices lie at area + kXchgRecvOffset as [sender][group in slice][row] float4, followed by
// [sender][m | l][row]; thread (row, half) merges half of the CTA's slice of the row's features.
template <bool kBf16>
__device__ __noinline__ void cluster_merge(const Params &p, unsigned char *area, int rank, int b, int hk, int row_tile,
                                           bool valid, int tid256, volatile int *abort_flag) {
    int *const flag = &reinterpret_cast<Smem *>(area)->direct;      // (the area is the start of the CTA's shared memory)
    const int k = p.cluster_k;
    const int cgps = 32 / k;                      // groups of 4 features per slice: 16, 8, 4 or 2
    cluster_sync_all();
    const int row = tid256 & 127, half = tid256 >> 7;
    const int node = row_tile * p.rows_per_tile_nodes + row / p.g;
    const uint32_t recv = smem_u32(area) + kXchgRecvOffset, recv_ml = recv + kRows * kD * 4;
    if (p.cluster_split > 1) {
        // several clusters (of eight, or of four) share the unit: this one's result is a part
        const bool has_row = valid && node < p.N;
        float f[kMaxCluster], raw[2] = {-INFINITY, 0.f};
        const int x0 = half * (cgps / 2);
        if (has_row) {
            if (k == 8) merge_weights<8>(recv_ml, k, row, f, raw);
            else merge_weights<4>(recv_ml, k, row, f, raw);
        }
        const int unit = ((int)blockIdx.x / k) / p.cluster_split;
        const int head = hk * p.g + row % p.g;
        unsigned char *dst = static_cast<unsigned char *>(p.out) +
                             ((((size_t)b * p.N + node) * p.Hq + head) * kD + (rank * cgps + x0) * 4) * 2;
        const float *theirs[3];
        sibling_slots(p, 1, 0, theirs);
        float *mine = p.part + (size_t)(2 * (int)blockIdx.x) * kSlotFloats;
        auto sums = [&](int ch, float4 (&o)[2]) {                // two groups at a time: clusters of eight have two per thread, of four four
            if (k == 8) merge_sums<2, 8>(recv, k, cgps, row, x0 + 2 * ch, f, o);
            else merge_sums<2, 4>(recv, k, cgps, row, x0 + 2 * ch, f, o);
        };
        finish_with_siblings<kBf16, 2>(mine, theirs, p.cluster_split - 1, p.tickets + unit * k + rank, flag, sums, k == 8 ? 1 : 2,
                                       raw[0], raw[1], has_row, half == 0, row, x0, dst, tid256, abort_flag);
        return;
    }
    if (!valid || node >= p.N || *abort_flag) return;
    float f[kMaxCluster];
    if (k <= 4) merge_weights<4>(recv_ml, k, row, f);
    else if (k == 8) merge_weights<8>(recv_ml, k, row, f);
    else merge_weights<16>(recv_ml, k, row, f);
    const int head = hk * p.g + row % p.g;
    const int x0 = half * (cgps / 2);
    unsigned char *dst = static_cast<unsigned char *>(p.out) +
                         ((((size_t)b * p.N + node) * p.Hq + head) * kD + (rank * cgps + x0) * 4) * 2;
    if (k == 2) merge_groups<kBf16, 8, 2>(recv, k, cgps, row, x0, f, dst);
    else if (k == 4) merge_groups<kBf16, 4, 4>(recv, k, cgps, row, x0, f, dst);
    else if (k == 8) merge_groups<kBf16, 2, 8>(recv, k, cgps, row, x0, f, dst);
    else merge_groups<kBf16, 1, 16>(recv, k, cgps, row, x0, f, dst);
}

}  // namespace tc
}  // namespace ht
