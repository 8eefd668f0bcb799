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
//                        merges all parts -- nobody waits on another CTA.  The ticket words
//                        reset themselves (a caller that keeps its workspace needs no kernel
//                        to clear them: HT_ATTN_WORKSPACE_CLEAN).  Few units: clusters, with
//                        the parts reduced through distributed shared memory.
//   launch             : serialized programmatically behind the kernel ahead in the stream.
//                        With the caller's word that lengths, trees and context rows were
//                        final before that kernel began (HT_ATTN_CONTEXT_FINAL) the plan and
//                        the first context tiles do not wait for it; each role waits where it
//                        first touches what that kernel may still write or read.
//
// Every wait on an mbarrier is bounded; when one runs out the CTA raises an abort flag,
// reports HT_STATUS_TIMEOUT, runs to the end of its control flow without further waiting,
// drains its own copies, frees its TMEM and returns.
#include <stddef.h>

#include "attn_tc.cuh"

namespace ht {
namespace tc {

// Second softmax pass over the 128 scores of this thread's row: exponentials, row sum (into acc2), P to TMEM
// as packed 16-bit pairs over scores already consumed.  On entry chunk 0 (32 scores) is on its way into xa.
// kHiLo = false (tiles of context keys): P chunk c lands in columns [16 c, 16 c + 16).
// kHiLo = true (tiles with tree keys: a row may see a handful of keys only, and then the rounding of its
// weights to 16 bits is no longer averaged away): P goes to the tensor pipe as a pair hi + lo of 16-bit
// values, P V is issued for both; chunk c's hi lands in columns [32 c, 32 c + 16) and its lo = P - hi in
// [32 c + 16, 32 c + 32), i.e. every chunk's results take the chunk's own columns.
template <bool kBf16, bool kHiLo>
__device__ __forceinline__ void softmax_pass2(uint32_t s_addr, float *xa, float *xb, unsigned long long scale2,
                                              unsigned long long nbase2, unsigned long long &acc2) {
    constexpr int kStep = kHiLo ? 32 : 16;             // columns a chunk's results take
    // 32 scores -> 16 packed pairs at column `col`; with kHiLo eight pairs at a time, each with what its rounding
    // took away (few registers: these tiles share the hot loop's allocation)
    auto chunk = [&](const float *x, uint32_t col) {
        if (!kHiLo) {
            uint32_t r[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                float p0, p1;
                unpack_f32x2(fma_f32x2(pack_f32x2(x[2 * c], x[2 * c + 1]), scale2, nbase2), p0, p1);
                p0 = ex2(p0);
                p1 = ex2(p1);
                acc2 = add_f32x2(acc2, pack_f32x2(p0, p1));
                r[c] = pack2<kBf16>(p0, p1);
            }
            tmem_st16(col, r);
        } else {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[8], r_lo[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float p0, p1;
                    unpack_f32x2(fma_f32x2(pack_f32x2(x[16 * half + 2 * c], x[16 * half + 2 * c + 1]), scale2, nbase2), p0, p1);
                    p0 = ex2(p0);
                    p1 = ex2(p1);
                    acc2 = add_f32x2(acc2, pack_f32x2(p0, p1));
                    r[c] = pack2<kBf16>(p0, p1);
                    r_lo[c] = pack2_rest<kBf16>(p0, p1, r[c]);
                }
                tmem_st8(col + half * 8, r);
                tmem_st8(col + 16 + half * 8, r_lo);
            }
        }
    };
#pragma unroll 1
    for (int h = 0; h < 2; ++h) {
        tmem_ld_wait();
        tmem_ld32(s_addr + (2 * h + 1) * 32, xb);
        chunk(xa, s_addr + (2 * h) * kStep);
        tmem_ld_wait();
        if (h == 0) tmem_ld32(s_addr + 2 * 32, xa);
        chunk(xb, s_addr + (2 * h + 1) * kStep);
    }
}

// The Q tile of a segment: the N x g rows of the KV head's query heads, two 64-feature slabs.
__device__ __forceinline__ void fetch_q_tile(Smem &sm, const CUtensorMap &tm_q, const Params &p, int hk, int rt, int b) {
    mbar_expect_tx(&sm.q_full, kEntryBytes);
    tma_load_4d(sm.q, &tm_q, &sm.q_full, 0, hk * p.g, rt * p.rows_per_tile_nodes, b);
    tma_load_4d(sm.q + kSlabBytes, &tm_q, &sm.q_full, 64, hk * p.g, rt * p.rows_per_tile_nodes, b);
}

// kPaged: the cache is a pool of pages (separate instantiations, so that the contiguous kernels carry none of that code).
// kClustered: launched as clusters (p.cluster_k > 1); a template parameter so that the persistent form carries no cluster code.
template <bool kBf16, bool kPaged, bool kClustered>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const Params p, const PagedParams pp) {
    extern __shared__ unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sm.abort;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&sm.kv_full[i], 1); mbar_init(&sm.kv_empty[i], 1); }
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_empty, 1);
        mbar_init(&sm.mma_drain, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&sm.s_full[i], 1); mbar_init(&sm.p_ready[i], 128); mbar_init(&sm.o_done[i], 1); }
        sm.abort = 0;
        sm.wait_kcycles = p.wait_kcycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x == 32) {                 // descriptors on their way while the CTA sets itself up
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // The launch is serialized programmatically behind the kernel before it in the stream: the CTA has set itself
    // up while that kernel was still finishing, and everything it may have written is read from here on.
    // `early` (the caller vouches that lengths, trees and the cache rows below the lengths were final before that
    // kernel began): the plan is made and the first context tiles are fetched right away, and each role waits for
    // the kernel ahead where it first touches what that kernel may have written or may still read -- the producer
    // before the Q tile and before the first tile with tree rows, the softmax threads before their first scores
    // (status words, workspace and `out` are written behind that), the issuer before its first product.
    const bool early = p.early != 0;
    if (kPaged && early)
        for (int b = threadIdx.x; b < p.B; b += blockDim.x) sm.bad_page[b] = 0;     // (the plan's barriers come before any fetch)
    if (!early) wait_for_kernel_ahead();
    // Persistent form: CTA i takes the i-th range of the tile list.  Cluster form: one cluster per (sequence, KV head);
    // its CTAs take cost-equal shares of the unit's tiles.  (No cluster barrier here: the first remote access comes
    // after the one all threads pass ahead of the exchange.)  One thread works the range and its first segment out.
    constexpr bool clustered = kClustered;
    uint32_t c_rank = 0;
    RangeAsk ask;
    ask.n_pos = p.grid; ask.my_pos = (int)blockIdx.x;
    ask.cluster_k = 0; ask.cl_rank = 0; ask.cl_b = 0; ask.cl_unit = 0;
    if (clustered) {
        // (two clusters on a unit, p.cluster_split == 2: their CTAs share the unit's tiles like one cluster of twice the size)
        c_rank = cluster_ctarank();
        ask.cluster_k = p.cluster_k * p.cluster_split;                 // a power of two
        ask.cl_rank = (int)blockIdx.x & (ask.cluster_k - 1);
        const int unit = (int)blockIdx.x >> (__ffs(ask.cluster_k) - 1);
        ask.cl_b = unit / p.Hkv;
        ask.cl_unit = unit - ask.cl_b * p.Hkv;
    }
    tc_fence_before();                              // (the tensor memory's base address crosses the plan's last barrier)
    plan_sequences<kThreads>(p, sm.len, sm.nkt, sm.pre, blockIdx.x == 0 && !early, kPaged, 1, ask, sm.plan);   // one unit per KV head in this kernel
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const Range range = read_range(sm.plan);
    const int per = range.per, t_begin = range.t_begin, t_end = range.t_end;
    const Segment first = range.first;

    if (warp == 8) {
        // ------------------------------- TMA producer -------------------------------
        // Contiguous cache: one thread.  Paged cache: the whole warp walks the same loop (identical state in
        // every lane), so that the pages of a tile are looked up and fetched by one lane each, in one
        // instruction, instead of one after the other; lane 0 alone arms the barriers and fetches Q.
        if (kPaged || lane == 0) {
            int ring_i = 0, seg_i = 0;
            const int n = t_end - t_begin;
            bool waited = !early;                  // early: the range's first Q tile is fetched by the issuing thread, behind its wait
            auto release = [&]() {
                if (!waited) {
                    wait_for_kernel_ahead();
                    waited = true;
                    if (kPaged) {                       // bad page entries met so far (the whole warp is here)
                        __syncwarp();
                        for (int b = lane; b < p.B; b += 32)
                            if (sm.bad_page[b]) p.status[b] = HT_STATUS_BAD_PAGE;
                    }
                }
            };
            TileCursor cur_k, cur_v, cur_p;          // the K and V streams of the ring order, and the page-id lookahead
            cur_k.init(t_begin, t_end, first);
            cur_v.init(t_begin, t_end, first);
            cur_p.init(t_begin, t_end, first);
            if (kPaged)
                for (int jt = 0; jt < kPgAhead; ++jt) pages_request(p, pp, sm.pre, sm.nkt, sm.pg, jt, cur_p, lane, 1);
            for (int e = 0; e < 2 * n; ++e) {
                if (kPaged ? __any_sync(0xFFFFFFFFu, *abort_flag != 0) : (*abort_flag != 0)) break;
                // entry e of the consumption order: K_0, K_1, V_0, K_2, V_1, ..., V_{n-1}
                const bool is_v = e == 2 * n - 1 || (e != 0 && (e & 1) == 0);
                const int j = e == 0 ? 0 : (e == 2 * n - 1 ? n - 1 : (is_v ? (e - 2) / 2 : (e + 1) / 2));
                if (is_v) cur_v.next(sm.pre, sm.nkt, p.B, 1);   // tile j of its stream
                else cur_k.next(sm.pre, sm.nkt, p.B, 1);
                struct { int b, hk, rt; } s;
                s.b = is_v ? cur_v.s.b : cur_k.s.b;
                s.hk = is_v ? cur_v.s.hk : cur_k.s.hk;
                s.rt = is_v ? cur_v.s.rt : cur_k.s.rt;
                const int kt = is_v ? cur_v.kt() : cur_k.kt();
                if (!is_v && cur_k.first()) {
                    // first tile of a segment: its Q tile, once the previous segment's scores are done with Q
                    if (seg_i > 0) release();
                    bool ok = seg_i == 0 || mbar_wait_quick(smem_u32(&sm.q_empty), (seg_i - 1) & 1, abort_flag);
                    if (kPaged) ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    if (lane == 0 && !(early && seg_i == 0)) fetch_q_tile(sm, tm_q, p, s.hk, s.rt, s.b);
                    ++seg_i;
                }
                // early: context tiles only, and no more of them than the ring holds, ahead of the wait
                if (!waited && ((kt + 1) * kTile > sm.len[s.b] || ring_i >= kStages)) release();
                const int slot = ring_i % kStages, use = ring_i / kStages;
                {
                    bool ok = use == 0 || mbar_wait_quick(smem_u32(&sm.kv_empty[slot]), (use - 1) & 1, abort_flag);
                    if (kPaged) ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                }
                const CUtensorMap *tm = is_v ? &tm_v : &tm_k;
                if (kPaged && !is_v) {
                    // the ids of tile j were asked for kPgAhead tiles ago; ask for those of tile j + kPgAhead
                    pages_request(p, pp, sm.pre, sm.nkt, sm.pg, j + kPgAhead, cur_p, lane, 1);
                    cp_async_wait<kPgAhead>();
                }
                if (lane == 0) mbar_expect_tx(&sm.kv_full[slot], kEntryBytes);
                if (kPaged) {
                    __syncwarp();                                     // the barrier is armed before any lane's copy can complete
                    fetch_kv_tile_paged(p, pp, sm.ring[slot], tm, &sm.kv_full[slot], s.b, s.hk, kt, sm.len[s.b] + p.N,
                                        sm.pg[j % kPgTiles], lane, waited ? nullptr : sm.bad_page);
                } else {
                    fetch_kv_tile(sm.ring[slot], tm, &sm.kv_full[slot], s.b, s.hk, kt);
                }
                ++ring_i;
            }
            if (kPaged) {
                cp_async_wait<0>();
                __syncwarp();
            }
            release();
            if (lane == 0) {
                // how many ring entries and Q tiles were asked for: should the CTA give up, the teardown waits for the
                // last of them (early: the first Q tile was fetched by the issuing thread, whatever else happened)
                sm.plan[9] = ring_i;
                sm.plan[10] = early && n > 0 && seg_i == 0 ? 1 : seg_i;
            }
        }
        if (clustered) {                               // the two barriers of the exchange (whole warp)
            cluster_sync_all();
            cluster_sync_all();
        }
    } else if (warp == 9) {
        // ------------------------------- MMA issuer -------------------------------
        // One thread: a chain of dependent instructions that shares its scheduler with two softmax warps, so the
        // instructions per tile are kept few: ring slots and phases are counted (no division), barrier addresses
        // and descriptor words are formed once, each product is one instruction sequence, and the abort flag is
        // looked at only when a wait has to spin.
        if (lane == 0) {
            if (early) {
                // q is the kernel ahead's to write: the range's first Q tile is fetched here, behind the wait, while the
                // producer is busy with the first context tiles
                wait_for_kernel_ahead();
                if (t_end > t_begin) fetch_q_tile(sm, tm_q, p, first.hk, first.rt, first.b);
            }
            const uint32_t idesc_qk = instr_desc(kBf16, 0), idesc_pv = instr_desc(kBf16, 1);
            const uint32_t hi_k = desc_hi(1, 1024 >> 4), hi_v = desc_hi(kSlabBytes >> 4, 1024 >> 4);
            const uint32_t q_lo = desc_lo_with_lbo(smem_u32(sm.q), 1);
            const uint32_t ring_k_lo = desc_lo_with_lbo(smem_u32(sm.ring[0]), 1);            // slot x: + x * (kEntryBytes / 16)
            const uint32_t ring_v_lo = desc_lo_with_lbo(smem_u32(sm.ring[0]), kSlabBytes >> 4);
            const uint32_t bar_kv_full = smem_u32(&sm.kv_full[0]), bar_kv_empty = smem_u32(&sm.kv_empty[0]);
            const uint32_t bar_s_full = smem_u32(&sm.s_full[0]), bar_p_ready = smem_u32(&sm.p_ready[0]), bar_o_done = smem_u32(&sm.o_done[0]);
            const int n = t_end - t_begin;
            int b_hint = 0, j = 0, seg_i = 0;
            int prev_first = 0;          // is tile j-1 the first of its stream within its segment?
            bool prev_tree = false;      // does tile j-1 hold tree keys?  Its P is then a hi + lo pair (see the softmax)
            bool alive = !*abort_flag;   // false once a wait of this thread has given up: no further waits or products
            // ring entries in consumption order K_0, K_1, V_0, K_2, V_1, ...: slot and phase of the next K and V entry
            uint32_t k_slot = 0, k_ph = 0, v_slot = 2 % kStages, v_ph = 0;
            auto advance = [](uint32_t &slot, uint32_t &ph, uint32_t by) {
                slot += by;
                if (slot >= (uint32_t)kStages) { slot -= kStages; ph ^= 1u; }
            };
            auto issue_pv = [&](int jj, int first, bool tree) {
                const uint32_t s = jj & 1;
                alive = alive && mbar_wait_quick(bar_p_ready + s * 8, (jj >> 1) & 1, abort_flag);
                alive = alive && mbar_wait_quick(bar_kv_full + v_slot * 8, v_ph, abort_flag);
                tc_fence_after();
                if (alive) {
                    // V tile as B operand, MN-major: 64 features contiguous (one swizzled 128-byte line per key), the
                    // second 64-feature slab one slab further (LBO), groups of 8 keys 1 KiB apart (SBO); 16 keys per
                    // instruction = 2 KiB.
                    const uint32_t v_lo = ring_v_lo + v_slot * (kEntryBytes >> 4);
                    if (!tree) mma_block_pv128(tmem + 256 + s * 128, tmem + s * 128, v_lo, hi_v, idesc_pv, first ? 0u : 1u);
                    else mma_block_pv128_hilo(tmem + 256 + s * 128, tmem + s * 128, v_lo, hi_v, idesc_pv, first ? 0u : 1u);
                }
                tc_commit_addr(bar_kv_empty + v_slot * 8);
                tc_commit_addr(bar_o_done + s * 8);
                advance(v_slot, v_ph, jj + 2 == n ? 1 : 2);                  // V entries: 2, 4, ..., 2n - 2, then 2n - 1
            };
            if (n == 1) v_slot = 1;                                          // a single tile: K_0, V_0
            for (int t = t_begin; t < t_end;) {
                const Segment sg = t == t_begin ? first : locate(sm.pre, sm.nkt, p.B, 1, t, t_end, b_hint);
                const int L = sm.len[sg.b];
                alive = alive && mbar_wait_quick(smem_u32(&sm.q_full), seg_i & 1, abort_flag);
                for (int i = 0; i < sg.len; ++i) {
                    const uint32_t s = j & 1;
                    alive = alive && mbar_wait_quick(bar_kv_full + k_slot * 8, k_ph, abort_flag);
                    tc_fence_after();
                    // K-major operands: 16 features = 32 bytes inside the 128-byte swizzled line; the second
                    // 64-feature slab lies one slab further.
                    if (alive) mma_block_qk(tmem + s * 128, q_lo, ring_k_lo + k_slot * (kEntryBytes >> 4), hi_k, idesc_qk);
                    tc_commit_addr(bar_s_full + s * 8);
                    tc_commit_addr(bar_kv_empty + k_slot * 8);
                    if (i == sg.len - 1) tc_commit(&sm.q_empty);
                    advance(k_slot, k_ph, j == 0 ? 1 : 2);                    // K entries: 0, 1, 3, 5, ...
                    if (j > 0) issue_pv(j - 1, prev_first, prev_tree);
                    prev_first = i < 2;
                    prev_tree = (sg.kt0 + i + 1) * kTile > L;
                    ++j;
                }
                t += sg.len;
                ++seg_i;
            }
            if (j > 0) issue_pv(j - 1, prev_first, prev_tree);
            // No tensor-core operation of this CTA may be in flight when its TMEM is freed.
            tc_commit(&sm.mma_drain);
            mbar_wait(&sm.mma_drain, 0, abort_flag, false);
        }
        if (clustered) {                               // the two barriers of the exchange (whole warp)
            cluster_sync_all();
            cluster_sync_all();
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
        bool waited = !early;
        // early: the status words (all of them from the first CTA) go out behind the wait
        auto release = [&]() {
            if (!waited) {
                wait_for_kernel_ahead();
                waited = true;
                if (blockIdx.x == 0 && tid256 < p.B) {
                    const int L = sm.len[tid256];
                    const int code = (L < 0 || (long long)L + p.N > p.cap) ? HT_STATUS_BAD_LEN
                                     : (sm.nkt[tid256] == 0 ? HT_STATUS_BAD_TREE : HT_STATUS_OK);
                    // (paged cache: the words were cleared ahead of the launch and a fetch may have reported a bad page)
                    if (!kPaged || code != HT_STATUS_OK) p.status[tid256] = code;
                }
            }
        };
        for (int t = t_begin; t < t_end;) {
            const Segment sg = t == t_begin ? first : locate(sm.pre, sm.nkt, p.B, 1, t, t_end, b_hint);
            const int L = sm.len[sg.b];
            // --- ancestor masks of this tile's rows (kept while sequence and row tile stay the same) ---
            const int node = sg.rt * p.rows_per_tile_nodes + row / p.g;
            const bool real = node < p.N;
            // a warp none of whose 32 rows is a query row keeps step with the barriers but computes nothing
            const bool warp_real = sg.rt * p.rows_per_tile_nodes + (row & ~31) / p.g < p.N;
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
            release();

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
                cu.cta_mul = 1; cu.cta_add = 0;
            }

            float m_ref = -INFINITY, l_sum = 0.f;
#pragma unroll 1
            for (int i = 0; i < sg.len; ++i) {
                const int jj = J + i;
                if ((jj & 1) != s) continue;
                const int kt = sg.kt0 + i;
                if (!complete && !clustered && tid256 == 0) {
                    delivered_old = delivered;
                    delivered = ld_relaxed_gpu(&p.tickets[cut[cut_k].unit]);
                }
                mbar_wait(&sm.s_full[s], (jj >> 1) & 1, abort_flag);
                tc_fence_after();
                const uint32_t s_addr = tmem + lane_base + s * 128;
                const int tile_lo = kt * kTile;
                float *const xa = xa_e, *const xb = xb_e;
                if (warp_real) {
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
                if (tile_lo + kTile > L) softmax_pass2<kBf16, true>(s_addr, xa, xb, scale2, nbase2, acc2);
                else softmax_pass2<kBf16, false>(s_addr, xa, xb, scale2, nbase2, acc2);
                {
                    float a0, a1;
                    unpack_f32x2(acc2, a0, a1);
                    l_sum += a0 + a1;
                }
                tmem_st_wait();
                }
                // --- last tile of the unit: rows of V past the tree are not data; make them zero ---
                if (kt == sg.nkt - 1) {
                    const int valid = L + p.N - tile_lo;
                    if (valid < kTile) {
                        const int e = ring_entry_v(jj, t_end - t_begin), slot = e % kStages;
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
                mbar_arrive(&sm.p_ready[s]);
            }
            // --- segment epilogue: merge the two streams, write the result or a partial.  The streams' maxima and sums
            // are exchanged and the weights formed while the last products are still running; the accumulators are read
            // behind the wait for both streams' last product (every thread reads both). ---
            sm.ml[s][row][0] = m_ref;
            sm.ml[s][row][1] = l_sum;
            // With one other part and that part already in the workspace, this CTA finishes the unit
            // from its registers; otherwise it leaves its own part there.
            if (tid256 == 0) {
                sm.direct = !clustered && !complete && cut[cut_k].c_hi - cut[cut_k].c_lo == 1 && delivered_old == 1u;
                // nobody touches the unit's counter any more: it is left at zero for the next call on this workspace
                if (sm.direct) p.tickets[cut[cut_k].unit] = 0u;
            }
            softmax_groups_sync();
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
            // a part goes to the workspace -- or, in a cluster, slice by slice to the peers' (by now idle) Q buffers and rings
            float *pslot = clustered ? nullptr : p.part + (size_t)(2 * (int)blockIdx.x + cut_k) * kSlotFloats;
            const int xk_sh = clustered ? 5 - __ffs(p.cluster_k) + 1 : 0;        // log2 of the 4-feature groups per peer's slice
            const uint32_t xrecv = smem_u32(&sm.q[0]) + kXchgRecvOffset;           // same offset in every CTA of the cluster
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
                const float inv = (complete && !clustered) ? 1.f / l_tot : 1.f;
                g0 = f0 * inv;
                g1 = f1 * inv;
            }
            {
                const int last_any = J + sg.len - 1;                       // the segment's last tile; x's last: same parity
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const int lx = ((last_any & 1) == x) ? last_any : last_any - 1;
                    if (lx >= J) mbar_wait(&sm.o_done[x], (lx >> 1) & 1, abort_flag);
                }
                tc_fence_after();
            }
            // In a cluster the part goes straight from the accumulators into the peers' shared memory (each
            // peer owns a slice of the features), so the barrier that says "every CTA of the cluster is done with
            // its Q buffer and ring" comes first: every thread of every CTA takes part in it, the producer and
            // issuer warps once their work is done.
            if (clustered) cluster_sync_all();
            const bool final = (complete && !clustered) || direct;
#pragma unroll 1
            for (int c2 = 0; c2 < (warp_real ? 2 : 0); ++c2) {
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
                } else if (clustered) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {    // feature group cg belongs to peer cg >> xk_sh, as that slice's group x
                        const int cg = col0 / 4 + c, x = cg & ((1 << xk_sh) - 1);
                        st_peer_f4(map_to_peer(xrecv + (uint32_t)((((int)c_rank << xk_sh) + x) * kRows + row) * 16u, (uint32_t)(cg >> xk_sh)),
                                   make_float4(xa_e[4 * c], xa_e[4 * c + 1], xa_e[4 * c + 2], xa_e[4 * c + 3]));
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c)      // 32 consecutive rows of one feature group: 512 contiguous bytes per warp
                        reinterpret_cast<float4 *>(pslot)[(col0 / 4 + c) * kRows + row] = make_float4(xa_e[4 * c], xa_e[4 * c + 1], xa_e[4 * c + 2], xa_e[4 * c + 3]);
                }
            }
            if (clustered) {
                // every peer gets this part's maximum (from stream 0's threads) and sum (from stream 1's)
                if (real)
                    for (int c = 0; c < p.cluster_k; ++c)
                        st_peer_f1(map_to_peer(xrecv + (uint32_t)(kRows * kD + ((int)c_rank * 2 + s) * kRows + row) * 4u, (uint32_t)c), s == 0 ? M : l_tot);
            } else if (!final && s == 0 && real) {
                pslot[kRows * kD + row] = M;
                pslot[kRows * kD + kRows + row] = l_tot;
            }
            tc_fence_before();
            softmax_groups_sync();                     // both accumulators are free for the next segment
            if (!final && !clustered) {
                // This CTA's part is in the workspace: take the unit's ticket.  One thread orders the
                // CTA's stores (the barrier above collected them) and draws; the answer is looked at
                // after the CTA's last segment.
                cut[cut_k].valid = 1;
                if (tid256 == 0) {
                    __threadfence();
                    ticket[cut_k] = atomicAdd(&p.tickets[cut[cut_k].unit], 1u);
                }
            }
            J += sg.len;
            t += sg.len;
        }
        release();
        if (clustered) {
            if (t_end <= t_begin) {                    // an empty share still delivers a part: nothing seen
                cluster_sync_all();
                const uint32_t xrecv = smem_u32(&sm.q[0]) + kXchgRecvOffset;
                for (int c = 0; c < p.cluster_k; ++c)
                    st_peer_f1(map_to_peer(xrecv + (uint32_t)(kRows * kD + ((int)c_rank * 2 + s) * kRows + row) * 4u, (uint32_t)c), s == 0 ? -INFINITY : 0.f);
            }
            const int unit = (int)blockIdx.x / (p.cluster_k * p.cluster_split), b = unit / p.Hkv;
            cluster_merge<kBf16>(p, &sm.q[0], (int)c_rank, b, unit - b * p.Hkv, 0, sm.nkt[b] > 0, tid256, abort_flag);
        }
        // --- cut units: the CTA that delivers the last part of a unit merges all parts; nobody waits ---
        if (cut[0].valid || cut[1].valid) {
            if (tid256 == 0)
                for (int k = 0; k < 2; ++k) {
                    sm.merge_here[k] = cut[k].valid && ticket[k] == (unsigned)(cut[k].c_hi - cut[k].c_lo);
                    if (sm.merge_here[k]) p.tickets[cut[k].unit] = 0u;      // all parts have arrived: zero again for the next call
                }
            softmax_groups_sync();
            for (int k = 0; k < 2; ++k)
                if (sm.merge_here[k]) {
                    __threadfence();
                    merge_parts<kBf16>(p, cut[k], per, tid256, cut[k].rt, 0, 1);
                }
        }
        }

    // ------------------------------- teardown -------------------------------
    tc_fence_before();
    __syncthreads();
    // (cluster mode: the exchange's second barrier already guarantees that no peer writes here any more)
    if (sm.abort && threadIdx.x == 0) {
        for (int b = 0; b < p.B; ++b)
            if (sm.nkt[b] > 0) p.status[b] = HT_STATUS_TIMEOUT;
    }
    if (sm.abort && threadIdx.x == 8 * 32) {
        // Some wait of this CTA ran out, wherever: every copy it asked for must have landed before it exits (this
        // warp leaves last: it frees the tensor memory below).  Wait, with the full bound, for the latest armed
        // phase of each ring slot and of the Q buffer.
        const int ring_i = sm.plan[9], q_fetches = sm.plan[10];
        for (int e = max(0, ring_i - kStages); e < ring_i; ++e)
            mbar_wait(&sm.kv_full[e % kStages], (e / kStages) & 1, abort_flag, false);
        if (q_fetches > 0) mbar_wait(&sm.q_full, (q_fetches - 1) & 1, abort_flag, false);
    }
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// What must be zero when the attention kernel starts: the units' arrival counters (and, for a paged cache, the
// status words).  A kernel rather than a memset node so that the launches can be chained by programmatic stream
// serialization: this one is in place, waiting, before the previous kernel of the stream has finished, and the
// attention kernel behind it has its CTAs set up by the time this one is done.
__global__ void attn_prepare_kernel(unsigned int *tickets, int n_tickets, int32_t *status, int n_status) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int stride = gridDim.x * blockDim.x, first = blockIdx.x * blockDim.x + threadIdx.x;
    for (int i = first; i < n_tickets; i += stride) tickets[i] = 0u;
    for (int i = first; i < n_status; i += stride) status[i] = 0;
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

// 128-row tiles of the N * Hq/Hkv query rows that share a KV head.  One tile: the one-tile kernel
// (two streams over the keys); more: the tile-pair kernel, whose units are pairs of tiles.
static int row_tiles(const ht_attn_desc &d) { return (d.N * (d.Hq / d.Hkv) + tc::kRows - 1) / tc::kRows; }
static bool pair_mode(const ht_attn_desc &d) { return row_tiles(d) >= 2; }
static int units_per_head(const ht_attn_desc &d) { return pair_mode(d) ? (row_tiles(d) + 1) / 2 : 1; }

// Cluster size when the (sequence, KV head[, tile pair]) units are so few that a CTA per unit would
// leave most SMs idle: the largest of 16 (see below), 8, 4, 2 whose clusters fit the GPU at once.
static int clusters16_fit();
static int clusters_fit(int k);

static int cluster_size(const ht_attn_desc &d) {
    const long long units = (long long)d.B * d.Hkv * units_per_head(d);
    const int sms = sm_count();
    // A handful of units with long caches: clusters of 16, beyond the portable size, where the device can hold one per
    // unit at once (a B200 holds seven: one sequence on four KV heads gets them, one on eight does not).  Measured
    // against clusters of eight: 4 x 32768 keys x 152 rows 77.2 -> 49.5 us, x 8000 keys 25.8 -> 20.5 us, x 4096 keys
    // 19.1 -> 17.4 us (tile pairs); one tile of 91 rows: 47.9 -> 32.9 us at 32768 keys, level at 8000, behind at 4096.
    // Where it does not, two clusters of eight or four of four share a unit (cluster_split below), if the device holds those.
    if (units * 16 <= sms && d.cap > (pair_mode(d) ? 4096 : 8192)) {
        if (clusters_fit(16) >= units) return 16;
        if (clusters_fit(8) >= 2 * units) return 8;
        if (clusters_fit(4) >= 4 * units) return 4;
    }
    for (int k = 8; k >= 2; k /= 2)
        if (units * k <= sms) {
            // Clusters leave SMs idle when units * k falls well short of the GPU; that only pays while the
            // cache is short (the capacity bounds its length) and latency, not bandwidth, decides: up to
            // about a dozen tiles per CTA.
            return (units * k * 4 >= 3ll * sms || d.cap <= (k == 8 ? 12288 : 6144)) ? k : 0;
        }
    return 0;
}

// The units' arrival counters sit at the start of the workspace, in an area of a fixed size whatever the
// descriptor (so that calls with different shapes on one workspace leave it clean for one another); more units than
// it holds get an area of their own size, which is then always cleared by the kernel.
constexpr size_t kTicketArea = 64 * 1024;
static size_t ticket_bytes(const ht_attn_desc &d) {
    const size_t units = (size_t)d.B * d.Hkv * units_per_head(d);
    const size_t need = (units * sizeof(unsigned int) + 255) / 256 * 256;
    return need > kTicketArea ? need : kTicketArea;
}
// Several clusters on a unit, where clusters of sixteen would be taken but the device does not hold one per unit (a
// B200 holds 7 of sixteen, 15 of eight, 33 of four: one sequence on eight KV heads gets four clusters of four per
// unit): each reduces its share of the keys through distributed shared memory, and the results meet in the workspace
// (an arrival counter per set of CTAs of one rank; the last finishes).
static int cluster_split(const ht_attn_desc &d) {
    const long long units = (long long)d.B * d.Hkv * units_per_head(d);
    if (!(units * 16 <= sm_count() && d.cap > (pair_mode(d) ? 4096 : 8192))) return 1;
    if (clusters_fit(16) >= units) return 1;
    if (clusters_fit(8) >= 2 * units) return 2;
    if (clusters_fit(4) >= 4 * units) return 4;
    return 1;
}

// Is the kernel that zeroes the counters (and, for a paged cache, the status words) part of the call?
static bool needs_prepare(const ht_attn_desc &d, bool paged) {
    if (paged) return true;                                   // the paged kernels report bad pages from any CTA
    if (cluster_size(d) > 1 && cluster_split(d) == 1) return false;   // one cluster per unit: no counters
    const size_t units = (size_t)d.B * d.Hkv * units_per_head(d);
    return !(d.flags & HT_ATTN_WORKSPACE_CLEAN) || units * sizeof(unsigned int) > kTicketArea;
}

// Arrival counters of the units, then two partial-result slots per CTA (a slot holds one part
// per tile of the unit).
size_t attn_tc_workspace(const ht_attn_desc &d) {
    return ticket_bytes(d) + (size_t)2 * sm_count() * (pair_mode(d) ? 2 : 1) * tc::kSlotFloats * sizeof(float);
}

typedef void (*AttnKernelFn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const tc::Params, const tc::PagedParams);
static AttnKernelFn attn_tc_fn(bool bf16, bool paged, bool clustered) {
    static const AttnKernelFn fns[8] = {
        tc::attn_tc_kernel<false, false, false>, tc::attn_tc_kernel<true, false, false>, tc::attn_tc_kernel<false, true, false>,
        tc::attn_tc_kernel<true, true, false>,   tc::attn_tc_kernel<false, false, true>, tc::attn_tc_kernel<true, false, true>,
        tc::attn_tc_kernel<false, true, true>,   tc::attn_tc_kernel<true, true, true>};
    return fns[(bf16 ? 1 : 0) + (paged ? 2 : 0) + (clustered ? 4 : 0)];
}

// Kernels per call: the attention kernel, and ahead of it the one that zeroes the arrival counters where it is needed.
int attn_tc_launches(const ht_attn_desc &d) { return needs_prepare(d, false) ? 2 : 1; }

// The kernels' dynamic shared memory limit is raised once per device.
static cudaError_t ensure_smem_attr(size_t smem) {
    static bool done[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    for (int i = 0; i < 8; ++i) {
        e = cudaFuncSetAttribute(attn_tc_fn(i & 1, (i >> 1) & 1, i >> 2), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (i >> 2) {                        // the cluster form may be launched in clusters of 16
            e = cudaFuncSetAttribute(attn_tc_fn(i & 1, (i >> 1) & 1, 1), cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e != cudaSuccess) return e;
        }
    }
    if (dev >= 0 && dev < 64) done[dev] = true;
    return cudaSuccess;
}

// Clusters of 16 CTAs of these kernels (one CTA per SM: all of its shared and tensor memory) that the device holds at
// once; 0 where it cannot be asked (no device) or cannot hold any.  The tile-pair kernel has the same footprint.
static int clusters_fit(int k) {
    static int cached[64][3];                // per device and size 4 / 8 / 16; 0: not asked yet, -1: none
    const int slot = k == 16 ? 2 : (k == 8 ? 1 : 0);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return 0;
    }
    if (cached[dev][slot] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(k * 64));
        cfg.blockDim = dim3(tc::kThreads);
        cfg.dynamicSmemBytes = sizeof(tc::Smem) + 1024;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)k;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (ensure_smem_attr(sizeof(tc::Smem) + 1024) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, attn_tc_fn(true, false, true), &cfg) != cudaSuccess) {
            cudaGetLastError();
            n = 0;
        }
        trace("clusters of %d CTAs the device holds at once: %d", k, n);
        cached[dev][slot] = n > 0 ? n : -1;
    }
    return cached[dev][slot] > 0 ? cached[dev][slot] : 0;
}
static int clusters16_fit() { return clusters_fit(16); }

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


int launch_attn_tc_pair_kernel(const CUtensorMap &tm_q, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const tc::Params &p,
                               const tc::PagedParams &pp, bool bf16, bool paged, cudaStream_t s);

int launch_attn_tc(const ht_attn_desc &d, const void *q, const void *kc, const void *vc, const int32_t *kv_len,
                   const int32_t *parent, void *out, void *ws, size_t ws_bytes, int32_t *status, cudaStream_t s,
                   const ht_paged_desc *pages, const int32_t *block_table) {
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
    if (pages) {
        // [page][head][row][D]: a box is the rows of one tile that one page holds
        const long long ph = pages->head_stride ? pages->head_stride : (long long)pages->page_size * d.D;
        const long long pp = pages->page_stride ? pages->page_stride : (long long)d.Hkv * pages->page_size * d.D;
        const cuuint64_t dims[4] = {(cuuint64_t)d.D, (cuuint64_t)pages->page_size, (cuuint64_t)d.Hkv, (cuuint64_t)pages->n_pages};
        const cuuint64_t strides[3] = {(cuuint64_t)d.D * 2, (cuuint64_t)ph * 2, (cuuint64_t)pp * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)(pages->page_size < tc::kTile ? pages->page_size : tc::kTile), 1, 1};
        int rc = make_map(&tm_k, kc, d.dtype, dims, strides, box);
        if (rc != HT_OK) return rc;
        rc = make_map(&tm_v, vc, d.dtype, dims, strides, box);
        if (rc != HT_OK) return rc;
    } else {
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
    p.n_row_tiles = row_tiles(d);
    p.n_rt = units_per_head(d);
    const float scale = d.scale > 0.f ? d.scale : 1.f / sqrtf((float)d.D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.is_bf16 = d.dtype == HT_BF16;
    p.grid = sm_count();
    p.cluster_k = 0;
    p.cluster_split = 1;
    p.wait_kcycles = (d.flags & HT_ATTN_TEST_SHORT_WAITS) ? tc::kWaitKcyclesTest : tc::kWaitKcycles;
    // An early start pays at the edges of a launch (about 3 us).  In the tile-pair kernel, CTAs that start when their
    // SM happens to come free no longer walk a shared head's tiles in step, which costs long launches a little (0.5-1 %
    // from about a hundred tiles per CTA on): there the kernel waits at its start as usual.
    const long long tiles_bound = (long long)d.B * d.Hkv * units_per_head(d) * ((d.cap + tc::kTile - 1) / tc::kTile);
    p.early = ((d.flags & HT_ATTN_CONTEXT_FINAL) && (!pair_mode(d) || tiles_bound <= 96ll * sm_count())) ? 1 : 0;
    tc::PagedParams pp;
    pp.block_table = pages ? block_table : nullptr;
    pp.page_size = pages ? pages->page_size : 0;
    pp.page_shift = 0;
    while (pages && (1 << pp.page_shift) < pages->page_size) ++pp.page_shift;
    pp.max_pages = pages ? pages->max_pages : 0;
    pp.n_pages = pages ? pages->n_pages : 0;
    const size_t smem = offsetof(tc::Smem, anc) + (size_t)((d.N + 31) / 32) * tc::kRows * sizeof(uint32_t) + 1024;
    const long long units = (long long)d.B * d.Hkv * p.n_rt;
    if (units > 0x7fffffffLL) return fail(HT_ERR_UNSUPPORTED, "too many (sequence, head, row tile) units");
    const int k = cluster_size(d), split = k > 1 ? cluster_split(d) : 1;
    cudaError_t e = cudaSuccess;
    if (needs_prepare(d, pages != nullptr)) {
        const int n_t = k <= 1 ? (int)units : (split > 1 ? (int)units * k : 0), n_s = pages ? d.B : 0;
        const int n = n_t > n_s ? n_t : n_s;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((n + 255) / 256 < 64 ? (n + 255) / 256 : 64));
        cfg.blockDim = dim3(256);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, tc::attn_prepare_kernel, p.tickets, n_t, status, n_s);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(HT_ERR_CUDA, "ht_tree_attention (preparation): %s", cudaGetErrorString(e));
        }
    }
    if (k > 1) {
        p.cluster_k = k;
        p.cluster_split = split;
        p.grid = (int)units * k * split;
    }
    if (knobs().log) trace("clusters the device holds: %d of 4, %d of 8, %d of 16", clusters_fit(4), clusters_fit(8), clusters_fit(16));
    trace("ht_tree_attention -> %s kernel, %s, %d CTAs%s%s", pair_mode(d) ? "tile-pair" : "one-tile",
          k > 1 ? (k == 16 ? "clusters of 16" : (k == 8 ? (split == 2 ? "two clusters of 8 per unit" : "clusters of 8") : (k == 4 ? (split == 4 ? "four clusters of 4 per unit" : "clusters of 4") : "clusters of 2"))) : "persistent",
          p.grid, p.early ? ", early start" : "", needs_prepare(d, pages != nullptr) ? ", counters cleared by a kernel" : "");
    if (pair_mode(d)) return launch_attn_tc_pair_kernel(tm_q, tm_k, tm_v, p, pp, d.dtype == HT_BF16, pages != nullptr, s);
    e = ensure_smem_attr(sizeof(tc::Smem) + 1024);
    if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    // Few (sequence, KV head) units: one cluster of 16, 8, 4 or 2 CTAs per unit, parts reduced through
    // distributed shared memory; otherwise one persistent CTA per SM.  Either way the launch is serialized
    // programmatically behind the kernel before it.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(tc::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)(k > 1 ? k : 1);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = k > 1 ? 2 : 1;
    e = cudaLaunchKernelEx(&cfg, attn_tc_fn(d.dtype == HT_BF16, pages != nullptr, k > 1), tm_q, tm_k, tm_v, p, pp);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "ht_tree_attention (tcgen05, clusters of %d): %s", k > 1 ? k : 1, cudaGetErrorString(e));
    }
    return HT_OK;
}

}  // namespace ht
