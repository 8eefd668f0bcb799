// Tree attention on the 5th-generation tensor cores, variant for more than 128 query rows per
// KV head (grouped-query attention: N * Hq/Hkv rows; Section "Tree attention").
//
// With several 128-row tiles per KV head, streaming the cache once per tile would fetch and
// stage every K/V tile several times.  Here a CTA works on TWO row tiles at once: each K/V tile
// is fetched into shared memory once and multiplied with both Q tiles.  The roles are those of
// the one-tile kernel (warp 8: TMA producer, warps 9 and 10: tcgen05.mma issue for stream 0 / 1,
// warps 0-3 / 4-7: one softmax group per row tile, thread i owns row i of its tile), with these
// differences:
//   - stream s = row tile 2*pair + s; every stream sees every K/V tile, keeps its own running
//     max, sum and TMEM accumulator, and there is nothing to merge between streams.
//   - the unit of softmax / MMA work is half a K/V tile (64 keys).  Each stream has two 64-column
//     score buffers in TMEM, so Q K^T of the next half is computed while the softmax of the
//     current one runs, and P V follows as soon as P is written.  TMEM: 4 x 64 (S/P) + 2 x 128 (O).
//   - shared memory: two Q tiles and a ring of three 32 KiB K / V tiles (a fourth bought nothing and its
//     32 KB of footprint cost 1-4 %).
//   - a unit (sequence, KV head, tile pair) whose second tile does not exist runs with stream 1 idle.
// Work split, cut units, tickets and merges are those of the one-tile kernel; a workspace slot
// holds one part per stream.  Every wait is bounded.
#include <stddef.h>

#include "attn_tc.cuh"

namespace ht {
namespace tc {

constexpr int kPStages = 3;
constexpr int kPolyEvery = 4;                  // one pair of exponentials in this many goes to the FMA pipe (a power of two)
constexpr int kPThreads = kThreads + 32;      // + the second MMA-issuing warp
constexpr int kHalf = 64;                     // keys per softmax / MMA step

// 2^x for a pair of values on the FMA pipe instead of the special-function unit (which does 16 a clock
// per SM and is what the tile-pair kernel's exponential pass runs into): x = n + r with n the nearest
// integer (read off the low mantissa bits of x + 1.5 * 2^23) and r in [-1/2, 1/2]; 2^r by a cubic (least
// maximum relative error on that interval, 7.6e-5: a sixth of the rounding of a 16-bit P); n goes into
// the exponent by an integer multiply-add.  x below -125 (masked scores are -inf) gives 2^-125 in place
// of 0, which is 0 to everything it meets afterwards.
__device__ __forceinline__ void ex2_poly_x2(unsigned long long x2, float &p0, float &p1) {
    float x0, x1;
    unpack_f32x2(x2, x0, x1);
    const unsigned long long x = pack_f32x2(fmaxf(x0, -125.f), fmaxf(x1, -125.f));
    const unsigned long long magic = pack_f32x2(12582912.f, 12582912.f);
    const unsigned long long fi = add_f32x2(x, magic);
    const unsigned long long xr = add_f32x2(fi, pack_f32x2(-12582912.f, -12582912.f));
    const unsigned long long r = fma_f32x2(xr, pack_f32x2(-1.f, -1.f), x);
    unsigned long long q = fma_f32x2(pack_f32x2(0.05516993626952171f, 0.05516993626952171f), r,
                                     pack_f32x2(0.24260683357715607f, 0.24260683357715607f));
    q = fma_f32x2(q, r, pack_f32x2(0.693260908126831f, 0.693260908126831f));
    q = fma_f32x2(q, r, pack_f32x2(0.99992835521698f, 0.99992835521698f));
    float q0, q1, f0, f1;
    unpack_f32x2(q, q0, q1);
    unpack_f32x2(fi, f0, f1);
    p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(f0) << 23));
    p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(f1) << 23));
}

// Cluster reduction of the tile-pair kernel: both streams' parts travel in one exchange.  Every CTA owns 128 / k of
// the output features; thread (row, stream) sends its row's 32 feature groups straight from the accumulator into the
// owners' shared memory (Q buffers and ring, idle by then), layout per stream [sender][group in slice][row] float4
// followed by [sender][m | l][row]; behind the second barrier of the cluster the same thread merges the k slices of
// its row and writes the CTA's features of the result.
constexpr int kPXchgMl = kRows * kD * 4;                         // bytes from a stream's area to its m, l
constexpr int kPXchgStream = kPXchgMl + kMaxCluster * 2 * kRows * 4;   // up to 16 senders
static_assert(2 * kPXchgStream <= (2 + kPStages) * kEntryBytes, "the exchange area is the Q buffers and the ring");

struct __align__(1024) PSmem {
    unsigned char q[2][kEntryBytes];
    unsigned char ring[kPStages][kEntryBytes];
    int32_t parent[kMaxWords * 32];
    int32_t len[kMaxB];
    int32_t nkt[kMaxB];
    int32_t pre[kMaxB + 1];
    int32_t plan[kPlanWords];          // the CTA's share of the tiles and its first segment (plan_sequences)
    unsigned char bad_page[kMaxB];     // paged cache, early start: sequences whose bad page entry is reported behind the wait
    unsigned long long kv_full[kPStages], kv_empty[kPStages], q_full, q_empty, s_full[2][2], p_ready[2][2], o_done[2][2], mma_drain;
    int abort, wait_kcycles;           // the abort flag, and right behind it the limit of a wait (the waits read both as one 8-byte word)
    uint32_t tmem_base;
    int merge_here[2];
    int direct;
    int32_t pg[kPgTiles][kPgSub];      // paged cache: page ids of the tiles about to be fetched
    uint32_t anc[2 * kMaxWords * kRows];   // ancestor words [stream][word][row]; last member: only 2 * ceil(N / 32) words are allocated
};

// A stream's received parts lie at `area` as [sender][group in slice][row] float4, followed (at kPXchgMl) by
// [sender][m | l][row]; thread `row` of the stream merges the CTA's whole slice of the row's features.
// (Called by all 256 softmax threads, the threads of stream s with that stream's area.)
// kSplit: the instantiation that knows of several clusters per unit (p.cluster_split > 1); the others carry none of that
// code, whose register needs would otherwise reach into the callers'.
template <bool kBf16, bool kSplit>
__device__ __noinline__ void cluster_merge_pair(const Params &p, const unsigned char *area, int rank, int b, int hk, int row_tile,
                                                bool valid, int row, volatile int *abort_flag) {
    cluster_sync_all();                                 // every part has arrived everywhere; nobody writes to a peer any more
    const int s = (int)threadIdx.x >> 7;                // the stream whose area this is
    const int k = p.cluster_k, cgps = 32 / k;
    const int node = row_tile * p.rows_per_tile_nodes + row / p.g;
    const uint32_t recv = smem_u32(area), recv_ml = recv + kPXchgMl;
    if (kSplit && p.cluster_split > 1) {
        // several clusters (of eight, or of four) share the unit: this one's result is a part
        const bool has_row = valid && row_tile < p.n_row_tiles && node < p.N;
        float f[kMaxCluster], raw[2] = {-INFINITY, 0.f};
        if (has_row) {
            if (k == 8) merge_weights<8>(recv_ml, k, row, f, raw);
            else merge_weights<4>(recv_ml, k, row, f, raw);
        }
        const int unit = ((int)blockIdx.x / k) / p.cluster_split;
        const int head = hk * p.g + row % p.g;
        unsigned char *dst = static_cast<unsigned char *>(p.out) + ((((size_t)b * p.N + node) * p.Hq + head) * kD + rank * cgps * 4) * 2;
        int *const flag = &reinterpret_cast<PSmem *>(const_cast<unsigned char *>(area) - s * kPXchgStream)->direct;   // (the areas start the CTA's shared memory)
        const float *theirs[3];
        sibling_slots(p, 2, s, theirs);
        float *mine = p.part + ((size_t)(2 * (int)blockIdx.x) * 2 + s) * kSlotFloats;
        auto sums = [&](int ch, float4 (&o)[4]) {                // four groups at a time: clusters of eight have four per thread, of four eight
            if (k == 8) merge_sums<4, 8>(recv, k, cgps, row, 4 * ch, f, o);
            else merge_sums<4, 4>(recv, k, cgps, row, 4 * ch, f, o);
        };
        finish_with_siblings<kBf16, 4>(mine, theirs, p.cluster_split - 1, p.tickets + unit * k + rank, flag, sums, k == 8 ? 1 : 2,
                                       raw[0], raw[1], has_row, true, row, 0, dst, (int)threadIdx.x, abort_flag);
        return;
    }
    if (!valid || row_tile >= p.n_row_tiles || node >= p.N || *abort_flag) return;
    float f[kMaxCluster];
    if (k <= 4) merge_weights<4>(recv_ml, k, row, f);
    else if (k == 8) merge_weights<8>(recv_ml, k, row, f);
    else merge_weights<16>(recv_ml, k, row, f);
    const int head = hk * p.g + row % p.g;
    unsigned char *dst = static_cast<unsigned char *>(p.out) + ((((size_t)b * p.N + node) * p.Hq + head) * kD + rank * cgps * 4) * 2;
    if (k == 2) {
        merge_groups<kBf16, 8, 2>(recv, k, cgps, row, 0, f, dst);
        merge_groups<kBf16, 8, 2>(recv, k, cgps, row, 8, f, dst + 64);
    } else if (k == 4) {
        merge_groups<kBf16, 8, 4>(recv, k, cgps, row, 0, f, dst);
    } else if (k == 8) {
        merge_groups<kBf16, 4, 8>(recv, k, cgps, row, 0, f, dst);
    } else {
        merge_groups<kBf16, 2, 16>(recv, k, cgps, row, 0, f, dst);
    }
}


template <bool kBf16, bool kPaged, bool kSplit>
__global__ void __launch_bounds__(kPThreads, 1)
attn_tc_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const Params p, const PagedParams pp) {
    extern __shared__ unsigned char smem_raw[];
    PSmem &sm = *reinterpret_cast<PSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sm.abort;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kPStages; ++i) { mbar_init(&sm.kv_full[i], 1); mbar_init(&sm.kv_empty[i], 2); }
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_empty, 2);          // one arrival per issuing thread
        mbar_init(&sm.mma_drain, 2);
        for (int s = 0; s < 2; ++s)
            for (int h = 0; h < 2; ++h) {
                mbar_init(&sm.s_full[s][h], 1);
                mbar_init(&sm.p_ready[s][h], 128);
                mbar_init(&sm.o_done[s][h], 1);
            }
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
    // up while that kernel was still finishing, and everything it may have written is read from here on.  `early`
    // (lengths, trees and the cache rows below the lengths were final before that kernel began): as in the one-tile
    // kernel, plan and first context tiles do not wait, and each role waits where it first needs to.
    const bool early = p.early != 0;
    if (kPaged && early)
        for (int b = threadIdx.x; b < p.B; b += blockDim.x) sm.bad_page[b] = 0;     // (the plan's barriers come before any fetch)
    if (!early) wait_for_kernel_ahead();
    // Without clusters, where a KV head has several tile pairs (units), the list of tiles is that of the HEADS: it is
    // cut into grid / n_rt ranges, and the n_rt CTAs of a range take one tile pair each.  They start together and walk
    // the same K / V tiles at the same pace, so that a tile crosses DRAM once and reaches the others from L2.  (With
    // the units laid end to end instead, the CTAs that share a head's tiles meet them dozens of tiles apart: twice the
    // algorithmic DRAM traffic on 4 x 8192 keys x 67 rows.)
    const bool clustered = p.cluster_k > 1;
    const bool grouped = !clustered && p.n_rt > 1;
    const int lrt = grouped ? 1 : p.n_rt;                                   // units per head in the list
    const int my_rt = grouped ? (int)blockIdx.x % p.n_rt : 0;               // grouped: this CTA's tile pair
    const int my_pos = grouped ? (int)blockIdx.x / p.n_rt : (int)blockIdx.x; // place in the list's partition
    const int n_pos = grouped ? p.grid / p.n_rt : p.grid;
    // Cluster form: one cluster per (sequence, KV head, tile pair); its CTAs take cost-equal shares of the unit's tiles.
    // (No cluster barrier here: the first remote access comes after the one all threads pass ahead of the exchange.)
    // One thread works the CTA's range and its first segment out.
    uint32_t c_rank = 0;
    RangeAsk ask;
    ask.n_pos = n_pos; ask.my_pos = my_pos;
    ask.cluster_k = 0; ask.cl_rank = 0; ask.cl_b = 0; ask.cl_unit = 0;
    if (clustered) {
        c_rank = cluster_ctarank();
        // (two clusters on a unit, p.cluster_split == 2: their CTAs share the unit's tiles like one cluster of twice the size)
        ask.cluster_k = p.cluster_k * p.cluster_split;                 // a power of two
        ask.cl_rank = (int)blockIdx.x & (ask.cluster_k - 1);
        const int unit = (int)blockIdx.x >> (__ffs(ask.cluster_k) - 1);
        ask.cl_b = unit / (p.Hkv * p.n_rt);
        ask.cl_unit = unit - ask.cl_b * p.Hkv * p.n_rt;
    }
    tc_fence_before();                              // (the tensor memory's base address crosses the plan's last barrier)
    plan_sequences<kPThreads>(p, sm.len, sm.nkt, sm.pre, blockIdx.x == 0 && !early, kPaged, lrt, ask, sm.plan);
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const Range range = read_range(sm.plan);
    const int per = range.per, t_begin = range.t_begin, t_end = range.t_end;
    Segment first = range.first;
    if (grouped) first.rt = my_rt;
    // the segment that holds tile t of the list; grouped: the tile pair is the CTA's own
    auto find = [&](int t, int te, int &hint) {
        if (t == t_begin) {
            hint = first.b;
            return first;
        }
        Segment sg = locate(sm.pre, sm.nkt, p.B, lrt, t, te, hint);
        if (grouped) sg.rt = my_rt;
        return sg;
    };
    unsigned char *const xarea = &sm.q[0][0];          // Q buffers and ring, idle once the CTA's tiles are done
    // The Q tiles of a segment's tile pair (one where the pair has no second tile).
    auto fetch_q = [&](const Segment &s) {
        const bool two = 2 * s.rt + 1 < p.n_row_tiles;
        mbar_expect_tx(&sm.q_full, two ? 2 * kEntryBytes : kEntryBytes);
        for (int x = 0; x < (two ? 2 : 1); ++x) {
            const int node0 = (2 * s.rt + x) * p.rows_per_tile_nodes;
            tma_load_4d(sm.q[x], &tm_q, &sm.q_full, 0, s.hk * p.g, node0, s.b);
            tma_load_4d(sm.q[x] + kSlabBytes, &tm_q, &sm.q_full, 64, s.hk * p.g, node0, s.b);
        }
    };
    // Cluster mode: the unit's parts are exchanged between two barriers of the whole cluster (the softmax threads pass
    // them around their sends, the other warps once their work is done).

    if (warp == 8) {
        // ------------------------------- TMA producer -------------------------------
        // Contiguous cache: one thread.  Paged cache: the whole warp walks the loop with identical state and
        // lane x looks up and fetches page x of a tile; lane 0 alone arms the barriers and fetches Q.
        if (kPaged || lane == 0) {
            int b_hint = 0, ring_i = 0, seg_i = 0;
            TileCursor cur_p;                         // page-id lookahead
            cur_p.init(t_begin, t_end, first);
            if (kPaged)
                for (int jt = 0; jt < kPgAhead; ++jt) pages_request(p, pp, sm.pre, sm.nkt, sm.pg, jt, cur_p, lane, lrt);
            bool stop = false;
            bool waited = !early;                  // early: the range's first Q tiles are fetched by stream 0's issuing thread, behind its wait
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
            for (int t = t_begin; t < t_end && !stop;) {
                if (kPaged ? __any_sync(0xFFFFFFFFu, *abort_flag != 0) : (*abort_flag != 0)) break;
                const Segment s = find(t, t_end, b_hint);
                if (seg_i > 0) release();
                {
                    bool ok = seg_i == 0 || mbar_wait_quick(smem_u32(&sm.q_empty), (seg_i - 1) & 1, abort_flag);
                    if (kPaged) ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                }
                if (lane == 0 && !(early && seg_i == 0)) fetch_q(s);
                ++seg_i;
                for (int i = 0; i < 2 * s.len; ++i) {
                    const int kt = s.kt0 + (i >> 1);
                    // early: context tiles only, and no more of them than the ring holds, ahead of the wait
                    if (!waited && ((kt + 1) * kTile > sm.len[s.b] || ring_i >= kPStages)) release();
                    const int slot = ring_i % kPStages, use = ring_i / kPStages;
                    bool ok = use == 0 || mbar_wait_quick(smem_u32(&sm.kv_empty[slot]), (use - 1) & 1, abort_flag);
                    if (kPaged) ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) { stop = true; break; }
                    const CUtensorMap *tm = (i & 1) ? &tm_v : &tm_k;
                    const int jt = t - t_begin + (i >> 1);            // tile of this CTA's range
                    if (kPaged && !(i & 1)) {
                        pages_request(p, pp, sm.pre, sm.nkt, sm.pg, jt + kPgAhead, cur_p, lane, lrt);
                        cp_async_wait<kPgAhead>();
                    }
                    if (lane == 0) mbar_expect_tx(&sm.kv_full[slot], kEntryBytes);
                    if (kPaged) {
                        __syncwarp();                                 // the barrier is armed before any lane's copy can complete
                        fetch_kv_tile_paged(p, pp, sm.ring[slot], tm, &sm.kv_full[slot], s.b, s.hk, kt, sm.len[s.b] + p.N,
                                            sm.pg[jt % kPgTiles], lane, waited ? nullptr : sm.bad_page);
                    } else {
                        fetch_kv_tile(sm.ring[slot], tm, &sm.kv_full[slot], s.b, s.hk, kt);
                    }
                    ++ring_i;
                }
                t += s.len;
            }
            if (kPaged) {
                cp_async_wait<0>();
                __syncwarp();
            }
            release();
            if (lane == 0) {
                // how many ring entries and Q fetches were asked for: should the CTA give up, the teardown waits for the
                // last of them (early: the first Q tiles were fetched by stream 0's issuing thread, whatever else happened)
                sm.plan[9] = ring_i;
                sm.plan[10] = early && t_end > t_begin && seg_i == 0 ? 1 : seg_i;
            }
        }
        if (clustered) { cluster_sync_all(); cluster_sync_all(); }
    } else if (warp >= 9) {
        // ------------------------------- MMA issuers -------------------------------
        // One issuing thread per stream (warp 9: stream 0, warp 10: stream 1), so that neither stream
        // ever waits for the other's softmax.  Per half tile H (64 keys): Q K^T into score buffer H & 1,
        // then P V of half H - 1; a score buffer is rewritten only after the P V that read it has been
        // issued.  A tcgen05.commit covers the issuing thread's own operations, so the K / V slots and the
        // Q buffers are released by one arrival from each of the two threads; in a unit without a second
        // tile the thread of stream 1 issues nothing and only keeps step with the ring.
        // Each thread is a chain of dependent instructions that shares its scheduler with two softmax warps, so the
        // instructions per half tile are kept few: ring slots and phases are counted (no division), barrier
        // addresses and descriptor words are formed once, each product is one instruction sequence, and the
        // abort flag is looked at only when a wait has to spin.
        if (lane == 0) {
            const int s = warp - 9;
            if (early) {
                // q is the kernel ahead's to write: the range's first Q tiles are fetched here (stream 0's thread),
                // behind the wait, while the producer is busy with the first context tiles
                wait_for_kernel_ahead();
                if (s == 0 && t_end > t_begin) {
                    int hint = 0;
                    fetch_q(find(t_begin, t_end, hint));
                }
            }
            const uint32_t idesc_qk = instr_desc(kBf16, 0, kHalf), idesc_pv = instr_desc(kBf16, 1, 128);
            const uint32_t hi_k = desc_hi(1, 1024 >> 4), hi_v = desc_hi(kSlabBytes >> 4, 1024 >> 4);
            const uint32_t q_lo = desc_lo_with_lbo(smem_u32(sm.q[s]), 1);
            const uint32_t ring_k_lo = desc_lo_with_lbo(smem_u32(sm.ring[0]), 1);            // slot x: + x * (kEntryBytes / 16)
            const uint32_t ring_v_lo = desc_lo_with_lbo(smem_u32(sm.ring[0]), kSlabBytes >> 4);
            const uint32_t bar_kv_full = smem_u32(&sm.kv_full[0]), bar_kv_empty = smem_u32(&sm.kv_empty[0]);
            const uint32_t bar_s_full = smem_u32(&sm.s_full[s][0]), bar_p_ready = smem_u32(&sm.p_ready[s][0]), bar_o_done = smem_u32(&sm.o_done[s][0]);
            const uint32_t s_tmem = tmem + s * 128, o_tmem = tmem + 256 + s * 128;
            int b_hint = 0, seg_i = 0;
            uint32_t uses0 = 0, uses1 = 0;                  // completed uses of p_ready[s][0 / 1]
            bool pend = false, pend_first = false;          // the half tile whose P V is still to be issued
            bool pend_tree = false;                         // it holds tree keys: its P is a hi + lo pair (see the softmax)
            uint32_t pend_h = 0, pend_slot = 0, pend_ph = 0; // ... its half, and the slot and phase of its V tile
            bool alive = !*abort_flag;                      // false once a wait of this thread has given up: no further waits or products
            uint32_t slot = 0, ph = 0;                      // ring entries alternate K, V: slot and phase of the next entry
            auto advance = [&]() {
                if (++slot == (uint32_t)kPStages) { slot = 0; ph ^= 1u; }
            };
            auto issue_pv = [&]() {
                if (pend_h == 0) alive = alive && mbar_wait_quick(bar_kv_full + pend_slot * 8, pend_ph, abort_flag);
                const uint32_t u = pend_h ? uses1 : uses0;
                alive = alive && mbar_wait_quick(bar_p_ready + pend_h * 8, u & 1, abort_flag);
                if (pend_h) ++uses1; else ++uses0;
                tc_fence_after();
                if (alive) {
                    // V as B operand, MN-major: 64 features contiguous per key (one swizzled 128-byte line), the
                    // second 64-feature slab one slab further (LBO), groups of 8 keys 1 KiB apart (SBO); 16 keys
                    // per instruction = 2 KiB.
                    const uint32_t v_lo = ring_v_lo + pend_slot * (kEntryBytes >> 4) + pend_h * (kHalf * 128 >> 4);
                    if (!pend_tree) mma_block_pv64(o_tmem, s_tmem + pend_h * kHalf, v_lo, hi_v, idesc_pv, pend_first ? 0u : 1u);
                    else mma_block_pv64_hilo(o_tmem, s_tmem + pend_h * kHalf, v_lo, hi_v, idesc_pv, pend_first ? 0u : 1u);
                }
                tc_commit_addr(bar_o_done + pend_h * 8);
                if (pend_h == 1) tc_commit_addr(bar_kv_empty + pend_slot * 8);
                pend = false;
            };
            for (int t = t_begin; t < t_end;) {
                const Segment sg = find(t, t_end, b_hint);
                const bool act = s == 0 || 2 * sg.rt + 1 < p.n_row_tiles;
                const int L = sm.len[sg.b];
                alive = alive && mbar_wait_quick(smem_u32(&sm.q_full), seg_i & 1, abort_flag);
                for (int i = 0; i < sg.len; ++i) {
                    const uint32_t k_slot = slot;
                    alive = alive && mbar_wait_quick(bar_kv_full + slot * 8, ph, abort_flag);
                    tc_fence_after();
                    advance();
                    const uint32_t v_slot = slot, v_ph = ph;
                    advance();
                    if (!act) {
                        // keep step with the ring: hand both slots of this tile back once they are loaded
                        if (pend) issue_pv();
                        tc_commit_addr(bar_kv_empty + k_slot * 8);
                        if (i == sg.len - 1) tc_commit(&sm.q_empty);
                        alive = alive && mbar_wait_quick(bar_kv_full + v_slot * 8, v_ph, abort_flag);
                        tc_commit_addr(bar_kv_empty + v_slot * 8);
                        continue;
                    }
                    const int key_hi = (sg.kt0 + i) * kTile + kHalf;        // end of the tile's first half
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        // K-major operands: 16 features = 32 bytes inside the 128-byte swizzled line; the second
                        // 64-feature slab lies one slab further.
                        if (alive) mma_block_qk(s_tmem + h * kHalf, q_lo, ring_k_lo + k_slot * (kEntryBytes >> 4) + h * (kHalf * 128 >> 4), hi_k, idesc_qk);
                        tc_commit_addr(bar_s_full + h * 8);
                        if (h == 1) {
                            tc_commit_addr(bar_kv_empty + k_slot * 8);
                            if (i == sg.len - 1) tc_commit(&sm.q_empty);
                        }
                        if (pend) issue_pv();
                        pend = true;
                        pend_first = (i == 0 && h == 0);
                        pend_tree = key_hi + h * kHalf > L;
                        pend_h = h;
                        pend_slot = v_slot;
                        pend_ph = v_ph;
                    }
                }
                t += sg.len;
                ++seg_i;
            }
            if (pend) issue_pv();
            // No tensor-core operation of this CTA may be in flight when its TMEM is freed.
            tc_commit(&sm.mma_drain);
            mbar_wait(&sm.mma_drain, 0, abort_flag, false);
        }
        if (clustered) { cluster_sync_all(); cluster_sync_all(); }
    } else {
        // ------------------------------- softmax groups -------------------------------
        const int s = warp >> 2;                       // stream of this group = which tile of the pair
        const int row = threadIdx.x & 127;             // query row within the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int tid256 = threadIdx.x;                // 0..255 among the softmax threads
        const int words = (p.N + 31) >> 5;
        const unsigned long long scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
        const uint32_t o_addr = tmem + lane_base + 256 + s * 128;
        int b_hint = 0, J = 0;
        float xa[32], xb[32];
        CutUnit cut[2];
        unsigned int ticket[2] = {0u, 0u};
        cut[0].valid = cut[1].valid = 0;
        int anc_b = -1, anc_rt = -1;                   // sequence / tile pair the ancestor words were built for
        uint32_t uses_s[2] = {0, 0}, uses_o[2] = {0, 0};   // uses of s_full[s][h] / o_done[s][h] so far
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
            const Segment sg = find(t, t_end, b_hint);
            const int L = sm.len[sg.b];
            const int row_tile = 2 * sg.rt + s;
            const bool active = row_tile < p.n_row_tiles;
            const bool two = 2 * sg.rt + 1 < p.n_row_tiles;
            const int node = row_tile * p.rows_per_tile_nodes + row / p.g;
            const bool real = active && node < p.N;
            // a warp none of whose 32 rows is a query row keeps step with the barriers but computes nothing
            const bool warp_real = active && row_tile * p.rows_per_tile_nodes + (row & ~31) / p.g < p.N;
            if (sg.b != anc_b || sg.rt != anc_rt) {
                softmax_groups_sync();                 // previous segment no longer reads parent / anc
                for (int c = tid256; c < p.N; c += 256) sm.parent[c] = p.parent[(size_t)sg.b * p.N + c];
                softmax_groups_sync();
                for (int w = 0; w < words; ++w) sm.anc[(s * words + w) * kRows + row] = 0u;   // padding rows see the context only; their results are dropped
                if (real)
                    for (int c = node; c >= 0; c = sm.parent[c]) sm.anc[(s * words + (c >> 5)) * kRows + row] |= 1u << (c & 31);
                softmax_groups_sync();
                anc_b = sg.b;
                anc_rt = sg.rt;
            }
            release();
            // A segment that is only part of its unit: see the one-tile kernel.
            const bool complete = sg.kt0 == 0 && sg.len == sg.nkt;
            const int cut_k = (t == t_begin) ? 0 : 1;
            unsigned int delivered = 0, delivered_old = 0;
            if (!complete) {
                CutUnit &cu = cut[cut_k];
                cu.unit = (sg.b * p.Hkv + sg.hk) * p.n_rt + sg.rt;
                cu.b = sg.b; cu.hk = sg.hk; cu.rt = sg.rt;
                cu.t0 = sm.pre[sg.b] + (grouped ? sg.hk : sg.hk * p.n_rt + sg.rt) * sg.nkt;
                cu.cta_mul = grouped ? p.n_rt : 1; cu.cta_add = my_rt;
                cu.c_lo = cu.t0 / per;
                cu.c_hi = (cu.t0 + sg.nkt - 1) / per;
            }

            float m_ref = -INFINITY, l_sum = 0.f;
            int last_h = -1;                            // score buffer of this stream's latest P V in this segment
            if (active) {
#pragma unroll 1
                for (int ih = 0; ih < 2 * sg.len; ++ih) {
                    const int i = ih >> 1, h = ih & 1;
                    const int kt = sg.kt0 + i;
                    if (!complete && !clustered && tid256 == 0 && h == 0) {
                        delivered_old = delivered;
                        delivered = ld_relaxed_gpu(&p.tickets[cut[cut_k].unit]);
                    }
                    mbar_wait(&sm.s_full[s][h], uses_s[h] & 1, abort_flag);
                    ++uses_s[h];
                    tc_fence_after();
                    const uint32_t s_addr = tmem + lane_base + s * 128 + h * kHalf;
                    const int key_lo = kt * kTile + h * kHalf;
                    if (warp_real) {
                    if (key_lo + kHalf > L) {
                        // Reaches into the tree rows / the tail: scores of keys this row must not see
                        // become -inf in place (context visible, tree key c iff ancestor bit c, tail never).
#pragma unroll 1
                        for (int w = 0; w < 2; ++w) {
                            const int cc0 = key_lo + 32 * w - L;
                            if (cc0 <= -32) continue;
                            const int wi = cc0 >> 5, sh = cc0 & 31;
                            const uint32_t lo = wi < 0 ? 0xFFFFFFFFu : (wi < words ? sm.anc[(s * words + wi) * kRows + row] : 0u);
                            const uint32_t hi = (wi + 1 >= 0 && wi + 1 < words) ? sm.anc[(s * words + wi + 1) * kRows + row] : 0u;
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
                    // --- pass 1: row maximum over the 64 scores (they stay in registers for pass 2) ---
                    float mx0 = -INFINITY, mx1 = -INFINITY;
                    tmem_ld32(s_addr, xa);
                    tmem_ld32(s_addr + 32, xb);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        mx0 = max3(mx0, xa[c], xa[c + 1]);
                        mx1 = max3(mx1, xa[c + 2], xa[c + 3]);
                    }
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        mx0 = max3(mx0, xb[c], xb[c + 1]);
                        mx1 = max3(mx1, xb[c + 2], xb[c + 3]);
                    }
                    const float mx = fmaxf(mx0, mx1) * p.scale_log2;
                    // --- running maximum, raised lazily ---
                    const float m_new = fmaxf(m_ref, mx);
                    const bool grow = (m_ref != -INFINITY) && (m_new > m_ref + kRescaleThreshold);
                    if (m_ref == -INFINITY) m_ref = m_new;
                    if (__any_sync(0xffffffffu, grow)) {
                        // The accumulator may be rescaled once this stream's latest P V has completed
                        // (the next one is not issued before this thread reports P ready).
                        if (last_h >= 0) {
                            mbar_wait(&sm.o_done[s][last_h], (uses_o[last_h] - 1) & 1, abort_flag);
                            tc_fence_after();
                        }
                        const float f = grow ? exp2f(m_ref - m_new) : 1.f;
#pragma unroll 1
                        for (int c4 = 0; c4 < 4; ++c4) {
                            float o[32];
                            uint32_t r[32];
                            tmem_ld32(o_addr + c4 * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(o[c] * f);
                            tmem_st32(o_addr + c4 * 32, r);
                        }
                        tmem_st_wait();
                        l_sum *= f;
                        if (grow) m_ref = m_new;
                    }
                    const float base = (m_ref == -INFINITY) ? 0.f : m_ref;
                    // --- pass 2: exponentials, row sum, P as packed 16-bit pairs over the consumed scores ---
                    const unsigned long long nbase2 = pack_f32x2(-base, -base);
                    unsigned long long acc2 = pack_f32x2(0.f, 0.f);
                    // 32 scores -> 16 packed pairs at column `col`.  Half tiles with tree keys (a row may see a handful
                    // of keys only, and then the rounding of its weights to 16 bits is no longer averaged away) send P
                    // to the tensor pipe as a pair hi + lo of 16-bit values: a second sweep forms the same exponentials
                    // again and stores what the rounding took away 32 columns further (all 64 scores are in registers,
                    // so the buffer's upper half is free), and P V is issued for both.
                    const bool hi_lo = key_lo + kHalf > L;
                    auto chunk = [&](const float *x, uint32_t col) {
                        uint32_t r[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float p0, p1;
                            const unsigned long long x2 = fma_f32x2(pack_f32x2(x[2 * c], x[2 * c + 1]), scale2, nbase2);
                            if ((c & (kPolyEvery - 1)) == kPolyEvery - 1) {
                                ex2_poly_x2(x2, p0, p1);
                            } else {
                                unpack_f32x2(x2, p0, p1);
                                p0 = ex2(p0);
                                p1 = ex2(p1);
                            }
                            acc2 = add_f32x2(acc2, pack_f32x2(p0, p1));
                            r[c] = pack2<kBf16>(p0, p1);
                        }
                        tmem_st16(col, r);
                        if (hi_lo) {
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                float p0, p1;
                                const unsigned long long x2 = fma_f32x2(pack_f32x2(x[2 * c], x[2 * c + 1]), scale2, nbase2);
                                if ((c & (kPolyEvery - 1)) == kPolyEvery - 1) {
                                    ex2_poly_x2(x2, p0, p1);
                                } else {
                                    unpack_f32x2(x2, p0, p1);
                                    p0 = ex2(p0);
                                    p1 = ex2(p1);
                                }
                                r[c] = pack2_rest<kBf16>(p0, p1, r[c]);
                            }
                            tmem_st16(col + 32, r);
                        }
                    };
                    chunk(xa, s_addr);
                    chunk(xb, s_addr + 16);
                    {
                        float a0, a1;
                        unpack_f32x2(acc2, a0, a1);
                        l_sum += a0 + a1;
                    }
                    tmem_st_wait();
                    }
                    // --- last tile of the unit: rows of V past the tree are not data; make them zero (both
                    // streams write the same zeros, each before it lets its own P V go) ---
                    if (kt == sg.nkt - 1 && h == 0) {
                        const int valid = L + p.N - kt * kTile;
                        if (valid < kTile) {
                            const int e = 2 * (J + i) + 1, slot = e % kPStages;
                            mbar_wait(&sm.kv_full[slot], (e / kPStages) & 1, abort_flag);
                            const int vecs = (kTile - valid) * 8;               // 16-byte vectors per slab
                            for (int v = row; v < vecs; v += 128) {
                                *reinterpret_cast<uint4 *>(sm.ring[slot] + valid * 128 + v * 16) = make_uint4(0, 0, 0, 0);
                                *reinterpret_cast<uint4 *>(sm.ring[slot] + kSlabBytes + valid * 128 + v * 16) = make_uint4(0, 0, 0, 0);
                            }
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        }
                    }
                    tc_fence_before();
                    mbar_arrive(&sm.p_ready[s][h]);
                    ++uses_o[h];                        // the P V of this half will arrive on o_done[s][h]
                    last_h = h;
                }
                // the segment's last P V of this stream
                mbar_wait(&sm.o_done[s][last_h], (uses_o[last_h] - 1) & 1, abort_flag);
                tc_fence_after();
            }
            // --- segment epilogue: write the result, finish a cut unit, or leave a part ---
            if (tid256 == 0) {
                sm.direct = !clustered && !complete && cut[cut_k].c_hi - cut[cut_k].c_lo == 1 && delivered_old == 1u;
                // nobody touches the unit's counter any more: it is left at zero for the next call on this workspace
                if (sm.direct) p.tickets[cut[cut_k].unit] = 0u;
            }
            tc_fence_before();
            softmax_groups_sync();
            tc_fence_after();
            const bool direct = sm.direct;
            const bool final = (complete && !clustered) || direct;
            // this stream's rows: normalised to `out` (fin), merged with the one other part first (dir), or as a part to dst
            const int xk_sh = clustered ? 5 - __ffs(p.cluster_k) + 1 : 0;        // log2 of the 4-feature groups per peer's slice
            const uint32_t xrecv = smem_u32(xarea) + (uint32_t)(s * kPXchgStream);  // this stream's receive area: same offset in every CTA
            auto emit = [&](float *dst, bool fin, bool dir, bool peer) {
                const int head = sg.hk * p.g + row % p.g;
                const float *oslot = dst;              // the other part, when finishing the unit here
                float g0, gb = 0.f;
                if (dir) {
                    const CutUnit &cu = cut[cut_k];
                    const int oc = (cu.c_lo == my_pos) ? cu.c_hi : cu.c_lo;
                    oslot = p.part + ((size_t)(2 * (oc * cu.cta_mul + cu.cta_add) + ((max(cu.t0, oc * per) == oc * per) ? 0 : 1)) * 2 + s) * kSlotFloats;
                    __threadfence();
                    const float m_o = __ldcg(oslot + kRows * kD + row), l_o = __ldcg(oslot + kRows * kD + kRows + row);
                    const float Mn = fmaxf(m_ref, m_o);
                    const float fa = (m_ref == -INFINITY) ? 0.f : exp2f(m_ref - Mn);
                    const float fb = (m_o == -INFINITY) ? 0.f : exp2f(m_o - Mn);
                    const float inv = 1.f / (l_sum * fa + l_o * fb);
                    g0 = fa * inv;
                    gb = fb * inv;
                } else {
                    g0 = fin ? 1.f / l_sum : 1.f;
                }
#pragma unroll 1
                for (int c4 = 0; c4 < (warp_real ? 4 : 0); ++c4) {
                    const int col0 = c4 * 32;
                    tmem_ld32(o_addr + col0, xa);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) xa[c] *= g0;
                    if (!real) continue;
                    if (dir) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const float4 v = __ldcg(reinterpret_cast<const float4 *>(oslot) + (col0 / 4 + c) * kRows + row);
                            xa[4 * c] = fmaf(gb, v.x, xa[4 * c]);
                            xa[4 * c + 1] = fmaf(gb, v.y, xa[4 * c + 1]);
                            xa[4 * c + 2] = fmaf(gb, v.z, xa[4 * c + 2]);
                            xa[4 * c + 3] = fmaf(gb, v.w, xa[4 * c + 3]);
                        }
                    }
                    if (fin) {
                        uint32_t w[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) w[c] = pack2<kBf16>(xa[2 * c], xa[2 * c + 1]);
                        unsigned char *o = static_cast<unsigned char *>(p.out) +
                                           ((((size_t)sg.b * p.N + node) * p.Hq + head) * kD + col0) * 2;
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4 *>(o + c * 16) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                    } else if (peer) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) {    // feature group cg belongs to peer cg >> xk_sh, as that slice's group x
                            const int cg = col0 / 4 + c, x = cg & ((1 << xk_sh) - 1);
                            st_peer_f4(map_to_peer(xrecv + (uint32_t)((((int)c_rank << xk_sh) + x) * kRows + row) * 16u, (uint32_t)(cg >> xk_sh)),
                                       make_float4(xa[4 * c], xa[4 * c + 1], xa[4 * c + 2], xa[4 * c + 3]));
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            reinterpret_cast<float4 *>(dst)[(col0 / 4 + c) * kRows + row] = make_float4(xa[4 * c], xa[4 * c + 1], xa[4 * c + 2], xa[4 * c + 3]);
                    }
                }
                if (peer) {
                    if (real)
                        for (int c = 0; c < p.cluster_k; ++c) {
                            const uint32_t ml = map_to_peer(xrecv + (uint32_t)(kPXchgMl + ((int)c_rank * 2 * kRows + row) * 4), (uint32_t)c);
                            st_peer_f1(ml, m_ref);
                            st_peer_f1(ml + kRows * 4, l_sum);
                        }
                } else if (!fin && real) {
                    dst[kRows * kD + row] = m_ref;
                    dst[kRows * kD + kRows + row] = l_sum;
                }
            };
            if (clustered) {
                // The unit's parts are reduced inside the cluster: behind a barrier that every thread of the cluster
                // passes once its work is done (all parts complete, no ring in use) each stream's threads send
                // their rows to the features' owners; the merge follows behind a second barrier.
                cluster_sync_all();
                if (active) emit(nullptr, false, false, true);
                tc_fence_before();
                cluster_merge_pair<kBf16, kSplit>(p, xarea + s * kPXchgStream, (int)c_rank, sg.b, sg.hk, row_tile, true, row, abort_flag);
            } else if (active) {
                emit(p.part + ((size_t)(2 * (int)blockIdx.x + cut_k) * 2 + s) * kSlotFloats, final || direct, direct, false);
            }
            tc_fence_before();
            softmax_groups_sync();                     // the accumulators are free for the next segment
            if (!final && !clustered) {
                cut[cut_k].valid = two ? 3 : 1;         // which streams left a part
                if (tid256 == 0) {
                    __threadfence();
                    ticket[cut_k] = atomicAdd(&p.tickets[cut[cut_k].unit], 1u);
                }
            }
            J += sg.len;
            t += sg.len;
        }
        release();
        if (clustered && t_end <= t_begin) {
            // an empty share still takes part in the cluster's exchange, with parts that saw nothing
            const int unit = (int)blockIdx.x / (p.cluster_k * p.cluster_split), b = unit / (p.Hkv * p.n_rt);
            const int rem = unit - b * p.Hkv * p.n_rt, hk = rem / p.n_rt, rt = rem - hk * p.n_rt;
            cluster_sync_all();
            if (2 * rt + s < p.n_row_tiles)
                for (int c = 0; c < p.cluster_k; ++c) {
                    const uint32_t ml = map_to_peer(smem_u32(xarea) + (uint32_t)(s * kPXchgStream + kPXchgMl + ((int)c_rank * 2 * kRows + row) * 4), (uint32_t)c);
                    st_peer_f1(ml, -INFINITY);
                    st_peer_f1(ml + kRows * 4, 0.f);
                }
            cluster_merge_pair<kBf16, kSplit>(p, xarea + s * kPXchgStream, (int)c_rank, b, hk, 2 * rt + s, sm.nkt[b] > 0, row, abort_flag);
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
                    for (int x = 0; x < 2; ++x)
                        if (cut[k].valid & (1 << x)) merge_parts<kBf16>(p, cut[k], per, tid256, 2 * cut[k].rt + x, x, 2);
                }
        }
    }

    // ------------------------------- teardown -------------------------------
    tc_fence_before();
    __syncthreads();
    // (cluster mode: the last exchange's second barrier already guarantees that no peer writes here any more)
    if (sm.abort && threadIdx.x == 0) {
        for (int b = 0; b < p.B; ++b)
            if (sm.nkt[b] > 0) p.status[b] = HT_STATUS_TIMEOUT;
    }
    if (sm.abort && threadIdx.x == 8 * 32) {
        // Some wait of this CTA ran out, wherever: every copy it asked for must have landed before it exits (this
        // warp leaves last: it frees the tensor memory below).
        const int ring_i = sm.plan[9], q_fetches = sm.plan[10];
        for (int e = max(0, ring_i - kPStages); e < ring_i; ++e)
            mbar_wait(&sm.kv_full[e % kPStages], (e / kPStages) & 1, abort_flag, false);
        if (q_fetches > 0) mbar_wait(&sm.q_full, (q_fetches - 1) & 1, abort_flag, false);
    }
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace tc

// Raises the kernels' dynamic shared memory limit (once per device) and launches.
int launch_attn_tc_pair_kernel(const CUtensorMap &tm_q, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const tc::Params &p,
                               const tc::PagedParams &pp, bool bf16, bool paged, cudaStream_t s) {
    typedef void (*Fn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const tc::Params, const tc::PagedParams);
    const Fn fns[8] = {tc::attn_tc_pair_kernel<false, false, false>, tc::attn_tc_pair_kernel<true, false, false>,
                       tc::attn_tc_pair_kernel<false, true, false>,  tc::attn_tc_pair_kernel<true, true, false>,
                       tc::attn_tc_pair_kernel<false, false, true>,  tc::attn_tc_pair_kernel<true, false, true>,
                       tc::attn_tc_pair_kernel<false, true, true>,   tc::attn_tc_pair_kernel<true, true, true>};
    const Fn fn = fns[(bf16 ? 1 : 0) + (paged ? 2 : 0) + (p.cluster_split > 1 ? 4 : 0)];
    static bool done[64];
    const size_t smem_max = sizeof(tc::PSmem) + 1024;
    const size_t smem = offsetof(tc::PSmem, anc) + (size_t)2 * ((p.N + 31) / 32) * tc::kRows * sizeof(uint32_t) + 1024;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (!(dev >= 0 && dev < 64 && done[dev])) {
        for (int i = 0; i < 8 && e == cudaSuccess; ++i) {
            e = cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(fns[i], cudaFuncAttributeNonPortableClusterSizeAllowed, 1);   // clusters of 16
        }
        if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        if (dev >= 0 && dev < 64) done[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(tc::kPThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // see launch_attn_tc
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)(p.cluster_k > 1 ? p.cluster_k : 1);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.cluster_k > 1 ? 2 : 1;
    e = cudaLaunchKernelEx(&cfg, fn, tm_q, tm_k, tm_v, p, pp);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "ht_tree_attention (tcgen05, tile pairs, clusters of %d): %s", p.cluster_k > 1 ? p.cluster_k : 1,
                    cudaGetErrorString(e));
    }
    return HT_OK;
}

}  // namespace ht
