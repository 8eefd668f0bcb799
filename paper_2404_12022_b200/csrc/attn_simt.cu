// Tree attention on the fp32 ALUs (Section "Tree attention"; pseudo rows: Section
// "Training stage").  This is the kernel for fp32 inputs -- where the stated tolerance of
// 1e-5 rules out reduced-precision tensor-core products -- and the fallback for shapes
// the tensor-core kernel does not take.  It is a split-KV design with online softmax:
//
//   grid  = (row blocks of 8 query rows, Hq, B * splits)
//   block = 8 warps; warp w owns query row r = 8*blockIdx.x + w of head blockIdx.y
//   loop  : the block stages 32 keys (K and V rows, converted to fp32) into shared memory
//           with coalesced 16-byte loads; lane j scores key j against the warp's q
//           (K rows are padded by one float, so the 32 lanes hit 32 banks); the row's
//           visibility of tree key c is bit c of its ancestor bitmask, built once per
//           warp by walking parent[]; running max / sum are warp-shuffle reductions;
//           O += P.V with each lane owning D/32 output features.
//   end   : splits == 1 writes out = O / l; otherwise (m, l, O) partials go to the
//           workspace and a second kernel merges them by log-sum-exp.
#include "ht_common.cuh"

namespace ht {

constexpr int kRows = 8;          // query rows (warps) per block
constexpr int kKeys = 32;         // keys per staged tile
constexpr int kMaxWords = 32;     // ancestor bitmask words per row -> N <= 1024
constexpr float kLog2e = 1.4426950408889634f;

struct SimtParams {
    const void *q, *kc, *vc;
    void *out;
    float *part;                  // [B, N, Hq, splits, 2 + D] when splits > 1
    const int32_t *kv_len, *parent;
    int32_t *status;
    int B, N, Hq, Hkv, D, cap, splits;
    long long stride_b, stride_h; // elements
    float scale_log2;
};

template <typename T, int D>
__global__ void __launch_bounds__(kRows * 32)
attn_simt_kernel(SimtParams p) {
    constexpr int DPL = D / 32;                       // output features per lane
    constexpr int VE = Vec16<T>::n;
    __shared__ float Ks[kKeys][D + 1];
    __shared__ float Vs[kKeys][D];
    __shared__ float Qs[kRows][D];
    __shared__ uint32_t anc[kRows][kMaxWords];
    __shared__ int s_bad;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y;
    const int b = blockIdx.z / p.splits;
    const int split = blockIdx.z - b * p.splits;
    const int r = blockIdx.x * kRows + warp;
    const int N = p.N;
    const int L = p.kv_len[b];
    const int32_t *par = p.parent + (size_t)b * N;

    // Legality of this sequence's inputs; every block of the sequence comes to the same decision.
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    for (int c = threadIdx.x; c < N; c += blockDim.x)
        if (par[c] < -1 || par[c] >= c) s_bad = HT_STATUS_BAD_TREE;
    __syncthreads();
    int code = s_bad;
    if (L < 0 || (long long)L + N > p.cap) code = HT_STATUS_BAD_LEN;
    if (blockIdx.x == 0 && h == 0 && split == 0 && threadIdx.x == 0) p.status[b] = code;
    if (code != HT_STATUS_OK) return;

    const int words = (N + 31) >> 5;
    const bool row_ok = r < N;
    for (int w = lane; w < words; w += 32) anc[warp][w] = 0;
    __syncwarp();
    if (row_ok && lane == 0)
        for (int c = r; c >= 0; c = par[c]) anc[warp][c >> 5] |= 1u << (c & 31);
    const T *qrow = static_cast<const T *>(p.q) + (((size_t)b * N + (row_ok ? r : 0)) * p.Hq + h) * D;
    for (int x = lane; x < D; x += 32) Qs[warp][x] = to_float<T>(qrow[x]);
    __syncwarp();

    const int total = L + N;
    int chunk = (total + p.splits - 1) / p.splits;
    chunk = (chunk + kKeys - 1) / kKeys * kKeys;
    const int k_begin = split * chunk;
    const int k_end = min(total, k_begin + chunk);

    const int hk = h / (p.Hq / p.Hkv);
    const T *kbase = static_cast<const T *>(p.kc) + (size_t)b * p.stride_b + (size_t)hk * p.stride_h;
    const T *vbase = static_cast<const T *>(p.vc) + (size_t)b * p.stride_b + (size_t)hk * p.stride_h;

    float m = -INFINITY, l = 0.f, o[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) o[i] = 0.f;

    for (int k0 = k_begin; k0 < k_end; k0 += kKeys) {
        __syncthreads();                               // previous tile fully consumed
        constexpr int VPR = D / VE;                    // 16-byte vectors per row
        for (int t = threadIdx.x; t < kKeys * VPR; t += blockDim.x) {
            const int j = t / VPR, v = t - j * VPR;
            float kf[VE], vf[VE];
            if (k0 + j < k_end) {
                unpack16<T>(ld_nc16(kbase + (size_t)(k0 + j) * D + v * VE), kf);
                unpack16<T>(ld_nc16(vbase + (size_t)(k0 + j) * D + v * VE), vf);
            } else {
#pragma unroll
                for (int e = 0; e < VE; ++e) kf[e] = vf[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < VE; ++e) {
                Ks[j][v * VE + e] = kf[e];
                Vs[j][v * VE + e] = vf[e];
            }
        }
        __syncthreads();
        if (!row_ok) continue;

        const int key = k0 + lane;
        float s = 0.f;
#pragma unroll 8
        for (int x = 0; x < D; ++x) s = fmaf(Qs[warp][x], Ks[lane][x], s);
        s *= p.scale_log2;
        bool visible = key < k_end;
        if (visible && key >= L) {
            const int c = key - L;
            visible = (anc[warp][c >> 5] >> (c & 31)) & 1u;
        }
        s = visible ? s : -INFINITY;
        float tile_max = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, off));
        if (tile_max == -INFINITY) continue;           // nothing of this tile is visible to the row
        const float m_new = fmaxf(m, tile_max);
        const float corr = exp2f(m - m_new);           // m = -inf gives 0
        const float pj = visible ? exp2f(s - m_new) : 0.f;
        float psum = pj;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
        l = l * corr + psum;
        m = m_new;
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[i] *= corr;
#pragma unroll 4
        for (int j = 0; j < kKeys; ++j) {
            const float pb = __shfl_sync(0xffffffffu, pj, j);
#pragma unroll
            for (int i = 0; i < DPL; ++i) o[i] = fmaf(pb, Vs[j][lane + 32 * i], o[i]);
        }
    }
    if (!row_ok) return;
    if (p.splits == 1) {
        T *orow = static_cast<T *>(p.out) + (((size_t)b * N + r) * p.Hq + h) * D;
        const float inv = 1.f / l;
#pragma unroll
        for (int i = 0; i < DPL; ++i) orow[lane + 32 * i] = from_float<T>(o[i] * inv);
    } else {
        float *pp = p.part + ((((size_t)b * N + r) * p.Hq + h) * p.splits + split) * (2 + D);
        if (lane == 0) { pp[0] = m; pp[1] = l; }
#pragma unroll
        for (int i = 0; i < DPL; ++i) pp[2 + lane + 32 * i] = o[i];
    }
}

// One warp per (b, r, h): out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.
template <typename T, int D>
__global__ void __launch_bounds__(128)
attn_simt_combine_kernel(SimtParams p) {
    constexpr int DPL = D / 32;
    const long long item = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const long long items = (long long)p.B * p.N * p.Hq;
    if (item >= items) return;
    const int b = (int)(item / ((long long)p.N * p.Hq));
    if (p.status[b] != HT_STATUS_OK) return;           // written by the main kernel on this stream
    const float *pp = p.part + (size_t)item * p.splits * (2 + D);
    float M = -INFINITY;
    for (int s = 0; s < p.splits; ++s) M = fmaxf(M, pp[(size_t)s * (2 + D)]);
    float l = 0.f, o[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) o[i] = 0.f;
    for (int s = 0; s < p.splits; ++s) {
        const float *ps = pp + (size_t)s * (2 + D);
        const float ms = ps[0];
        if (ms == -INFINITY) continue;                 // the split saw nothing visible
        const float w = exp2f(ms - M);
        l += w * ps[1];
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[i] = fmaf(w, ps[2 + lane + 32 * i], o[i]);
    }
    T *orow = static_cast<T *>(p.out) + (size_t)item * D;
    const float inv = 1.f / l;
#pragma unroll
    for (int i = 0; i < DPL; ++i) orow[lane + 32 * i] = from_float<T>(o[i] * inv);
}

static int choose_splits(const ht_attn_desc &d) {
    if (d.num_splits > 0) return d.num_splits;
    const long long blocks = (long long)((d.N + kRows - 1) / kRows) * d.Hq * d.B;
    const long long target = 4 * 148;
    long long s = (target + blocks - 1) / blocks;
    const long long max_by_len = (d.cap + 255) / 256;   // at least ~256 keys per split
    if (s > max_by_len) s = max_by_len;
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    return (int)s;
}

size_t attn_simt_workspace(const ht_attn_desc &d, int *splits_out) {
    const int splits = choose_splits(d);
    if (splits_out) *splits_out = splits;
    if (splits == 1) return 0;
    return (size_t)d.B * d.N * d.Hq * splits * (2 + d.D) * sizeof(float);
}

template <typename T, int D>
static int launch_typed(const SimtParams &p, cudaStream_t s) {
    dim3 grid((p.N + kRows - 1) / kRows, p.Hq, p.B * p.splits);
    attn_simt_kernel<T, D><<<grid, kRows * 32, 0, s>>>(p);
    int rc = check_launch("ht_tree_attention (simt)");
    if (rc != HT_OK || p.splits == 1) return rc;
    const long long items = (long long)p.B * p.N * p.Hq;
    attn_simt_combine_kernel<T, D><<<(unsigned)((items + 3) / 4), 128, 0, s>>>(p);
    return check_launch("ht_tree_attention (simt combine)");
}

int launch_attn_simt(const ht_attn_desc &d, const void *q, const void *kc, const void *vc,
                     const int32_t *kv_len, const int32_t *parent, void *out, void *ws, size_t ws_bytes,
                     int32_t *status, cudaStream_t s) {
    SimtParams p;
    int splits;
    const size_t need = attn_simt_workspace(d, &splits);
    if (need > ws_bytes) return fail(HT_ERR_WORKSPACE, "workspace holds %zu bytes, %zu needed", ws_bytes, need);
    if (d.N > kMaxWords * 32) return fail(HT_ERR_UNSUPPORTED, "N = %d exceeds %d query rows", d.N, kMaxWords * 32);
    p.q = q; p.kc = kc; p.vc = vc; p.out = out; p.part = static_cast<float *>(ws);
    p.kv_len = kv_len; p.parent = parent; p.status = status;
    p.B = d.B; p.N = d.N; p.Hq = d.Hq; p.Hkv = d.Hkv; p.D = d.D; p.cap = d.cap; p.splits = splits;
    p.stride_h = d.kv_stride_h ? d.kv_stride_h : (long long)d.cap * d.D;
    p.stride_b = d.kv_stride_b ? d.kv_stride_b : (long long)d.Hkv * d.cap * d.D;
    const float scale = d.scale > 0.f ? d.scale : 1.f / sqrtf((float)d.D);
    p.scale_log2 = scale * kLog2e;
#define HT_DISPATCH(T)                                          \
    (d.D == 64 ? launch_typed<T, 64>(p, s) : launch_typed<T, 128>(p, s))
    switch (d.dtype) {
        case HT_F32: return HT_DISPATCH(float);
        case HT_F16: return HT_DISPATCH(__half);
        default: return HT_DISPATCH(__nv_bfloat16);
    }
#undef HT_DISPATCH
}

}  // namespace ht
