// Rotary position embedding at the tree's position ids and placement of the new K / V rows
// behind the context (the step ahead of tree attention).  The flattened tree keeps "the
// original positional indices of each token" (Section "Tree attention"; pseudo states: position
// id j + i, Section "Training stage"); the paper's models (LLaMA-2 / Vicuna, Section "Setup")
// encode positions with the rotary embedding in the half-split pairing (feature i with
// feature i + D/2, angle pos * base^(-2i/D)).
//
// One block per (sequence, row): D/2 threads compute the row's cosines and sines once -- the
// angle in fp64, because a position of tens of thousands times a frequency near 1 loses the
// low bits that matter in fp32 -- and the block then rotates all query heads and KV heads of
// the row with 16-byte loads and stores, writing q to q_out and K, V to cache row kv_len + r.
// A few hundred KB per call: latency-bound, one launch.
#include "ht_common.cuh"

namespace ht {

template <typename T, int D>
__global__ void __launch_bounds__(128)
rope_kv_append_kernel(const T *__restrict__ q_in, const T *__restrict__ k_in, const T *__restrict__ v_in,
                      const int32_t *__restrict__ pos, const int32_t *__restrict__ kv_len, double log2_base,
                      T *__restrict__ q_out, T *__restrict__ k_cache, T *__restrict__ v_cache, int N, int Hq, int Hkv,
                      int cap, long long stride_b, long long stride_h, int32_t *__restrict__ status, const PageMap pm) {
    // lets a kernel that is serialized programmatically behind this one (the attention call) set itself up meanwhile
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int VE = Vec16<T>::n, HALF = D / 2, VPH = HALF / VE;     // 16-byte vectors per half row
    __shared__ float s_cos[HALF], s_sin[HALF];
    const int b = blockIdx.x / N, r = blockIdx.x - b * N;
    const int L = kv_len[b];
    const bool bad = L < 0 || (long long)L + N > cap;
    // paged cache: the status words were zeroed ahead of the launch and any block may report a bad page
    if (r == 0 && threadIdx.x == 0 && (bad || !pm.table)) status[b] = bad ? HT_STATUS_BAD_LEN : HT_STATUS_OK;
    if (bad) return;
    // where cache row L + r of this sequence starts, short of the head's offset
    long long row_off = (long long)b * stride_b + (long long)(L + r) * D;
    bool no_page = false;
    if (pm.table) {
        const int page = pm.table[(size_t)b * pm.max_pages + ((L + r) >> pm.shift)];
        no_page = (unsigned)page >= (unsigned)pm.n_pages;
        if (no_page && threadIdx.x == 0) status[b] = HT_STATUS_BAD_PAGE;   // the row's K and V are not stored; its q is rotated
        row_off = (long long)page * pm.page_stride + (long long)((L + r) & ((1 << pm.shift) - 1)) * D;
    }
    const double p = (double)pos[(size_t)b * N + r];
    for (int i = threadIdx.x; i < HALF; i += blockDim.x) {
        double s, c;
        sincos(p * exp2(-2.0 * i / D * log2_base), &s, &c);
        s_cos[i] = (float)c;
        s_sin[i] = (float)s;
    }
    __syncthreads();
    // work items: (head, vector within the half row); query heads first, then K heads, then V heads
    const int items = (Hq + 2 * Hkv) * VPH;
    for (int it = threadIdx.x; it < items; it += blockDim.x) {
        const int h = it / VPH, vx = it - h * VPH;
        const T *src;
        T *dst;
        bool rotate = true;
        if (h < Hq) {
            src = q_in + (((size_t)b * N + r) * Hq + h) * D;
            dst = q_out + (((size_t)b * N + r) * Hq + h) * D;
        } else if (no_page) {
            continue;
        } else if (h < Hq + Hkv) {
            src = k_in + (((size_t)b * N + r) * Hkv + (h - Hq)) * D;
            dst = k_cache + row_off + (size_t)(h - Hq) * stride_h;
        } else {
            src = v_in + (((size_t)b * N + r) * Hkv + (h - Hq - Hkv)) * D;
            dst = v_cache + row_off + (size_t)(h - Hq - Hkv) * stride_h;
            rotate = false;
        }
        const uint4 lo_raw = *reinterpret_cast<const uint4 *>(src + vx * VE);
        const uint4 hi_raw = *reinterpret_cast<const uint4 *>(src + HALF + vx * VE);
        if (!rotate) {
            *reinterpret_cast<uint4 *>(dst + vx * VE) = lo_raw;
            *reinterpret_cast<uint4 *>(dst + HALF + vx * VE) = hi_raw;
            continue;
        }
        float lo[VE], hi[VE];
        unpack16<T>(lo_raw, lo);
        unpack16<T>(hi_raw, hi);
        T out_lo[VE], out_hi[VE];
#pragma unroll
        for (int e = 0; e < VE; ++e) {
            const float c = s_cos[vx * VE + e], s = s_sin[vx * VE + e];
            out_lo[e] = from_float<T>(lo[e] * c - hi[e] * s);
            out_hi[e] = from_float<T>(hi[e] * c + lo[e] * s);
        }
        *reinterpret_cast<uint4 *>(dst + vx * VE) = *reinterpret_cast<const uint4 *>(out_lo);
        *reinterpret_cast<uint4 *>(dst + HALF + vx * VE) = *reinterpret_cast<const uint4 *>(out_hi);
    }
}

template <typename T>
static int launch_t(const ht_attn_desc &d, const void *q_in, const void *k_in, const void *v_in, const int32_t *pos,
                    const int32_t *kv_len, float base, void *q_out, void *kc, void *vc, int32_t *status, cudaStream_t s,
                    const PageMap &pm) {
    const long long sh = pm.table ? pm.head_stride : (d.kv_stride_h ? d.kv_stride_h : (long long)d.cap * d.D);
    const long long sb = d.kv_stride_b ? d.kv_stride_b : (long long)d.Hkv * d.cap * d.D;
    const double l2b = log2((double)base);
    const unsigned blocks = (unsigned)(d.B * d.N);
#define HT_ROPE_LAUNCH(DD)                                                                                                   \
    rope_kv_append_kernel<T, DD><<<blocks, 128, 0, s>>>(static_cast<const T *>(q_in), static_cast<const T *>(k_in),         \
                                                        static_cast<const T *>(v_in), pos, kv_len, l2b, static_cast<T *>(q_out), \
                                                        static_cast<T *>(kc), static_cast<T *>(vc), d.N, d.Hq, d.Hkv, d.cap, sb, sh, status, pm)
    if (d.D == 64) HT_ROPE_LAUNCH(64);
    else HT_ROPE_LAUNCH(128);
#undef HT_ROPE_LAUNCH
    return check_launch("ht_rope_kv_append");
}

int launch_rope(const ht_attn_desc &d, const void *q_in, const void *k_in, const void *v_in, const int32_t *pos,
                const int32_t *kv_len, float base, void *q_out, void *kc, void *vc, int32_t *status, cudaStream_t s,
                const PageMap &pm) {
    if (pm.table) {
        const cudaError_t e = cudaMemsetAsync(status, 0, (size_t)d.B * sizeof(int32_t), s);
        if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    }
    switch (d.dtype) {
        case HT_F32: return launch_t<float>(d, q_in, k_in, v_in, pos, kv_len, base, q_out, kc, vc, status, s, pm);
        case HT_F16: return launch_t<__half>(d, q_in, k_in, v_in, pos, kv_len, base, q_out, kc, vc, status, s, pm);
        default: return launch_t<__nv_bfloat16>(d, q_in, k_in, v_in, pos, kv_len, base, q_out, kc, vc, status, s, pm);
    }
}

}  // namespace ht
