// KV compaction: the accepted path's K/V rows are moved directly behind the context, in
// place, for every layer and KV head in one launch (Fig. 1 caption and Section "Inference
// stage" imply it: verification runs against a KV cache, and only accepted tokens may
// stay in it).
//
// The data are tiny (a few rows per head), so the kernel is a chain of dependent round trips
// to memory: lengths -> path -> rows -> stores.  A block takes one (layer, sequence) and a
// contiguous share of its 2*Hkv pairs, and moves as many pairs per pass as its registers hold
// (16 vectors per thread; 8 in the fused verification kernel, which keeps its registers for four blocks per SM), all loads of a pass in flight together.  The work of a block is
// compact_item (compact.cuh), which the fused verification kernel runs as well.
#include "compact.cuh"

namespace ht {

__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const CompactArgs c) {
    __shared__ CompactSmem sm;
    // The launch is serialized programmatically behind the kernel before it in the stream (the verification, as a
    // rule): the blocks are in place while that kernel finishes, and read what it wrote from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int idx = blockIdx.x;
    const int grp = idx % c.groups;
    idx /= c.groups;
    const int b = idx % c.B;
    const int layer = idx / c.B;
    compact_item<16>(c, sm, layer, b, grp, c.accept_len[b], c.kv_len[b]);
}

CompactArgs make_compact_args(void *kc, void *vc, const ht_cache_desc &d, const int32_t *kv_len, const int32_t *accept_len,
                              const int32_t *accept_path, int max_path, int32_t *new_kv_len, int32_t *status,
                              const PageMap &pm_elems, int blocks) {
    const long long e = elem_bytes(d.dtype);
    CompactArgs c{};
    c.pm = pm_elems;                       // the kernels take the page strides in bytes
    c.pm.page_stride *= e;
    c.pm.head_stride *= e;
    c.k_cache = static_cast<unsigned char *>(kc);
    c.v_cache = static_cast<unsigned char *>(vc);
    c.layers = d.layers; c.B = d.B; c.Hkv = d.Hkv; c.cap = d.cap; c.N = d.N;
    c.row_bytes = d.D * (int)e;
    c.stride_h_b = c.pm.table ? c.pm.head_stride : (d.stride_h ? d.stride_h : (long long)d.cap * d.D) * e;
    c.stride_b_b = (d.stride_b ? d.stride_b : (long long)d.Hkv * d.cap * d.D) * e;
    c.stride_layer_b = (d.stride_layer ? d.stride_layer : (c.pm.table ? (long long)c.pm.n_pages * pm_elems.page_stride : (long long)d.B * d.Hkv * d.cap * d.D)) * e;
    c.kv_len = kv_len; c.accept_len = accept_len; c.accept_path = accept_path; c.max_path = max_path;
    c.new_kv_len = new_kv_len; c.status = status;
    const long long lb = (long long)d.layers * d.B;
    long long groups = blocks / lb;
    if (groups < 1) groups = 1;
    if (groups > 2ll * d.Hkv) groups = 2ll * d.Hkv;
    c.groups = (int)groups;
    return c;
}

int launch_compact(void *kc, void *vc, const ht_cache_desc &d, const int32_t *kv_len,
                   const int32_t *accept_len, const int32_t *accept_path, int max_path,
                   int32_t *new_kv_len, int32_t *status, cudaStream_t s, const PageMap &pm_elems) {
    const CompactArgs c = make_compact_args(kc, vc, d, kv_len, accept_len, accept_path, max_path, new_kv_len, status, pm_elems,
                                            2 * 148 + d.layers * d.B - 1);   // enough blocks to occupy the GPU about twice over
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((long long)d.layers * d.B * c.groups));
    cfg.blockDim = dim3(kCompactThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, compact_kernel, c);
    if (le != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "ht_kv_compact: %s", cudaGetErrorString(le));
    }
    return HT_OK;
}

}  // namespace ht
