// ht_tree_attention_static: tree attention for callers that cannot allocate.
//
// Some hosts of this library have no way to hand it scratch memory: code that runs where
// cudaMalloc is off limits (inside a region of the application that must not touch the
// allocator, a plugin interface that passes only inputs and outputs, a process whose
// memory pool is fully committed up front).  For them this entry point runs the split-KV
// fp32-ALU attention kernel with its split partials kept in a fixed array that is part of
// the library image, so the call needs nothing but its inputs and outputs.
//
// The array lives in every GPU context that loads the library, from load until exit,
// whether or not this entry point is ever called; that is why its size is modest and
// fixed.  All calls share it and it keeps whatever the last call left: nothing in it has
// to start at zero (every partial that the merge kernel reads is written by the main
// kernel of the same call first), but two calls that overlap on the GPU -- different
// streams, or different host threads -- race on it.  Serialise them.
#include <mutex>

#include "ht_common.cuh"

namespace ht {

// Split partials of one call: (max, sum, D outputs) in fp32 per (row, head, split).
static __device__ __align__(256) unsigned char g_static_scratch[HT_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_setup_mutex;
static void *g_scratch_addr[kMaxDevices];   // device address of g_static_scratch, per device
static bool g_scratch_ready[kMaxDevices];

// In host code the name g_static_scratch is only a handle for the runtime; the address a
// kernel can use has to be asked for, once per device, with that device current.
static int scratch_address(void **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(HT_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(HT_ERR_UNSUPPORTED, "device index %d out of range", dev);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ready[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || p == nullptr)
            return fail(HT_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_addr[dev];
    return HT_OK;
}

}  // namespace ht

using namespace ht;

extern "C" int ht_tree_attention_static(const ht_attn_desc *desc, const void *q, const void *k_cache,
                                        const void *v_cache, const int32_t *kv_len, const int32_t *parent,
                                        void *out, int32_t *status, void *stream) {
    int rc = check_attn_desc(desc);
    if (rc != HT_OK) return rc;
    if (desc->B == 0 || desc->N == 0) return HT_OK;
    if (!q || !k_cache || !v_cache || !kv_len || !parent || !out || !status)
        return fail(HT_ERR_INVALID_ARG, "NULL pointer");
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out))
        return fail(HT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    const size_t need = attn_simt_workspace(*desc, nullptr);
    if (need > (size_t)HT_STATIC_SCRATCH_BYTES)
        return fail(HT_ERR_WORKSPACE,
                    "this problem needs %zu bytes of split scratch but the built-in scratch holds %zu: "
                    "lower num_splits (1 needs none) or call ht_tree_attention with a workspace",
                    need, (size_t)HT_STATIC_SCRATCH_BYTES);
    // The array's address is looked up for the current device: the buffers must live there too (a kernel given
    // another device's address would write through it into the wrong memory).
    int dev = -1;
    cudaPointerAttributes attr;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaPointerGetAttributes(&attr, q) != cudaSuccess) {
        cudaGetLastError();
        return fail(HT_ERR_CUDA, "cannot tell which device the current one is, or which one holds q");
    }
    if (attr.type == cudaMemoryTypeDevice && attr.device != dev)
        return fail(HT_ERR_INVALID_ARG, "q lives on device %d but device %d is current: make the buffers' device current", attr.device, dev);
    void *scratch = nullptr;
    rc = scratch_address(&scratch);
    if (rc != HT_OK) return rc;
    return launch_attn_simt(*desc, q, k_cache, v_cache, kv_len, parent, out, scratch,
                            (size_t)HT_STATIC_SCRATCH_BYTES, status, static_cast<cudaStream_t>(stream));
}
