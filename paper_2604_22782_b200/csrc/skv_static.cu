// skv_decode_attn_static: decode attention for callers that cannot allocate device memory
// (see include/skv.h).  The split-K scratch is a fixed array in the library image.
#include "../../include/skv.h"

#include <cuda_runtime.h>
#include <mutex>

// The scratch itself.  In host code this name is only a handle for the runtime's symbol calls, not
// a device address: it must never be passed to a kernel directly.
static __device__ __align__(256) unsigned char g_static_scratch[SKV_STATIC_SCRATCH_BYTES];

namespace {

constexpr int MAX_DEVICES = 64;
std::mutex g_lock;
void *g_scratch_addr[MAX_DEVICES];   // device address of g_static_scratch on each device, once looked up

// Device address of the scratch array on the current device; looked up once per device, with that
// device current.  Returns nullptr if the runtime refuses.
void *scratch_address()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
        (void)cudaGetLastError();
        return nullptr;
    }
    std::lock_guard<std::mutex> hold(g_lock);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_scratch_addr[dev] = ptr;
    }
    return g_scratch_addr[dev];
}

}  // namespace

extern "C" int skv_decode_attn_static(skv_cache *cache, int layer, const void *Q, const int32_t *page_table,
                                      const int32_t *seq_lens, void *out, int batch, int q_heads, int pt_stride,
                                      float scale, void *stream)
{
    if (!cache) return SKV_ERR_ARG;
    size_t need = 0;
    const int rc = skv_decode_workspace_bytes(cache, batch, q_heads, &need);
    if (rc) return rc;
    if (need > SKV_STATIC_SCRATCH_BYTES) return SKV_ERR_TOO_LARGE;
    void *scratch = scratch_address();
    if (!scratch) return SKV_ERR_CUDA;
    // The same two launches as skv_decode_attn, on the library's own area.  Nothing in the area has to be
    // cleared: the merge kernel only reads slots that the split-K launch of the same call has just
    // written.  Calls on one stream may follow each other without anything in between because a split-K
    // launch writes its first partial only after its wait on the kernel before it, i.e. after the merge
    // of the previous call has read the area.
    return skv_decode_attn(cache, layer, Q, page_table, seq_lens, out, batch, q_heads, pt_stride, scale, scratch,
                           SKV_STATIC_SCRATCH_BYTES, stream);
}
