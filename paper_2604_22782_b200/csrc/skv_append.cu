// "Update" of Algorithm 2: scatter the new tokens' K,V rows into the pages of an
// owner layer, and the inverse read-back.  Pure 16-byte copies, bit-exact.
#include "skv_common.cuh"

namespace skv {

namespace {

constexpr int COPY_THREADS = 256;

// One thread moves one 16-byte chunk (8 bf16 of one head of one token); grid.y picks K or V,
// grid.z the owner layer when one launch serves several.
// Reads are fully coalesced along the token row; writes land 16 bytes apart at
// a stride of PAGE*16 bytes (the chunk-major page layout).
__global__ void __launch_bounds__(COPY_THREADS) append_kernel(AppendParams p)
{
    const int CH = p.D / CHUNK_ELEMS;
    const int64_t row_chunks = (int64_t)p.Hkv * CH;
    const int64_t idx = (int64_t)blockIdx.x * COPY_THREADS + threadIdx.x;
    if (idx >= p.n_tokens * row_chunks) return;
    const int64_t tok = idx / row_chunks;
    const int rem = (int)(idx - tok * row_chunks);
    const int h = rem / CH, c = rem - h * CH;
    const int64_t slot = p.slot_map[tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (rem == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;                       // 0 = K, 1 = V
    const int64_t layer = blockIdx.z;                   // owner layers of one launch, consecutive in the pool
    const uint4 *src = (which ? p.V : p.K) + layer * p.n_tokens * row_chunks;
    uint8_t *dst = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)h * block_bytes(p.D) +
                   (int64_t)which * half_bytes(p.D) + ((int64_t)c * PAGE + off) * 16;
    *reinterpret_cast<uint4 *>(dst) = __ldg(src + idx);
}

__global__ void __launch_bounds__(COPY_THREADS) gather_kernel(GatherParams p)
{
    const int CH = p.D / CHUNK_ELEMS;
    const int64_t row_chunks = (int64_t)p.Hkv * CH;
    const int64_t idx = (int64_t)blockIdx.x * COPY_THREADS + threadIdx.x;
    if (idx >= p.n * row_chunks) return;
    const int64_t tok = idx / row_chunks;
    const int rem = (int)(idx - tok * row_chunks);
    const int h = rem / CH, c = rem - h * CH;
    const int64_t slot = p.slot_ids[tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (rem == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;
    const uint8_t *src = p.layer_base + page * p.page_stride + (int64_t)h * block_bytes(p.D) +
                         (int64_t)which * half_bytes(p.D) + ((int64_t)c * PAGE + off) * 16;
    uint4 *dst = which ? p.V_out : p.K_out;
    dst[idx] = *reinterpret_cast<const uint4 *>(src);
}

}  // namespace

// n_layers consecutive owner layers (grid.z) take rows from K/V [n_layers][n_tokens][Hkv][D] with one slot map
cudaError_t launch_append(const AppendParams &p, int n_layers, cudaStream_t s)
{
    const int64_t chunks = p.n_tokens * p.Hkv * (p.D / CHUNK_ELEMS);
    const int64_t blocks = (chunks + COPY_THREADS - 1) / COPY_THREADS;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    if (n_layers < 1 || n_layers > 65535) return cudaErrorInvalidConfiguration;
    append_kernel<<<dim3((unsigned)blocks, 2, (unsigned)n_layers), COPY_THREADS, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_gather(const GatherParams &p, cudaStream_t s)
{
    const int64_t chunks = p.n * p.Hkv * (p.D / CHUNK_ELEMS);
    const int64_t blocks = (chunks + COPY_THREADS - 1) / COPY_THREADS;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    gather_kernel<<<dim3((unsigned)blocks, 2), COPY_THREADS, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace skv
