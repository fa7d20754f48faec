// "Update" of Algorithm 2: scatter the new tokens' K,V rows into the pages of an
// owner layer, and the inverse read-back.  Pure 16-byte copies, bit-exact.
#include "skv_common.cuh"

namespace skv {

namespace {

constexpr int COPY_THREADS = 256;

// One thread moves one 16-byte chunk (8 bf16 of one head of one token); grid.y picks K or V,
// grid.z the owner layer when one launch serves several.  A warp takes 16 tokens x 2 adjacent
// chunks of one head: lane = token (low 4 bits) + 16 * chunk parity, so that the reads of a token's
// two chunks fill one 32-byte sector and, when the 16 tokens sit in consecutive slots of a page
// (pre-fill), each half-warp writes one contiguous 256-byte run of the chunk-major page layout.
struct CopyCoord {
    int64_t tok;
    int h, c;
    bool in_range;
};

__device__ __forceinline__ CopyCoord coord_of(int64_t n_tok, int Hkv, int CH)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * COPY_THREADS + threadIdx.x) >> 5;
    const int pairs = CH / 2;                             // head_dim is 64 or 128: CH is even
    const int64_t per_group = (int64_t)Hkv * pairs;       // warps per group of 16 tokens
    const int64_t g16 = warp / per_group;
    const int rem = (int)(warp - g16 * per_group);
    CopyCoord k;
    k.h = rem / pairs;
    k.c = 2 * (rem - k.h * pairs) + (lane >> 4);
    k.tok = g16 * 16 + (lane & 15);
    k.in_range = k.tok < n_tok;
    return k;
}

__global__ void __launch_bounds__(COPY_THREADS) append_kernel(AppendParams p)
{
    const int CH = p.D / CHUNK_ELEMS;
    const CopyCoord k = coord_of(p.n_tokens, p.Hkv, CH);
    if (!k.in_range) return;
    const int64_t slot = p.slot_map[k.tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (k.h == 0 && k.c == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;                       // 0 = K, 1 = V
    const int64_t layer = blockIdx.z;                   // owner layers of one launch, consecutive in the pool
    const int64_t row_chunks = (int64_t)p.Hkv * CH;
    const uint4 *src = (which ? p.V : p.K) + (layer * p.n_tokens + k.tok) * row_chunks + (int64_t)k.h * CH + k.c;
    uint8_t *dst = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)k.h * block_bytes(p.D) +
                   (int64_t)which * half_bytes(p.D) + ((int64_t)k.c * PAGE + off) * 16;
    *reinterpret_cast<uint4 *>(dst) = __ldg(src);
}

__global__ void __launch_bounds__(COPY_THREADS) gather_kernel(GatherParams p)
{
    const int CH = p.D / CHUNK_ELEMS;
    const CopyCoord k = coord_of(p.n, p.Hkv, CH);
    if (!k.in_range) return;
    const int64_t slot = p.slot_ids[k.tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (k.h == 0 && k.c == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;
    const uint8_t *src = p.layer_base + page * p.page_stride + (int64_t)k.h * block_bytes(p.D) +
                         (int64_t)which * half_bytes(p.D) + ((int64_t)k.c * PAGE + off) * 16;
    uint4 *dst = (which ? p.V_out : p.K_out) + (k.tok * p.Hkv + k.h) * CH + k.c;
    *dst = *reinterpret_cast<const uint4 *>(src);
}

// blocks needed for n tokens: one warp per (16 tokens, head, chunk pair)
int64_t copy_blocks(int64_t n, int Hkv, int D)
{
    const int64_t warps = ((n + 15) / 16) * Hkv * (D / CHUNK_ELEMS / 2);
    return (warps * 32 + COPY_THREADS - 1) / COPY_THREADS;
}

}  // namespace

// n_layers consecutive owner layers (grid.z) take rows from K/V [n_layers][n_tokens][Hkv][D] with one slot map
cudaError_t launch_append(const AppendParams &p, int n_layers, cudaStream_t s)
{
    const int64_t blocks = copy_blocks(p.n_tokens, p.Hkv, p.D);
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    if (n_layers < 1 || n_layers > 65535) return cudaErrorInvalidConfiguration;
    append_kernel<<<dim3((unsigned)blocks, 2, (unsigned)n_layers), COPY_THREADS, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_gather(const GatherParams &p, cudaStream_t s)
{
    const int64_t blocks = copy_blocks(p.n, p.Hkv, p.D);
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    gather_kernel<<<dim3((unsigned)blocks, 2), COPY_THREADS, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace skv
