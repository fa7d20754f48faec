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

// ---- FP8 pages -----------------------------------------------------------------------------
// One warp per (token, kv head); grid.y picks K or V, grid.z the owner layer.  The row's D values
// are spread over the lanes (D/32 each); amax by shuffles; scale = amax / 448, codes =
// E4M3(x * (448 / amax)) round-to-nearest-even, saturating; every step a single fp32 operation.
__global__ void __launch_bounds__(COPY_THREADS) append_fp8_kernel(AppendFp8Params p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * COPY_THREADS + threadIdx.x) >> 5;
    if (warp >= p.n_tokens * p.Hkv) return;
    const int64_t tok = warp / p.Hkv;
    const int h = (int)(warp - tok * p.Hkv);
    const int64_t slot = p.slot_map[tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (h == 0 && lane == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;
    const int64_t layer = blockIdx.z;
    const int D = p.D, PER = D / 32;                  // 4 values per lane at D = 128, 2 at D = 64
    const uint16_t *src = (which ? p.V : p.K) + ((layer * p.n_tokens + tok) * p.Hkv + h) * D + lane * PER;
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    if (PER == 4) {
        const uint2 w = __ldg(reinterpret_cast<const uint2 *>(src));
        x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    } else {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(src));
        x[0] = bf16_lo(w); x[1] = bf16_hi(w);
    }
    float amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
    const float inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    const uint32_t c01 = pack_e4m3x2(__fmul_rn(x[0], inv), __fmul_rn(x[1], inv));
    const uint32_t c23 = pack_e4m3x2(__fmul_rn(x[2], inv), __fmul_rn(x[3], inv));
    uint8_t *blk = p.layer_base + layer * p.layer_stride + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    if (which == 0) {                                  // K: a lane's dims are neighbours inside one 16-byte piece
        uint8_t *dst = blk + fp8_k_pos(D, off, lane * PER);
        if (PER == 4) *reinterpret_cast<uint32_t *>(dst) = c01 | (c23 << 16);
        else *reinterpret_cast<uint16_t *>(dst) = (uint16_t)c01;
    } else {                                           // V: dim-major, this token's column
        uint8_t *dst = blk + fp8_v_off(D) + (lane * PER) * PAGE + off;
        dst[0] = (uint8_t)(c01 & 0xFF);
        dst[PAGE] = (uint8_t)(c01 >> 8);
        if (PER == 4) {
            dst[2 * PAGE] = (uint8_t)(c23 & 0xFF);
            dst[3 * PAGE] = (uint8_t)(c23 >> 8);
        }
    }
    if (lane == 0)
        *reinterpret_cast<float *>(blk + (which ? fp8_vs_off(D) : fp8_ks_off(D)) + 4 * off) = __fdiv_rn(amax, 448.f);
}

// read-back: codes as [n][Hkv][D] for both K and V, scales as [n][Hkv]
__global__ void __launch_bounds__(COPY_THREADS) gather_fp8_kernel(GatherFp8Params p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * COPY_THREADS + threadIdx.x) >> 5;
    if (warp >= p.n * p.Hkv) return;
    const int64_t tok = warp / p.Hkv;
    const int h = (int)(warp - tok * p.Hkv);
    const int64_t slot = p.slot_ids[tok];
    if (slot < 0) return;
    if (slot >= p.n_slots) {
        if (h == 0 && lane == 0) atomicOr(p.status, STATUS_BOUNDS);
        return;
    }
    const int64_t page = slot / PAGE;
    const int off = (int)(slot - page * PAGE);
    const int which = blockIdx.y;
    const int D = p.D;
    const uint8_t *blk = p.layer_base + page * p.page_stride + (int64_t)h * fp8_block_bytes(D);
    uint8_t *out = (which ? p.V_codes : p.K_codes) + (tok * p.Hkv + h) * D;
    for (int d = lane; d < D; d += 32)
        out[d] = which ? blk[fp8_v_off(D) + d * PAGE + off] : blk[fp8_k_pos(D, off, d)];
    if (lane == 0)
        (which ? p.V_scales : p.K_scales)[tok * p.Hkv + h] =
            *reinterpret_cast<const float *>(blk + (which ? fp8_vs_off(D) : fp8_ks_off(D)) + 4 * off);
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

namespace skv {

cudaError_t launch_append_fp8(const AppendFp8Params &p, int n_layers, cudaStream_t s)
{
    const int64_t warps = p.n_tokens * p.Hkv;
    const int64_t blocks = (warps * 32 + 255) / 256;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll || n_layers < 1 || n_layers > 65535) return cudaErrorInvalidConfiguration;
    append_fp8_kernel<<<dim3((unsigned)blocks, 2, (unsigned)n_layers), 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_gather_fp8(const GatherFp8Params &p, cudaStream_t s)
{
    const int64_t warps = p.n * p.Hkv;
    const int64_t blocks = (warps * 32 + 255) / 256;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    gather_fp8_kernel<<<dim3((unsigned)blocks, 2), 256, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace skv
