// FP8 pages -> bf16 pages of the same owner layer in a scratch area, for the pre-fill attention on the tensor
// cores' bf16 path: the pages that a call's sequences reach are turned back into bf16 (code value x the
// row's scale, rounded to nearest even) in the bf16 page layout, and the bf16 kernel then runs on the scratch.
// A prompt's attention is compute-bound (its bytes are read once per 128 query rows), so the extra pass
// over the pages costs a few per cent, where converting inside the attention kernel would put the
// conversions on the warps that already set its pace.
#include "skv_common.cuh"

namespace skv {

namespace {

constexpr int DQ_WARPS = 4;

// four E4M3 codes (one word) x scale -> four bf16 (two words)
__device__ __forceinline__ void dequant4(uint32_t codes, float scale, uint32_t &lo, uint32_t &hi)
{
    uint32_t h01, h23;
    e4m3x4_to_f16x2(codes, h01, h23);
    float f0, f1, f2, f3;
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}" : "=f"(f0), "=f"(f1) : "r"(h01));
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}" : "=f"(f2), "=f"(f3) : "r"(h23));
    lo = pack_bf16x2(f0 * scale, f1 * scale);
    hi = pack_bf16x2(f2 * scale, f3 * scale);
}

// One warp per (sequence b, page pg of it, kv head h): grid.x covers the pages of the longest sequence.
template <int D>
__global__ void __launch_bounds__(DQ_WARPS * 32) dequant_pages_kernel(DequantParams p)
{
    constexpr int FB = fp8_block_bytes(D), HALF = half_bytes(D), CH = D / 8;
    __shared__ __align__(16) uint8_t blk[DQ_WARPS][FB];
    pdl_trigger();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.z, h = blockIdx.y;
    const int pg = (int)blockIdx.x * DQ_WARPS + warp;
    int n_b = __ldg(p.seq_lens + b);
    if ((int64_t)n_b > (int64_t)p.pt_stride * PAGE) n_b = p.pt_stride * PAGE;        // (flagged by the attention kernel)
    if (pg >= (n_b + PAGE - 1) / PAGE) return;                                        // warp-uniform
    const int id = __ldg(p.page_table + (int64_t)b * p.pt_stride + pg);
    if (id < 0 || (int64_t)id >= p.max_pages) return;                                 // (flagged by the attention kernel)
    const uint4 *src = reinterpret_cast<const uint4 *>(p.fp8_base + (int64_t)id * p.fp8_page_stride + (int64_t)h * FB);
    uint4 *mine = reinterpret_cast<uint4 *>(blk[warp]);
    for (int i = lane; i < FB / 16; i += 32) mine[i] = __ldg(src + i);
    __syncwarp();
    const uint8_t *s = blk[warp];
    const float *ks = reinterpret_cast<const float *>(s + fp8_ks_off(D)), *vs = reinterpret_cast<const float *>(s + fp8_vs_off(D));
    uint4 *dst = reinterpret_cast<uint4 *>(p.bf16_base + (int64_t)id * p.bf16_page_stride + (int64_t)h * block_bytes(D));
    // 16-byte unit u of a bf16 half = (chunk c = u / 16: dims 8c .. 8c+7, token t = u % 16)
    for (int u = lane; u < CH * PAGE; u += 32) {
        const int c = u / PAGE, t = u % PAGE;
        // K: the 8 dims are 8 consecutive bytes of the token's 16-dim piece
        const uint2 kc = *reinterpret_cast<const uint2 *>(s + fp8_k_pos(D, t, 8 * c));
        uint4 o;
        dequant4(kc.x, ks[t], o.x, o.y);
        dequant4(kc.y, ks[t], o.z, o.w);
        dst[u] = o;
        // V: dim-major codes, byte (d, t) at d * 16 + t
        const uint8_t *vcol = s + fp8_v_off(D) + (8 * c) * PAGE + t;
        const uint32_t v0 = (uint32_t)vcol[0] | ((uint32_t)vcol[PAGE] << 8) | ((uint32_t)vcol[2 * PAGE] << 16) | ((uint32_t)vcol[3 * PAGE] << 24);
        const uint32_t v1 = (uint32_t)vcol[4 * PAGE] | ((uint32_t)vcol[5 * PAGE] << 8) | ((uint32_t)vcol[6 * PAGE] << 16) |
                            ((uint32_t)vcol[7 * PAGE] << 24);
        dequant4(v0, vs[t], o.x, o.y);
        dequant4(v1, vs[t], o.z, o.w);
        dst[HALF / 16 + u] = o;
    }
}

}  // namespace

cudaError_t launch_dequant_pages(const DequantParams &p, int D, int max_pages_per_seq, cudaStream_t s)
{
    if (max_pages_per_seq <= 0) return cudaSuccess;
    const dim3 grid((unsigned)((max_pages_per_seq + DQ_WARPS - 1) / DQ_WARPS), (unsigned)p.Hkv, (unsigned)p.B);
    if (D == 128) dequant_pages_kernel<128><<<grid, DQ_WARPS * 32, 0, s>>>(p);
    else if (D == 64) dequant_pages_kernel<64><<<grid, DQ_WARPS * 32, 0, s>>>(p);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace skv
