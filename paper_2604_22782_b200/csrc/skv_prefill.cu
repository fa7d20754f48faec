// Pre-fill attention (Section 3.1.1: the prompt's tokens are processed in parallel): Eq. (3.1)
// for many query tokens at once, each attending the cached tokens 0..pos of its sequence in the
// owner layer's pages (causal).  A dense contraction, unlike the decode step: one CTA owns a
// tile of 64 query rows (64/G tokens x the G query heads of one kv head, so that the group
// shares every K/V read), streams the pages it needs through a shared-memory ring of bulk
// copies, and keeps the online-softmax state of its rows in registers (flash attention).
// No split over the keys and therefore no workspace.
#include "skv_common.cuh"

#include <math.h>

namespace skv {

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int ROWS = 64;        // query rows per CTA: 4 warps x 16
constexpr int KB = 4;           // pages per key block (64 keys)
constexpr int NSTAGE = 3;       // key blocks in flight

template <int D>
__global__ void __launch_bounds__(128, 2) prefill_kernel(PrefillParams p, int G)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = block_bytes(D);          // K half + V half of one (page, kv head)
    constexpr int KS = D / 16;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int b = blockIdx.z, h = blockIdx.y;
    const int TQ = ROWS / G;                       // query tokens per tile

    const uint32_t base = smem_u32(smem_raw);
    const uint32_t pad = (128u - (base & 127u)) & 127u;
    const uint32_t ring = base + pad;
    const uint32_t bars = ring + NSTAGE * KB * BLOCK;
    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) mbar_init(bars + 8 * s, 1);
        fence_barrier_init();
    }
    pdl_wait();                                    // inputs may come from the kernel before this one
    const int q_begin = __ldg(p.cu_q + b), q_len = __ldg(p.cu_q + b + 1) - q_begin;
    const int n_b = __ldg(p.seq_lens + b);
    const int n_tiles = (q_len + TQ - 1) / TQ;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;      // tiles with the most keys are scheduled first
    if (blockIdx.x == 0 && threadIdx.x == 0 && (q_len < 0 || q_len > n_b || n_tiles > (int)gridDim.x))
        atomicOr(p.status, STATUS_BOUNDS);         // more queries than cached tokens, or than the caller's bound
    __syncthreads();
    if (q_len <= 0 || q_len > n_b || qt >= n_tiles) return;
    const int q0 = qt * TQ;
    const int q_end = (q0 + TQ < q_len) ? q0 + TQ : q_len;    // tokens [q0, q_end) of the sequence's new ones
    const int pos0 = n_b - q_len;                             // position of the sequence's first new token
    const int n_keys = pos0 + q_end;                          // keys 0 .. n_keys-1 are visible to some row
    const int n_pages = (n_keys + PAGE - 1) / PAGE;
    const int n_kb = (n_pages + KB - 1) / KB;

    // producer (thread 0): key block kb -> stage kb % NSTAGE
    auto issue = [&](int kb) {
        const int s = kb % NSTAGE;
        const int pg0 = kb * KB;
        const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
        int ids[KB];
#pragma unroll
        for (int j = 0; j < KB; ++j) ids[j] = j < np ? __ldg(p.page_table + (int64_t)b * p.pt_stride + pg0 + j) : 0;
        const uint32_t bar = bars + 8 * s;
        mbar_expect_tx(bar, (uint32_t)(np * BLOCK));
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (j < np) {
                int id = ids[j];
                if (id < 0 || (int64_t)id >= p.max_pages) {
                    atomicOr(p.status, STATUS_BOUNDS);
                    id = 0;
                }
                bulk_copy_g2s(ring + (uint32_t)((s * KB + j) * BLOCK),
                              p.layer_base + (int64_t)id * p.page_stride + (int64_t)h * BLOCK, BLOCK, bar);
            }
        }
    };
    int issued = 0;                                // key blocks handed to the copy engine (thread 0's count)
    if (threadIdx.x == 0)
        for (; issued < NSTAGE && issued < n_kb; ++issued) issue(issued);

    // this thread's two rows of the tile: r_lo = 16*warp + gid, r_hi = r_lo + 8; row r = token r/G, head r%G
    const int r_lo = 16 * warp + gid, r_hi = r_lo + 8;
    const int qi_lo = r_lo / G, g_lo = r_lo - qi_lo * G, qi_hi = r_hi / G, g_hi = r_hi - qi_hi * G;
    const bool ok_lo = qi_lo < TQ && q0 + qi_lo < q_end, ok_hi = qi_hi < TQ && q0 + qi_hi < q_end;
    // rows outside the tile run unmasked on whatever is there; nothing of theirs is stored
    const int pos_lo = ok_lo ? pos0 + q0 + qi_lo : 0x7FFFFFFF, pos_hi = ok_hi ? pos0 + q0 + qi_hi : 0x7FFFFFFF;
    const int64_t row_lo = ((int64_t)(q_begin + q0 + qi_lo) * p.Hq + (int64_t)h * G + g_lo) * D;
    const int64_t row_hi = ((int64_t)(q_begin + q0 + qi_hi) * p.Hq + (int64_t)h * G + g_hi) * D;

    uint32_t qa[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        const int c = 16 * ks + 2 * tig;
        qa[ks][0] = ok_lo ? __ldg(reinterpret_cast<const unsigned int *>(p.Q + row_lo + c)) : 0u;
        qa[ks][1] = ok_hi ? __ldg(reinterpret_cast<const unsigned int *>(p.Q + row_hi + c)) : 0u;
        qa[ks][2] = ok_lo ? __ldg(reinterpret_cast<const unsigned int *>(p.Q + row_lo + c + 8)) : 0u;
        qa[ks][3] = ok_hi ? __ldg(reinterpret_cast<const unsigned int *>(p.Q + row_hi + c + 8)) : 0u;
    }
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    const uint32_t k_off = (uint32_t)((((lane >> 3) & 1) * PAGE + (lane >> 4) * 8 + (lane & 7)) * 16);
    const uint32_t v_off = (uint32_t)(((lane >> 4) * PAGE + ((lane >> 3) & 1) * 8 + (lane & 7)) * 16);
    int failed_at = -1;
    for (int kb = 0; kb < n_kb; ++kb) {
        const int s = kb % NSTAGE;
        const uint32_t parity = (uint32_t)((kb / NSTAGE) & 1);
        const bool ok = mbar_wait_bounded(bars + 8 * s, parity);
        if (!__syncthreads_and(ok)) {              // a copy never arrived: flag it and leave together
            if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
            failed_at = kb;
            break;
        }
        const int pg0 = kb * KB;
        const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
        const uint32_t stage = ring + (uint32_t)(s * KB * BLOCK);
        // slots of the sequence's last page that were never written may hold anything: zero their V rows
        // so that 0 * x stays 0 (their scores are masked below)
        const int last_valid = n_b - (pg0 + np - 1) * PAGE;       // tokens in use in the block's last page
        if (last_valid < PAGE) {
            const uint32_t sV = stage + (uint32_t)((np - 1) * BLOCK) + half_bytes(D);
            for (int i = threadIdx.x; i < (D / 8) * PAGE; i += blockDim.x)
                if ((i & (PAGE - 1)) >= last_valid)
                    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(sV + (uint32_t)(i * 16)), "r"(0u) : "memory");
            fence_proxy_async();
            __syncthreads();
        }
        // S = Q K^T for up to 64 keys
        float sc[2 * KB][4];
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            sc[2 * j][0] = sc[2 * j][1] = sc[2 * j][2] = sc[2 * j][3] = 0.f;
            sc[2 * j + 1][0] = sc[2 * j + 1][1] = sc[2 * j + 1][2] = sc[2 * j + 1][3] = 0.f;
            if (j < np) {
                const uint32_t sK = stage + (uint32_t)(j * BLOCK) + k_off;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t r0, r1, r2, r3;
                    ldmatrix_x4(sK + (uint32_t)(ks * 2 * PAGE * 16), r0, r1, r2, r3);
                    mma_bf16_16816(sc[2 * j], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], r0, r1);
                    mma_bf16_16816(sc[2 * j + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], r2, r3);
                }
            }
        }
        // scale, causal mask, row maxima
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2 * KB; ++nt) {
            const int t0 = (pg0 + (nt >> 1)) * PAGE + (nt & 1) * 8 + 2 * tig;    // key of elements [0] and [2]
            const bool there = (nt >> 1) < np;
            sc[nt][0] = (there && t0 <= pos_lo) ? sc[nt][0] * p.scale_log2 : -INFINITY;
            sc[nt][1] = (there && t0 + 1 <= pos_lo) ? sc[nt][1] * p.scale_log2 : -INFINITY;
            sc[nt][2] = (there && t0 <= pos_hi) ? sc[nt][2] * p.scale_log2 : -INFINITY;
            sc[nt][3] = (there && t0 + 1 <= pos_hi) ? sc[nt][3] * p.scale_log2 : -INFINITY;
            mx_lo = fmaxf(mx_lo, fmaxf(sc[nt][0], sc[nt][1]));
            mx_hi = fmaxf(mx_hi, fmaxf(sc[nt][2], sc[nt][3]));
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(FULL, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(FULL, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(FULL, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(FULL, mx_hi, 2));
        // key 0 is visible to every row, so after the first block the running maxima are finite; a block
        // that is entirely in a row's future leaves that row unchanged (alpha = 1, all p = 0)
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const float a_lo = fast_exp2(m_lo - mn_lo), a_hi = fast_exp2(m_hi - mn_hi);
        m_lo = mn_lo;
        m_hi = mn_hi;
        float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
        for (int nt = 0; nt < 2 * KB; ++nt) {
            sc[nt][0] = fast_exp2(sc[nt][0] - mn_lo); sc[nt][1] = fast_exp2(sc[nt][1] - mn_lo);
            sc[nt][2] = fast_exp2(sc[nt][2] - mn_hi); sc[nt][3] = fast_exp2(sc[nt][3] - mn_hi);
            sum_lo += sc[nt][0] + sc[nt][1];
            sum_hi += sc[nt][2] + sc[nt][3];
        }
        l_lo = l_lo * a_lo + sum_lo;
        l_hi = l_hi * a_hi + sum_hi;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            o[i][0] *= a_lo; o[i][1] *= a_lo;
            o[i][2] *= a_hi; o[i][3] *= a_hi;
        }
        // O += P V
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (j < np) {
                const uint32_t pa0 = pack_bf16x2(sc[2 * j][0], sc[2 * j][1]), pa1 = pack_bf16x2(sc[2 * j][2], sc[2 * j][3]);
                const uint32_t pa2 = pack_bf16x2(sc[2 * j + 1][0], sc[2 * j + 1][1]);
                const uint32_t pa3 = pack_bf16x2(sc[2 * j + 1][2], sc[2 * j + 1][3]);
                const uint32_t sV = stage + (uint32_t)(j * BLOCK) + half_bytes(D) + v_off;
#pragma unroll
                for (int jd = 0; jd < KS; ++jd) {
                    uint32_t r0, r1, r2, r3;
                    ldmatrix_x4_trans(sV + (uint32_t)(jd * 2 * PAGE * 16), r0, r1, r2, r3);
                    mma_bf16_16816(o[2 * jd], pa0, pa1, pa2, pa3, r0, r1);
                    mma_bf16_16816(o[2 * jd + 1], pa0, pa1, pa2, pa3, r2, r3);
                }
            }
        }
        __syncthreads();                           // every warp is done with this stage
        if (threadIdx.x == 0 && issued < n_kb) issue(issued++);
    }
    if (failed_at >= 0) {
        // copies still in flight must land before the CTA (and its shared memory) goes away: wait, bounded,
        // for every block that was issued after the one that gave up
        if (threadIdx.x == 0)
            for (int kb = failed_at + 1; kb < issued; ++kb)
                mbar_wait_bounded(bars + 8 * (kb % NSTAGE), (uint32_t)((kb / NSTAGE) & 1));
        return;
    }
    pdl_trigger();
    l_lo += __shfl_xor_sync(FULL, l_lo, 1);
    l_lo += __shfl_xor_sync(FULL, l_lo, 2);
    l_hi += __shfl_xor_sync(FULL, l_hi, 1);
    l_hi += __shfl_xor_sync(FULL, l_hi, 2);
    if (ok_lo) {
        const float inv = 1.f / l_lo;
        uint16_t *dst = p.out + row_lo + 2 * tig;
#pragma unroll
        for (int i = 0; i < D / 8; ++i)
            *reinterpret_cast<uint32_t *>(dst + 8 * i) = pack_bf16x2(o[i][0] * inv, o[i][1] * inv);
    }
    if (ok_hi) {
        const float inv = 1.f / l_hi;
        uint16_t *dst = p.out + row_hi + 2 * tig;
#pragma unroll
        for (int i = 0; i < D / 8; ++i)
            *reinterpret_cast<uint32_t *>(dst + 8 * i) = pack_bf16x2(o[i][2] * inv, o[i][3] * inv);
    }
}

}  // namespace

size_t prefill_smem_bytes(int D)
{
    if (D != 64 && D != 128) return 0;
    return 128 + (size_t)NSTAGE * KB * block_bytes(D) + NSTAGE * 8;
}

int prefill_tile_tokens(int G) { return ROWS / G; }

cudaError_t launch_prefill(const PrefillParams &p, int D, int G, int q_tiles, bool pdl, cudaStream_t s)
{
    const size_t smem = prefill_smem_bytes(D);
    if (smem == 0 || q_tiles <= 0) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)q_tiles, (unsigned)p.Hkv, (unsigned)p.B);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (D == 128) {
        cudaError_t e = cudaFuncSetAttribute(prefill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, prefill_kernel<128>, p, G);
    }
    cudaError_t e = cudaFuncSetAttribute(prefill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, prefill_kernel<64>, p, G);
}

}  // namespace skv
