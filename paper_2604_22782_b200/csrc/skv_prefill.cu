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
    const bool too_long = (int64_t)n_b > (int64_t)p.pt_stride * PAGE;     // more pages than a page-table row holds
    const int n_tiles = (q_len + TQ - 1) / TQ;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;      // tiles with the most keys are scheduled first
    if (blockIdx.x == 0 && threadIdx.x == 0 && (q_len < 0 || q_len > n_b || too_long || n_tiles > (int)gridDim.x))
        atomicOr(p.status, STATUS_BOUNDS);         // more queries than cached tokens, or than the caller's bound
    __syncthreads();
    if (q_len <= 0 || q_len > n_b || too_long || qt >= n_tiles) return;
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

// ---------------------------------------------------------------------------
// The same tile scheme on FP8 pages (E4M3 codes + one fp32 scale per token and kv head): the codes go
// to mma.sync as f16 (exact), the scales stay outside the contractions as in the decode kernel:
//   score = qmax_row kscale_key (Q/qmax . Kc),     P' = p vscale_key / c,     O = c sum P' Vc,
// c a power of two >= every vscale seen so far.  Fragments are 32-bit shared-memory loads of four
// consecutive dims (scores) or keys (values) of one row of the page: the order of the contraction
// index inside an instruction is free as long as both operands agree, and the score instructions
// take the page's key rows in the order 0,1,4,5,8,9,12,13 | 2,3,6,7,10,11,14,15, so that a thread's
// four probabilities of a page are keys 4tig .. 4tig+3, the four keys of its V words.
// ---------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128, 2) prefill_fp8_kernel(PrefillParams p, int G)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = fp8_block_bytes(D);      // K codes | V codes | K scales | V scales of one (page, kv head)
    constexpr int KS = D / 16;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int b = blockIdx.z, h = blockIdx.y;
    const int TQ = ROWS / G;

    const uint32_t base = smem_u32(smem_raw);
    const uint32_t pad = (128u - (base & 127u)) & 127u;
    const uint32_t ring = base + pad;
    const uint32_t bars = ring + NSTAGE * KB * BLOCK;
    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) mbar_init(bars + 8 * s, 1);
        fence_barrier_init();
    }
    pdl_wait();
    const int q_begin = __ldg(p.cu_q + b), q_len = __ldg(p.cu_q + b + 1) - q_begin;
    const int n_b = __ldg(p.seq_lens + b);
    const bool too_long = (int64_t)n_b > (int64_t)p.pt_stride * PAGE;     // more pages than a page-table row holds
    const int n_tiles = (q_len + TQ - 1) / TQ;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;
    if (blockIdx.x == 0 && threadIdx.x == 0 && (q_len < 0 || q_len > n_b || too_long || n_tiles > (int)gridDim.x))
        atomicOr(p.status, STATUS_BOUNDS);
    __syncthreads();
    if (q_len <= 0 || q_len > n_b || too_long || qt >= n_tiles) return;
    const int q0 = qt * TQ;
    const int q_end = (q0 + TQ < q_len) ? q0 + TQ : q_len;
    const int pos0 = n_b - q_len;
    const int n_keys = pos0 + q_end;
    const int n_pages = (n_keys + PAGE - 1) / PAGE;
    const int n_kb = (n_pages + KB - 1) / KB;

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
    int issued = 0;
    if (threadIdx.x == 0)
        for (; issued < NSTAGE && issued < n_kb; ++issued) issue(issued);

    const int r_lo = 16 * warp + gid, r_hi = r_lo + 8;
    const int qi_lo = r_lo / G, g_lo = r_lo - qi_lo * G, qi_hi = r_hi / G, g_hi = r_hi - qi_hi * G;
    const bool ok_lo = qi_lo < TQ && q0 + qi_lo < q_end, ok_hi = qi_hi < TQ && q0 + qi_hi < q_end;
    const int pos_lo = ok_lo ? pos0 + q0 + qi_lo : 0x7FFFFFFF, pos_hi = ok_hi ? pos0 + q0 + qi_hi : 0x7FFFFFFF;
    const int64_t row_lo = ((int64_t)(q_begin + q0 + qi_lo) * p.Hq + (int64_t)h * G + g_lo) * D;
    const int64_t row_hi = ((int64_t)(q_begin + q0 + qi_hi) * p.Hq + (int64_t)h * G + g_hi) * D;

    // Q / qmax of the thread's two rows as f16; k-step ks, thread tig: dims 16ks + 4tig .. +3
    uint32_t qa[KS][4];
    float qmax_lo = 0.f, qmax_hi = 0.f;
    {
        float ql[KS][4], qh[KS][4];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int c = 16 * ks + 4 * tig;
            const uint2 wl = ok_lo ? __ldg(reinterpret_cast<const uint2 *>(p.Q + row_lo + c)) : make_uint2(0u, 0u);
            const uint2 wh = ok_hi ? __ldg(reinterpret_cast<const uint2 *>(p.Q + row_hi + c)) : make_uint2(0u, 0u);
            ql[ks][0] = bf16_lo(wl.x); ql[ks][1] = bf16_hi(wl.x); ql[ks][2] = bf16_lo(wl.y); ql[ks][3] = bf16_hi(wl.y);
            qh[ks][0] = bf16_lo(wh.x); qh[ks][1] = bf16_hi(wh.x); qh[ks][2] = bf16_lo(wh.y); qh[ks][3] = bf16_hi(wh.y);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                qmax_lo = fmaxf(qmax_lo, fabsf(ql[ks][i]));
                qmax_hi = fmaxf(qmax_hi, fabsf(qh[ks][i]));
            }
        }
        qmax_lo = fmaxf(qmax_lo, __shfl_xor_sync(FULL, qmax_lo, 1));
        qmax_lo = fmaxf(qmax_lo, __shfl_xor_sync(FULL, qmax_lo, 2));
        qmax_hi = fmaxf(qmax_hi, __shfl_xor_sync(FULL, qmax_hi, 1));
        qmax_hi = fmaxf(qmax_hi, __shfl_xor_sync(FULL, qmax_hi, 2));
        const float il = qmax_lo > 0.f ? 1.f / qmax_lo : 0.f, ih = qmax_hi > 0.f ? 1.f / qmax_hi : 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = pack_f16x2(ql[ks][0] * il, ql[ks][1] * il);
            qa[ks][1] = pack_f16x2(qh[ks][0] * ih, qh[ks][1] * ih);
            qa[ks][2] = pack_f16x2(ql[ks][2] * il, ql[ks][3] * il);
            qa[ks][3] = pack_f16x2(qh[ks][2] * ih, qh[ks][3] * ih);
        }
    }
    const float qs_lo = qmax_lo * p.scale_log2, qs_hi = qmax_hi * p.scale_log2;
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f, cs = 0.f;

    // key rows of the two score tiles of a page, and this thread's bytes in them
    const int krow = 4 * (gid >> 1) + (gid & 1);
    const uint32_t k_off0 = (uint32_t)(fp8_k_pos(D, krow, 0) + 4 * tig), k_off1 = (uint32_t)(fp8_k_pos(D, krow + 2, 0) + 4 * tig);
    const uint32_t v_off = (uint32_t)(fp8_v_off(D) + gid * PAGE + 4 * tig);
    int failed_at = -1;
    for (int kb = 0; kb < n_kb; ++kb) {
        const int s = kb % NSTAGE;
        const uint32_t parity = (uint32_t)((kb / NSTAGE) & 1);
        const bool ok = mbar_wait_bounded(bars + 8 * s, parity);
        if (!__syncthreads_and(ok)) {
            if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
            failed_at = kb;
            break;
        }
        const int pg0 = kb * KB;
        const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
        const uint32_t stage = ring + (uint32_t)(s * KB * BLOCK);
        const int last_valid = n_b - (pg0 + np - 1) * PAGE;       // tokens in use in the block's last page
        // scores: sc[2j] = keys 4tig, 4tig+1 and sc[2j+1] = keys 4tig+2, 4tig+3 of page j ([0],[1]: row lo; [2],[3]: row hi)
        float sc[2 * KB][4];
        float4 vsc[KB];
        float svmax = 0.f;
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            sc[2 * j][0] = sc[2 * j][1] = sc[2 * j][2] = sc[2 * j][3] = 0.f;
            sc[2 * j + 1][0] = sc[2 * j + 1][1] = sc[2 * j + 1][2] = sc[2 * j + 1][3] = 0.f;
            vsc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (j < np) {
                const uint32_t blk = stage + (uint32_t)(j * BLOCK);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t w0, w1, b0, b1;
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w0) : "r"(blk + k_off0 + (uint32_t)(ks * 128)));
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w1) : "r"(blk + k_off1 + (uint32_t)(ks * 128)));
                    e4m3x4_to_f16x2(w0, b0, b1);
                    mma_f16_16816(sc[2 * j], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                    e4m3x4_to_f16x2(w1, b0, b1);
                    mma_f16_16816(sc[2 * j + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                }
                float4 ksc;
                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(ksc.x), "=f"(ksc.y), "=f"(ksc.z), "=f"(ksc.w)
                             : "r"(blk + (uint32_t)(fp8_ks_off(D) + 16 * tig)));
                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(vsc[j].x), "=f"(vsc[j].y), "=f"(vsc[j].z), "=f"(vsc[j].w)
                             : "r"(blk + (uint32_t)(fp8_vs_off(D) + 16 * tig)));
                const int t0 = (pg0 + j) * PAGE + 4 * tig;       // key of sc[2j][0]
                const int nv = (j == np - 1) ? last_valid : PAGE; // slots past the sequence's end may hold anything
                const float kk[4] = {ksc.x, ksc.y, ksc.z, ksc.w};
                float *vv = &vsc[j].x;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const bool there = 4 * tig + i < nv;
                    float &e_lo = sc[2 * j + (i >> 1)][i & 1], &e_hi = sc[2 * j + (i >> 1)][2 + (i & 1)];
                    e_lo = (there && t0 + i <= pos_lo) ? e_lo * (qs_lo * kk[i]) : -INFINITY;
                    e_hi = (there && t0 + i <= pos_hi) ? e_hi * (qs_hi * kk[i]) : -INFINITY;
                    if (!there) vv[i] = 0.f;
                    svmax = fmaxf(svmax, vv[i]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) sc[2 * j][i] = sc[2 * j + 1][i] = -INFINITY;
            }
        }
        float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2 * KB; ++nt) {
            mx_lo = fmaxf(mx_lo, fmaxf(sc[nt][0], sc[nt][1]));
            mx_hi = fmaxf(mx_hi, fmaxf(sc[nt][2], sc[nt][3]));
        }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(FULL, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(FULL, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(FULL, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(FULL, mx_hi, 2));
        svmax = fmaxf(svmax, __shfl_xor_sync(FULL, svmax, 1));
        svmax = fmaxf(svmax, __shfl_xor_sync(FULL, svmax, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        float a_lo = fast_exp2(m_lo - mn_lo), a_hi = fast_exp2(m_hi - mn_hi);
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
        // reference scale of the V side: the smallest power of two >= every vscale so far
        const float up = __uint_as_float((__float_as_uint(svmax) + 0x007FFFFFu) & 0x7F800000u);
        const float cs_new = fmaxf(cs, up);
        const float inv_cs = cs_new > 0.f ? __uint_as_float(0x7F000000u - __float_as_uint(cs_new)) : 0.f;
        const float ca = cs * inv_cs;                      // 1 unless the reference grew
        cs = cs_new;
        a_lo *= ca;
        a_hi *= ca;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            o[i][0] *= a_lo; o[i][1] *= a_lo;
            o[i][2] *= a_hi; o[i][3] *= a_hi;
        }
        // O += P' Vc
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (j < np) {
                const float w0 = vsc[j].x * inv_cs, w1 = vsc[j].y * inv_cs, w2 = vsc[j].z * inv_cs, w3 = vsc[j].w * inv_cs;
                const uint32_t pa0 = pack_f16x2(sc[2 * j][0] * w0, sc[2 * j][1] * w1);
                const uint32_t pa1 = pack_f16x2(sc[2 * j][2] * w0, sc[2 * j][3] * w1);
                const uint32_t pa2 = pack_f16x2(sc[2 * j + 1][0] * w2, sc[2 * j + 1][1] * w3);
                const uint32_t pa3 = pack_f16x2(sc[2 * j + 1][2] * w2, sc[2 * j + 1][3] * w3);
                uint32_t vmask = 0xFFFFFFFFu;              // bytes of a V word that belong to tokens in use
                if (j == np - 1 && last_valid < PAGE) {
                    const int keep = last_valid - 4 * tig;
                    vmask = keep >= 4 ? 0xFFFFFFFFu : keep <= 0 ? 0u : (0xFFFFFFFFu >> (8 * (4 - keep)));
                }
                const uint32_t sV = stage + (uint32_t)(j * BLOCK) + v_off;
#pragma unroll
                for (int nt = 0; nt < D / 8; ++nt) {
                    uint32_t wv, b0, b1;
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(wv) : "r"(sV + (uint32_t)(nt * 8 * PAGE)));
                    e4m3x4_to_f16x2(wv & vmask, b0, b1);
                    mma_f16_16816(o[nt], pa0, pa1, pa2, pa3, b0, b1);
                }
            }
        }
        __syncthreads();
        if (threadIdx.x == 0 && issued < n_kb) issue(issued++);
    }
    if (failed_at >= 0) {
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
        const float inv = cs / l_lo;
        uint16_t *dst = p.out + row_lo + 2 * tig;
#pragma unroll
        for (int i = 0; i < D / 8; ++i)
            *reinterpret_cast<uint32_t *>(dst + 8 * i) = pack_bf16x2(o[i][0] * inv, o[i][1] * inv);
    }
    if (ok_hi) {
        const float inv = cs / l_hi;
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

size_t prefill_fp8_smem_bytes(int D)
{
    if (D != 64 && D != 128) return 0;
    return 128 + (size_t)NSTAGE * KB * fp8_block_bytes(D) + NSTAGE * 8;
}

int prefill_tile_tokens(int G) { return ROWS / G; }

cudaError_t launch_prefill_fp8(const PrefillParams &p, int D, int G, int q_tiles, bool pdl, cudaStream_t s)
{
    const size_t smem = prefill_fp8_smem_bytes(D);
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
    auto kern = D == 128 ? prefill_fp8_kernel<128> : prefill_fp8_kernel<64>;
    cudaError_t e = ensure_dynamic_smem(kern, smem);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, kern, p, G);
}

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
        cudaError_t e = ensure_dynamic_smem(prefill_kernel<128>, smem);
        if (e != cudaSuccess) return e;
        return cudaLaunchKernelEx(&cfg, prefill_kernel<128>, p, G);
    }
    cudaError_t e = ensure_dynamic_smem(prefill_kernel<64>, smem);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, prefill_kernel<64>, p, G);
}

}  // namespace skv
