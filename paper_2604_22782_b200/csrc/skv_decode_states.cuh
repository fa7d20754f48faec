// Per-warp compute state of the decode split-K kernels: what one warp does with one (page, kv head) block
// that has landed in shared memory, for the three storage / arithmetic variants.  Every State has
//   begin(p, b, h, G, lane)          load the G query heads of kv head h of sequence b, clear the running state
//   page(blk, valid, scale_log2, lane)  fold one block (shared address blk, `valid` tokens in use) into it
//   finish(part_o, part_ml, slot, G, lane)  write the run's partial (running max in log2 units, sum,
//                                        unnormalised output) to slot `slot` of the given arrays
//                                        (global or shared memory: generic pointers)
#pragma once
#include "skv_common.cuh"

#include <math.h>

namespace skv {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int WIN = 128;   // page ids a warp keeps in registers (4 per lane)

// ---------------------------------------------------------------------------
// Per-warp compute state, tensor-core variant: the G query heads of one kv head
// are rows of a 16-row A operand (rows >= G are zero), one page is 16 key
// columns.  S = Q K^T  (m16 n16 k D) and  O += P V  (m16 n D k16) with
// mma.m16n8k16; softmax runs on the accumulator fragment in fp32.
// ---------------------------------------------------------------------------
template <int D>
struct TensorCoreState {
    static constexpr int BLOCK = block_bytes(D);   // bytes of one (page, kv head) block
    static constexpr int MAX_CTA_CONSUMERS = 8;    // consumer warps of the CTA-per-range kernel that the registers allow
    static constexpr bool CTA_COMBINER = true;     // ... and a warp of its own that combines the consumers' states
    static constexpr int CTA_MAX_REGS = 160;       // 10 warps of it and a CTA of the merge kernel (64 x 208) fit one SM
    static constexpr int KS = D / 16;   // k-steps of QK^T, and pairs of 8-dim tiles of PV
    uint32_t qa[KS][2];
    float o[D / 8][4];
    float m, l;

    __device__ __forceinline__ void begin(const DecodeParams &p, int b, int h, int G, int lane)
    {
        begin_rows(p.Q + ((int64_t)b * p.Hq + (int64_t)h * G) * D, G, lane);
    }

    // rows: the G query rows [G][D] of the kv head (global or shared memory)
    __device__ __forceinline__ void begin_rows(const uint16_t *rows, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        const uint16_t *q = rows + g * D + 2 * tig;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = (g < G) ? *reinterpret_cast<const unsigned int *>(q + 16 * ks) : 0u;
            qa[ks][1] = (g < G) ? *reinterpret_cast<const unsigned int *>(q + 16 * ks + 8) : 0u;
        }
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        m = -INFINITY;
        l = 0.f;
    }

    // one page: blk = shared address of the block (K half, V half), valid = tokens in use (1..16)
    __device__ __forceinline__ void page(uint32_t blk, int valid, float scale_log2, int lane)
    {
        const uint32_t sK = blk, sV = blk + half_bytes(D);
        const int tig = lane & 3;
        float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        // K fragments: matrices (chunk 2ks | 2ks+1) x (tokens 0-7 | 8-15)
        const uint32_t k_lane = sK + (uint32_t)((((lane >> 3) & 1) * PAGE + (lane >> 4) * 8 + (lane & 7)) * 16);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t r0, r1, r2, r3;
            ldmatrix_x4(k_lane + (uint32_t)(ks * 2 * PAGE * 16), r0, r1, r2, r3);
            mma_bf16_16816(s[0], qa[ks][0], 0u, qa[ks][1], 0u, r0, r1);
            mma_bf16_16816(s[1], qa[ks][0], 0u, qa[ks][1], 0u, r2, r3);
        }
        // this thread's four scores: tokens 2tig, 2tig+1, 8+2tig, 9+2tig of head lane>>2
        float v0 = s[0][0] * scale_log2, v1 = s[0][1] * scale_log2;
        float v2 = s[1][0] * scale_log2, v3 = s[1][1] * scale_log2;
        if (valid < PAGE) {
            const int t0 = 2 * tig;
            if (t0 >= valid) v0 = -INFINITY;
            if (t0 + 1 >= valid) v1 = -INFINITY;
            if (t0 + 8 >= valid) v2 = -INFINITY;
            if (t0 + 9 >= valid) v3 = -INFINITY;
            // rows of V past the valid tokens may hold anything: zero them so 0 * x stays 0
            for (int i = lane; i < (D / 8) * PAGE; i += 32) {
                const int t = i & (PAGE - 1);
                if (t >= valid) {
                    const uint32_t a = sV + (uint32_t)(i * 16);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                }
            }
            fence_proxy_async();
            __syncwarp();
        }
        float mx = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 2));
        const float m_new = fmaxf(m, mx);                 // finite: every page has a valid token
        const float alpha = fast_exp2(m - m_new);
        const float p0 = fast_exp2(v0 - m_new), p1 = fast_exp2(v1 - m_new);
        const float p2 = fast_exp2(v2 - m_new), p3 = fast_exp2(v3 - m_new);
        l = l * alpha + ((p0 + p1) + (p2 + p3));
        m = m_new;
        const uint32_t pa0 = pack_bf16x2(p0, p1), pa2 = pack_bf16x2(p2, p3);
        // V fragments (transposed): matrices (chunk nd | nd+1) x (tokens 0-7 | 8-15)
        const uint32_t v_lane = sV + (uint32_t)(((lane >> 4) * PAGE + ((lane >> 3) & 1) * 8 + (lane & 7)) * 16);
#pragma unroll
        for (int j = 0; j < KS; ++j) {
            uint32_t r0, r1, r2, r3;
            ldmatrix_x4_trans(v_lane + (uint32_t)(j * 2 * PAGE * 16), r0, r1, r2, r3);
            o[2 * j][0] *= alpha; o[2 * j][1] *= alpha;
            o[2 * j + 1][0] *= alpha; o[2 * j + 1][1] *= alpha;
            mma_bf16_16816(o[2 * j], pa0, 0u, pa2, 0u, r0, r1);
            mma_bf16_16816(o[2 * j + 1], pa0, 0u, pa2, 0u, r2, r3);
        }
    }

    // the run's partial (max, sum, unnormalised out) of every query head of the group -> slot
    __device__ __forceinline__ void finish(float *part_o, float *part_ml, int64_t slot, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        l += __shfl_xor_sync(FULL, l, 1);
        l += __shfl_xor_sync(FULL, l, 2);
        if (g < G) {
            float *po = part_o + (slot * G + g) * D + 2 * tig;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) *reinterpret_cast<float2 *>(po + 8 * i) = make_float2(o[i][0], o[i][1]);
            if (tig == 0) *reinterpret_cast<float2 *>(part_ml + (slot * G + g) * 2) = make_float2(m, l);
        }
    }

};

// ---------------------------------------------------------------------------
// CUDA-core variant for one query head per kv head (MHA): a GEMV per page, so
// no tensor cores.  Lane = (token slot t = lane&15, dim half = lane>>4); every
// lane runs its own online softmax over the tokens that fall in its slot and
// the 16 slots are combined once per run.
// ---------------------------------------------------------------------------
template <int D>
struct CudaCoreState {
    static constexpr int BLOCK = block_bytes(D);
    static constexpr int MAX_CTA_CONSUMERS = D > 64 ? 7 : 8;   // (64 query and 64 output values per lane at head_dim 128)
    static constexpr bool CTA_COMBINER = D <= 64;  // (at head_dim 128 the registers leave no room for a tenth warp)
    static constexpr int CTA_MAX_REGS = D <= 64 ? 160 : 200;
    static constexpr int HC = D / 16;   // 16-byte chunks per dim half
    float q[D / 2];
    float o[D / 2];
    float m, l;

    __device__ __forceinline__ void begin(const DecodeParams &p, int b, int h, int G, int lane)
    {
        begin_rows(p.Q + ((int64_t)b * p.Hq + h) * D, G, lane);
    }

    __device__ __forceinline__ void begin_rows(const uint16_t *rows, int /*G*/, int lane)
    {
        const int hf = lane >> 4;
        const uint16_t *qp = rows + hf * (D / 2);
#pragma unroll
        for (int c = 0; c < HC; ++c) {
            const uint4 w = *(reinterpret_cast<const uint4 *>(qp) + c);
            q[c * 8 + 0] = bf16_lo(w.x); q[c * 8 + 1] = bf16_hi(w.x);
            q[c * 8 + 2] = bf16_lo(w.y); q[c * 8 + 3] = bf16_hi(w.y);
            q[c * 8 + 4] = bf16_lo(w.z); q[c * 8 + 5] = bf16_hi(w.z);
            q[c * 8 + 6] = bf16_lo(w.w); q[c * 8 + 7] = bf16_hi(w.w);
        }
#pragma unroll
        for (int i = 0; i < D / 2; ++i) o[i] = 0.f;
        m = -INFINITY;
        l = 0.f;
    }

    __device__ __forceinline__ void page(uint32_t blk, int valid, float scale_log2, int lane)
    {
        const uint32_t sK = blk, sV = blk + half_bytes(D);
        const int t = lane & 15, hf = lane >> 4;
        const uint32_t off = (uint32_t)((hf * HC * PAGE + t) * 16);
        float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
        for (int c = 0; c < HC; ++c) {
            uint32_t x, y, z, w;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(sK + off + (uint32_t)(c * PAGE * 16)));
            acc0 = fmaf(q[c * 8 + 0], bf16_lo(x), acc0); acc1 = fmaf(q[c * 8 + 1], bf16_hi(x), acc1);
            acc0 = fmaf(q[c * 8 + 2], bf16_lo(y), acc0); acc1 = fmaf(q[c * 8 + 3], bf16_hi(y), acc1);
            acc0 = fmaf(q[c * 8 + 4], bf16_lo(z), acc0); acc1 = fmaf(q[c * 8 + 5], bf16_hi(z), acc1);
            acc0 = fmaf(q[c * 8 + 6], bf16_lo(w), acc0); acc1 = fmaf(q[c * 8 + 7], bf16_hi(w), acc1);
        }
        float acc = acc0 + acc1;
        acc += __shfl_xor_sync(FULL, acc, 16);
        const bool live = t < valid;
        const float v = live ? acc * scale_log2 : -INFINITY;
        const float m_new = fmaxf(m, v);
        const bool grew = m_new > m;
        if (__any_sync(FULL, grew)) {
            const float alpha = grew ? fast_exp2(m - m_new) : 1.f;
            l *= alpha;
#pragma unroll
            for (int i = 0; i < D / 2; ++i) o[i] *= alpha;
            m = m_new;
        }
        if (live) {
            const float pr = fast_exp2(v - m);
            l += pr;
#pragma unroll
            for (int c = 0; c < HC; ++c) {
                uint32_t x, y, z, w;
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(sV + off + (uint32_t)(c * PAGE * 16)));
                o[c * 8 + 0] = fmaf(pr, bf16_lo(x), o[c * 8 + 0]); o[c * 8 + 1] = fmaf(pr, bf16_hi(x), o[c * 8 + 1]);
                o[c * 8 + 2] = fmaf(pr, bf16_lo(y), o[c * 8 + 2]); o[c * 8 + 3] = fmaf(pr, bf16_hi(y), o[c * 8 + 3]);
                o[c * 8 + 4] = fmaf(pr, bf16_lo(z), o[c * 8 + 4]); o[c * 8 + 5] = fmaf(pr, bf16_hi(z), o[c * 8 + 5]);
                o[c * 8 + 6] = fmaf(pr, bf16_lo(w), o[c * 8 + 6]); o[c * 8 + 7] = fmaf(pr, bf16_hi(w), o[c * 8 + 7]);
            }
        }
    }

    // combine the 16 token slots: afterwards lanes with t == 0 hold the run's sum in o[], and (M, lt) everywhere
    __device__ __forceinline__ void reduce(float &M, float &lt, int lane)
    {
        M = m;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, d));
        const float wgt = (m == -INFINITY) ? 0.f : fast_exp2(m - M);
        lt = l * wgt;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) lt += __shfl_xor_sync(FULL, lt, d);
#pragma unroll
        for (int i = 0; i < D / 2; ++i) {
            float x = o[i] * wgt;
#pragma unroll
            for (int d = 1; d < 16; d <<= 1) x += __shfl_xor_sync(FULL, x, d);
            o[i] = x;
        }
    }

    __device__ __forceinline__ void finish(float *part_o, float *part_ml, int64_t slot, int /*G*/, int lane)
    {
        const int t = lane & 15, hf = lane >> 4;
        float M, lt;
        reduce(M, lt, lane);
        if (t == 0) {
            float *po = part_o + slot * D + hf * (D / 2);
#pragma unroll
            for (int i = 0; i < D / 2; i += 4)
                *reinterpret_cast<float4 *>(po + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
            if (hf == 0) *reinterpret_cast<float2 *>(part_ml + slot * 2) = make_float2(M, lt);
        }
    }

};

// ---------------------------------------------------------------------------
// FP8 pages (E4M3 codes + one fp32 scale per token for K and for V), any group size: tensor cores
// in f16, which holds every E4M3 value exactly.  Per page  S = (Q/qmax) Kc^T  and  O += P' Vc  on
// the raw codes; the per-token scales are applied outside the contractions:
//   score_t = qmax * kscale_t * S_t,      P'_t = p_t * vscale_t / c,
// with c a power of two >= every vscale seen so far (so P' <= 256 fits f16 whatever the magnitudes;
// when c grows O is scaled down with the softmax's own rescaling factor), and O * c at the end.
// Fragments come straight from shared memory without transposes because the contraction order
// within a k-step is free as long as both operands agree: a thread's k-slots {2tig,2tig+1,
// 2tig+8,2tig+9} carry FOUR CONSECUTIVE dims (QK^T) or tokens (PV), i.e. one 32-bit word of codes.
//   QK^T: thread (g = lane/4, tig) reads token rows 4*(g/2) + g%2 (+2 for the second 8-column tile),
//         dims [D/4*tig, D/4*(tig+1)) (K is stored in 8-token x 16-dim pieces, see fp8_k_pos), so
//         that its four scores are tokens 4tig .. 4tig+3;
//   PV:   V is stored dim-major, the word at dim 8*tile + g, byte 4*tig holds tokens 4tig .. 4tig+3.
// ---------------------------------------------------------------------------
template <int D>
struct Fp8State {
    static constexpr int BLOCK = fp8_block_bytes(D);
    static constexpr int MAX_CTA_CONSUMERS = 8;
    static constexpr bool CTA_COMBINER = true;
    static constexpr int CTA_MAX_REGS = 160;
    static constexpr int KS = D / 16;
    static constexpr int DT = D / 4;    // dims per thread of a quad
    uint32_t qa[KS][2];                 // f16x2: dims DT*tig + 4ks + {0,1} and + {2,3} of Q / qmax
    float o[D / 8][4];
    float m, l, qmax, cs;

    __device__ __forceinline__ void begin(const DecodeParams &p, int b, int h, int G, int lane)
    {
        begin_rows(p.Q + ((int64_t)b * p.Hq + (int64_t)h * G) * D, G, lane);
    }

    __device__ __forceinline__ void begin_rows(const uint16_t *rows, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        float q[DT];
        float amax = 0.f;
        if (g < G) {
            const uint4 *src = reinterpret_cast<const uint4 *>(rows + g * D + DT * tig);
#pragma unroll
            for (int c = 0; c < DT / 8; ++c) {
                const uint4 w = src[c];
                q[8 * c + 0] = bf16_lo(w.x); q[8 * c + 1] = bf16_hi(w.x);
                q[8 * c + 2] = bf16_lo(w.y); q[8 * c + 3] = bf16_hi(w.y);
                q[8 * c + 4] = bf16_lo(w.z); q[8 * c + 5] = bf16_hi(w.z);
                q[8 * c + 6] = bf16_lo(w.w); q[8 * c + 7] = bf16_hi(w.w);
            }
#pragma unroll
            for (int i = 0; i < DT; ++i) amax = fmaxf(amax, fabsf(q[i]));
        } else {
#pragma unroll
            for (int i = 0; i < DT; ++i) q[i] = 0.f;
        }
        amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 2));
        qmax = amax;
        const float inv = amax > 0.f ? 1.f / amax : 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = pack_f16x2(q[4 * ks] * inv, q[4 * ks + 1] * inv);
            qa[ks][1] = pack_f16x2(q[4 * ks + 2] * inv, q[4 * ks + 3] * inv);
        }
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        m = -INFINITY;
        l = 0.f;
        cs = 0.f;
    }

    __device__ __forceinline__ void page(uint32_t blk, int valid, float scale_log2, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        // ---- scores of tokens 4tig .. 4tig+3 for query head g ----
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        // token rows 4 (g/2) + g%2 and that + 2 (the same group of 8 tokens), 16-dim chunks (D/64) tig + c
        const int tok = 4 * (g >> 1) + (g & 1);
        const uint32_t k0 = blk + (uint32_t)((tok >> 3) * 8 * D + (DT / 16) * tig * 128 + (tok & 7) * 16), k1 = k0 + 2 * 16;
        uint32_t w0[DT / 4], w1[DT / 4];
#pragma unroll
        for (int c = 0; c < DT / 16; ++c) {
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(w0[4 * c]), "=r"(w0[4 * c + 1]), "=r"(w0[4 * c + 2]), "=r"(w0[4 * c + 3]) : "r"(k0 + 128 * c));
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(w1[4 * c]), "=r"(w1[4 * c + 1]), "=r"(w1[4 * c + 2]), "=r"(w1[4 * c + 3]) : "r"(k1 + 128 * c));
        }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t b0, b1;
            e4m3x4_to_f16x2(w0[ks], b0, b1);
            mma_f16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
            e4m3x4_to_f16x2(w1[ks], b0, b1);
            mma_f16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
        }
        float4 sk, sv;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(sk.x), "=f"(sk.y), "=f"(sk.z), "=f"(sk.w)
                     : "r"(blk + (uint32_t)(fp8_ks_off(D) + 16 * tig)));
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(sv.x), "=f"(sv.y), "=f"(sv.z), "=f"(sv.w)
                     : "r"(blk + (uint32_t)(fp8_vs_off(D) + 16 * tig)));
        const float qs = qmax * scale_log2;
        const int t0 = 4 * tig;
        float v0 = s0[0] * (qs * sk.x), v1 = s0[1] * (qs * sk.y), v2 = s1[0] * (qs * sk.z), v3 = s1[1] * (qs * sk.w);
        uint32_t vmask = 0xFFFFFFFFu;          // bytes of a V word (tokens 4tig..4tig+3) that are in use
        if (valid < PAGE) {                    // slots past the sequence's end may hold anything
            if (t0 >= valid) { v0 = -INFINITY; sv.x = 0.f; }
            if (t0 + 1 >= valid) { v1 = -INFINITY; sv.y = 0.f; }
            if (t0 + 2 >= valid) { v2 = -INFINITY; sv.z = 0.f; }
            if (t0 + 3 >= valid) { v3 = -INFINITY; sv.w = 0.f; }
            const int keep = valid - t0;       // leading bytes to keep
            vmask = keep >= 4 ? 0xFFFFFFFFu : keep <= 0 ? 0u : (0xFFFFFFFFu >> (8 * (4 - keep)));
        }
        float mx = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 2));
        // The reference m only follows the running maximum when that has grown by more than 2^8 (m is then
        // finite: every page has a valid token): until then the probabilities are at most 256, which f16
        // and the fp32 sums hold easily, and nothing has to be rescaled.  The result does not depend on
        // the reference.
        const float m_new = mx > m + 8.f ? mx : m;
        float alpha = fast_exp2(m - m_new);
        const float p0 = fast_exp2(v0 - m_new), p1 = fast_exp2(v1 - m_new);
        const float p2 = fast_exp2(v2 - m_new), p3 = fast_exp2(v3 - m_new);
        l = l * alpha + ((p0 + p1) + (p2 + p3));
        m = m_new;
        // reference scale of the V side: the smallest power of two >= every vscale so far
        float svmax = fmaxf(fmaxf(sv.x, sv.y), fmaxf(sv.z, sv.w));
        svmax = fmaxf(svmax, __shfl_xor_sync(FULL, svmax, 1));
        svmax = fmaxf(svmax, __shfl_xor_sync(FULL, svmax, 2));
        const float up = __uint_as_float((__float_as_uint(svmax) + 0x007FFFFFu) & 0x7F800000u);
        const float cs_new = fmaxf(cs, up);
        const float inv_cs = cs_new > 0.f ? 1.f / cs_new : 0.f;          // exact: a power of two
        alpha *= cs * inv_cs;                                             // 1 unless the reference grew
        cs = cs_new;
        const uint32_t pa0 = pack_f16x2(p0 * (sv.x * inv_cs), p1 * (sv.y * inv_cs));
        const uint32_t pa2 = pack_f16x2(p2 * (sv.z * inv_cs), p3 * (sv.w * inv_cs));
        if (__any_sync(FULL, alpha != 1.f)) {              // rare once the running maximum has settled
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) { o[nt][0] *= alpha; o[nt][1] *= alpha; }
        }
        // ---- O += P' Vc ----
        const uint32_t v_lane = blk + (uint32_t)(fp8_v_off(D) + g * PAGE + 4 * tig);
        uint32_t vw[D / 8];                    // all loads first: the volatile loads keep their order
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt)
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(vw[nt]) : "r"(v_lane + (uint32_t)(nt * 8 * PAGE)));
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            uint32_t b0, b1;
            e4m3x4_to_f16x2(vw[nt] & vmask, b0, b1);
            mma_f16_16816(o[nt], pa0, 0u, pa2, 0u, b0, b1);
        }
    }

    __device__ __forceinline__ void finish(float *part_o, float *part_ml, int64_t slot, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        l += __shfl_xor_sync(FULL, l, 1);
        l += __shfl_xor_sync(FULL, l, 2);
        if (g < G) {
            float *po = part_o + (slot * G + g) * D + 2 * tig;
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                *reinterpret_cast<float2 *>(po + 8 * i) = make_float2(o[i][0] * cs, o[i][1] * cs);
            if (tig == 0) *reinterpret_cast<float2 *>(part_ml + (slot * G + g) * 2) = make_float2(m, l);
        }
    }
};

}  // namespace skv
