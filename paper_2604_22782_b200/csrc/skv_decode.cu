// "Load + Attn" of Algorithm 2 for one new token per sequence (Eq. (3.1)):
// a split-K flash-decoding pass over the owner layer's pages and a
// log-sum-exp merge of the partial results.
//
// Work decomposition.  All (sequence, kv head, page) blocks of the call form
// one flattened list, b-major; it is cut into W equal contiguous ranges, one
// per WARP (W = grid * warps per CTA).  A warp streams its blocks through a
// private shared-memory ring filled by linear bulk copies (one 2*PAGE*D*2-byte
// copy per block, completion on an mbarrier), keeps a running (max, sum, out)
// per query head of the kv head's group, and at the end of every run inside a
// (sequence, kv head) segment writes one fp32 partial to slot  worker + segment.
// Every warp does the same number of blocks (+-1) whatever the length mix;
// warps never synchronise with each other after the prologue.  The merge
// kernel (one warp per segment) combines a segment's partials; it is launched
// so that it is already resident, waiting, when the split-K kernel ends.
#include "skv_common.cuh"
#include "skv_walk.cuh"

#include <math.h>

namespace skv {

namespace {

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
    static constexpr int KS = D / 16;   // k-steps of QK^T, and pairs of 8-dim tiles of PV
    uint32_t qa[KS][2];
    float o[D / 8][4];
    float m, l;

    __device__ __forceinline__ void begin(const DecodeParams &p, int b, int h, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        const uint16_t *q = p.Q + ((int64_t)b * p.Hq + (int64_t)h * G + g) * D + 2 * tig;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = (g < G) ? __ldg(reinterpret_cast<const unsigned int *>(q + 16 * ks)) : 0u;
            qa[ks][1] = (g < G) ? __ldg(reinterpret_cast<const unsigned int *>(q + 16 * ks + 8)) : 0u;
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
    __device__ __forceinline__ void finish(const DecodeParams &p, int64_t slot, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        l += __shfl_xor_sync(FULL, l, 1);
        l += __shfl_xor_sync(FULL, l, 2);
        if (g < G) {
            float *po = p.part_o + (slot * G + g) * D + 2 * tig;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) *reinterpret_cast<float2 *>(po + 8 * i) = make_float2(o[i][0], o[i][1]);
            if (tig == 0) *reinterpret_cast<float2 *>(p.part_ml + (slot * G + g) * 2) = make_float2(m, l);
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
    static constexpr int HC = D / 16;   // 16-byte chunks per dim half
    float q[D / 2];
    float o[D / 2];
    float m, l;

    __device__ __forceinline__ void begin(const DecodeParams &p, int b, int h, int /*G*/, int lane)
    {
        const int hf = lane >> 4;
        const uint16_t *qp = p.Q + ((int64_t)b * p.Hq + h) * D + hf * (D / 2);
#pragma unroll
        for (int c = 0; c < HC; ++c) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(qp) + c);
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

    __device__ __forceinline__ void finish(const DecodeParams &p, int64_t slot, int /*G*/, int lane)
    {
        const int t = lane & 15, hf = lane >> 4;
        float M, lt;
        reduce(M, lt, lane);
        if (t == 0) {
            float *po = p.part_o + slot * D + hf * (D / 2);
#pragma unroll
            for (int i = 0; i < D / 2; i += 4)
                *reinterpret_cast<float4 *>(po + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
            if (hf == 0) *reinterpret_cast<float2 *>(p.part_ml + slot * 2) = make_float2(M, lt);
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
    static constexpr int KS = D / 16;
    static constexpr int DT = D / 4;    // dims per thread of a quad
    uint32_t qa[KS][2];                 // f16x2: dims DT*tig + 4ks + {0,1} and + {2,3} of Q / qmax
    float o[D / 8][4];
    float m, l, qmax, cs;

    __device__ __forceinline__ void begin(const DecodeParams &p, int b, int h, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        float q[DT];
        float amax = 0.f;
        if (g < G) {
            const uint4 *src = reinterpret_cast<const uint4 *>(p.Q + ((int64_t)b * p.Hq + (int64_t)h * G + g) * D + DT * tig);
#pragma unroll
            for (int c = 0; c < DT / 8; ++c) {
                const uint4 w = __ldg(src + c);
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

    __device__ __forceinline__ void finish(const DecodeParams &p, int64_t slot, int G, int lane)
    {
        const int g = lane >> 2, tig = lane & 3;
        l += __shfl_xor_sync(FULL, l, 1);
        l += __shfl_xor_sync(FULL, l, 2);
        if (g < G) {
            float *po = p.part_o + (slot * G + g) * D + 2 * tig;
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                *reinterpret_cast<float2 *>(po + 8 * i) = make_float2(o[i][0] * cs, o[i][1] * cs);
            if (tig == 0) *reinterpret_cast<float2 *>(p.part_ml + (slot * G + g) * 2) = make_float2(m, l);
        }
    }
};

__device__ __forceinline__ void segment_partials(int64_t T, int64_t W, int64_t seg, int64_t s0, int pages, int &slot0,
                                                 int &n)
{
    if (T < W) {
        slot0 = (int)(s0 + seg);
        n = pages;
    } else {
        const int w_first = worker_of(s0, T, W);
        slot0 = (int)(w_first + seg);
        n = worker_of(s0 + pages - 1, T, W) - w_first + 1;
    }
}

// Log-sum-exp merge of the n partials at slots slot0 .. slot0+n-1 for the G query heads of a
// segment, by one warp:
//   out[g, :] = sum_i 2^(m_i - M) o_i / sum_i 2^(m_i - M) l_i,  M = max_i m_i.
// With G rounded up to a power of two G', the G'*D outputs are dealt to the 32 lanes in contiguous
// pieces of E2 = G'*D/64 float2 (a piece lies inside one head's row); NB partials are fetched
// together so that a typical segment costs one round trip to L2.
template <int D, int E2MAX, int NB>
__device__ __forceinline__ void merge_rows(const float *part_o, const float *part_ml, uint16_t *out_seg, int G,
                                           int slot0, int n, int lane)
{
    const int Gp = G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8;   // rows dealt out (lanes of rows >= G idle)
    const int E2 = Gp * D / 64;               // float2 per lane (<= E2MAX)
    const int e0 = lane * 2 * E2, g = e0 / D, d0 = e0 - g * D;
    if (g >= G) return;                       // no warp-wide operation below
    float2 acc[E2MAX];
#pragma unroll
    for (int e = 0; e < E2MAX; ++e) acc[e] = make_float2(0.f, 0.f);
    float M = -INFINITY, L = 0.f;
    const unsigned row = (unsigned)G * D;     // floats per partial
    const float2 *po = reinterpret_cast<const float2 *>(part_o + (size_t)slot0 * row + g * D + d0);
    const float2 *pm = reinterpret_cast<const float2 *>(part_ml + ((size_t)slot0 * G + g) * 2);
    for (int j0 = 0; j0 < n; j0 += NB) {
        float2 ml[NB];
        float2 v[NB][E2MAX];
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            ml[u] = make_float2(-INFINITY, 0.f);
            if (j0 + u < n) {
                ml[u] = __ldcg(pm + (j0 + u) * G);
                const float2 *src = po + (size_t)(j0 + u) * (row / 2);
#pragma unroll
                for (int e = 0; e < E2MAX; ++e)
                    if (e < E2) v[u][e] = __ldcg(src + e);
            }
        }
        float Mb = ml[0].x;
#pragma unroll
        for (int u = 1; u < NB; ++u) Mb = fmaxf(Mb, ml[u].x);
        const float M_new = fmaxf(M, Mb);            // finite: a partial holds at least one token
        const float keep = fast_exp2(M - M_new);     // 0 for the first batch
        L *= keep;
#pragma unroll
        for (int e = 0; e < E2MAX; ++e) { acc[e].x *= keep; acc[e].y *= keep; }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            if (j0 + u < n) {
                const float wt = fast_exp2(ml[u].x - M_new);
                L = fmaf(wt, ml[u].y, L);
#pragma unroll
                for (int e = 0; e < E2MAX; ++e)
                    if (e < E2) {
                        acc[e].x = fmaf(wt, v[u][e].x, acc[e].x);
                        acc[e].y = fmaf(wt, v[u][e].y, acc[e].y);
                    }
            }
        }
        M = M_new;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    uint32_t *dst = reinterpret_cast<uint32_t *>(out_seg + g * D + d0);
#pragma unroll
    for (int e = 0; e < E2MAX; ++e)
        if (e < E2) dst[e] = pack_bf16x2(acc[e].x * inv, acc[e].y * inv);
}

// ---------------------------------------------------------------------------
template <int D, class State>
__global__ void decode_splitk_kernel(DecodeParams p, int G, int stages)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = State::BLOCK;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint64_t t_entry = p.trace ? global_timer_ns() : 0;
    uint64_t t_first = 0;

    // carve shared memory: tables | rings | barriers | arrival word  (ring base rounded up to 128 bytes)
    const uint32_t base = smem_u32(smem_raw);
    const uint32_t pad = (128u - (base & 127u)) & 127u;
    int32_t *prefix = reinterpret_cast<int32_t *>(smem_raw + pad);
    int32_t *lens = prefix + p.B + 1;
    const size_t rings_off = pad + table_bytes(p.B);
    const uint32_t ring = base + (uint32_t)rings_off + (uint32_t)(warp * stages * BLOCK);
    const size_t bars_off = rings_off + (size_t)nwarps * stages * BLOCK;
    const uint32_t bars = base + (uint32_t)bars_off + (uint32_t)(warp * stages * 8);
    int *arrivals = reinterpret_cast<int *>(smem_raw + bars_off + (size_t)nwarps * stages * 8);

    if (lane == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(bars + 8 * s, 1);
        fence_barrier_init();
    }
    if (threadIdx.x == 0) *arrivals = 0;
    const bool late_wait = (p.flags & DECODE_LATE_WAIT) != 0;
    const bool reverse = (p.flags & DECODE_REVERSE) != 0;
    if (!late_wait) pdl_wait();            // anything read below may come from the kernel before this one

    // sequence lengths and cumulative page counts of the batch (warp 0), visible to all after the barrier
    if (warp == 0) scan_lengths(p.seq_lens, p.B, PAGE, prefix, lens, lane);
    __syncthreads();
    if (blockIdx.x == 0)       // the merge kernel reads the page counts from global memory
        for (int i = threadIdx.x; i <= p.B; i += blockDim.x) p.prefix[i] = prefix[i];

    const int64_t W = (int64_t)gridDim.x * nwarps, w = (int64_t)blockIdx.x * nwarps + warp;
    const int64_t T = (int64_t)prefix[p.B] * p.Hkv;
    int64_t x0 = 0;
    int n = 0;
    if (T > 0) {
        x0 = worker_begin(w, T, W);
        n = (int)(worker_begin(w + 1, T, W) - x0);
    }
    const int64_t x_first = reverse ? x0 + n - 1 : x0;

    // Half-way point of this worker: (in a chain of calls) wait for the kernel before this one, then let the
    // one after it be scheduled once every warp of the CTA has got here.
    bool synced = false;
    auto pdl_sync = [&]() {
        synced = true;
        if (late_wait) pdl_wait();
        __syncwarp();
        int last = 0;
        if (lane == 0) last = (atomicAdd(arrivals, 1) == nwarps - 1);
        if (__shfl_sync(FULL, last, 0)) pdl_trigger();
    };

    // ---- producer: keeps the ring full ----
    const uint64_t pol_stream = make_policy_evict_first(), pol_keep = make_policy_evict_normal();
    const int keep_from = n - (int)(((int64_t)n * p.keep_pct) / 100);
    Cursor prod = {0, 0, 0, 1};
    if (n > 0) prod = locate(prefix, p.B, p.Hkv, x_first);
    int prod_left = n, issued = 0, in_flight = 0, p_stage = 0;
    int win_b = -1, win_base = 0, ids0 = 0, ids1 = 0, ids2 = 0, ids3 = 0;   // page ids: 4 per lane
    auto issue = [&]() -> bool {
        if (prod_left == 0) return false;
        if (prod.b != win_b || prod.pg < win_base || prod.pg >= win_base + WIN) {
            win_b = prod.b;
            win_base = reverse ? (prod.pg >= WIN ? prod.pg - (WIN - 1) : 0) : prod.pg;
            const int32_t *row = p.page_table + (int64_t)prod.b * p.pt_stride + win_base + lane;
            const int left = prod.pages - win_base - lane;
            ids0 = left > 0 ? __ldg(row) : 0;
            ids1 = left > 32 ? __ldg(row + 32) : 0;
            ids2 = left > 64 ? __ldg(row + 64) : 0;
            ids3 = left > 96 ? __ldg(row + 96) : 0;
        }
        const int rel = prod.pg - win_base, sel = rel >> 5;
        const int mine = sel == 0 ? ids0 : sel == 1 ? ids1 : sel == 2 ? ids2 : ids3;
        int id = __shfl_sync(FULL, mine, rel & 31);
        if (lane == 0) {
            if (id < 0 || (int64_t)id >= p.max_pages) {
                atomicOr(p.status, STATUS_BOUNDS);
                id = 0;
            }
            const uint8_t *src = p.layer_base + (int64_t)id * p.page_stride + (int64_t)prod.h * BLOCK;
            const uint32_t bar = bars + 8 * p_stage;
            mbar_expect_tx(bar, BLOCK);
            bulk_copy_g2s_hint(ring + (uint32_t)(p_stage * BLOCK), src, BLOCK, bar,
                               issued >= keep_from ? pol_keep : pol_stream);
        }
        if (++p_stage == stages) p_stage = 0;
        ++in_flight;
        ++issued;
        if (--prod_left > 0) step(prod, prefix, p.Hkv, reverse);
        return true;
    };
    while (in_flight < stages && issue()) {}

    // ---- consumer: one iteration of the outer loop per run inside a (sequence, kv head) segment ----
    Cursor cons = {0, 0, 0, 1};
    if (n > 0) cons = locate(prefix, p.B, p.Hkv, x_first);
    int consumed = 0, c_stage = 0;
    const int half = n / 2;
    uint32_t parity = 0;
    bool failed = false;
    while (consumed < n && !failed) {
        const int b = cons.b, h = cons.h, pages = cons.pages, n_b = lens[cons.b];
        const int64_t seg = (int64_t)b * p.Hkv + h;
        {
            State st;                          // lives for this run only
            st.begin(p, b, h, G, lane);
            for (;;) {
                if (!synced && consumed >= half) pdl_sync();
                const bool ok = mbar_wait_bounded(bars + 8 * c_stage, parity);
                if (!__all_sync(FULL, ok)) {
                    // give up: flag it, let the copies still in flight land (bounded), leave
                    if (lane == 0) atomicOr(p.status, STATUS_TIMEOUT);
                    int s = c_stage;
                    uint32_t par = parity;
                    for (int k = 1; k < in_flight; ++k) {
                        if (++s == stages) { s = 0; par ^= 1u; }
                        mbar_wait_bounded(bars + 8 * s, par);
                    }
                    failed = true;
                    break;
                }
                if (p.trace && consumed == 0) t_first = global_timer_ns();
                const int left = n_b - cons.pg * PAGE;
                st.page(ring + (uint32_t)(c_stage * BLOCK), left < PAGE ? left : PAGE, p.scale_log2, lane);
                __syncwarp();                       // every lane is done reading this stage
                --in_flight;
                issue();                            // refill it
                if (++c_stage == stages) { c_stage = 0; parity ^= 1u; }
                ++consumed;
                const bool run_ends = (reverse ? (cons.pg == 0) : (cons.pg + 1 == pages)) || consumed == n;
                if (consumed < n) step(cons, prefix, p.Hkv, reverse);
                if (run_ends) break;
            }
            if (!failed) st.finish(p, partial_slot(T, W, w, x0, seg), G, lane);
        }
    }
    if (!synced) pdl_sync();
    if (p.trace && lane == 0) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        unsigned long long *t = p.trace + 4 * w;
        t[0] = smid; t[1] = t_entry; t[2] = t_first; t[3] = global_timer_ns();
    }
}

// ---------------------------------------------------------------------------
// Stand-alone merge kernel: one warp per (sequence, kv head) segment.
// ---------------------------------------------------------------------------
constexpr int MERGE_WARPS = 2;
#ifndef SKV_MERGE_PAYLOAD
#define SKV_MERGE_PAYLOAD 64                  // float2 in flight per lane while merging
#endif

// this warp's share of the segments: seg0, seg0 + stride, ...
template <int D, int E2MAX, int NB>
__device__ __forceinline__ void merge_loop(const MergeParams &p, int64_t seg0, int64_t stride, int lane)
{
    const int64_t n_seg = (int64_t)p.B * p.Hkv;
    const int G = p.Hq / p.Hkv;
    const int64_t T = (int64_t)p.prefix[p.B] * p.Hkv;
    for (int64_t seg = seg0; seg < n_seg; seg += stride) {
        const int b = (int)(seg / p.Hkv), kvh = (int)(seg - (int64_t)b * p.Hkv);
        const int pages = p.prefix[b + 1] - p.prefix[b];
        uint16_t *out_seg = p.out + ((int64_t)b * p.Hq + (int64_t)kvh * G) * D;
        if (pages == 0) {
            uint32_t *dst = reinterpret_cast<uint32_t *>(out_seg);
            for (int i = lane; i < G * D / 2; i += 32) dst[i] = 0u;
            continue;
        }
        const int64_t s0 = (int64_t)p.prefix[b] * p.Hkv + (int64_t)kvh * pages;
        int slot0, n_part;
        segment_partials(T, p.n_workers, seg, s0, pages, slot0, n_part);
        merge_rows<D, E2MAX, NB>(p.part_o, p.part_ml, out_seg, G, slot0, n_part, lane);
    }
}

// One warp per (sequence, kv head) segment, a grid of at most one CTA per SM walking the segments:
// every CTA must be resident (waiting for the split-K launch to end) before the launch after this
// one may be scheduled, so the grid has to fit beside the split-K CTAs in one wave.
template <int D>
__global__ void __launch_bounds__(MERGE_WARPS * 32) merge_kernel(MergeParams p)
{
    pdl_trigger();        // nothing after this kernel in the stream needs to wait for its start
    pdl_wait();           // the partials come from the kernel before this one
    const int lane = threadIdx.x & 31;
    const int64_t seg0 = (int64_t)blockIdx.x * MERGE_WARPS + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * MERGE_WARPS;
    const int G = p.Hq / p.Hkv;
    const int E2 = (G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8) * D / 64;   // float2 per lane, see merge_rows
    constexpr int P = SKV_MERGE_PAYLOAD;
    if (E2 <= 2) merge_loop<D, 2, (P / 2 > 16 ? 16 : P / 2)>(p, seg0, stride, lane);
    else if (E2 <= 4) merge_loop<D, 4, (P / 4 > 16 ? 16 : P / 4)>(p, seg0, stride, lane);
    else if (E2 <= 8) merge_loop<D, 8, P / 8>(p, seg0, stride, lane);
    else merge_loop<D, 16, P / 16>(p, seg0, stride, lane);
}

template <int D, class State>
cudaError_t launch_splitk_t(const DecodeParams &p, int G, int grid, int warps, int stages, bool pdl, cudaStream_t s)
{
    const size_t smem = 128 + table_bytes(p.B) + (size_t)warps * stages * State::BLOCK + (size_t)warps * stages * 8 + 16;
    auto kern = decode_splitk_kernel<D, State>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)(warps * 32));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p, G, stages);
}

}  // namespace

size_t decode_smem_bytes(int D, int B, int warps, int stages, bool fp8)
{
    if (D != 64 && D != 128) return 0;
    const size_t blk = fp8 ? fp8_block_bytes(D) : block_bytes(D);
    // 128 bytes of slack for aligning the ring base; 16 bytes for the arrival word
    return 128 + table_bytes(B) + (size_t)warps * stages * blk + (size_t)warps * stages * 8 + 16;
}

cudaError_t launch_decode_splitk(const DecodeParams &p, int D, int G, int kernel, int grid, int warps,
                                 int stages, bool pdl, cudaStream_t s)
{
    if (D == 128) {
        if (kernel == 2) return launch_splitk_t<128, Fp8State<128>>(p, G, grid, warps, stages, pdl, s);
        if (kernel == 1) return launch_splitk_t<128, TensorCoreState<128>>(p, G, grid, warps, stages, pdl, s);
        return launch_splitk_t<128, CudaCoreState<128>>(p, G, grid, warps, stages, pdl, s);
    }
    if (D == 64) {
        if (kernel == 2) return launch_splitk_t<64, Fp8State<64>>(p, G, grid, warps, stages, pdl, s);
        if (kernel == 1) return launch_splitk_t<64, TensorCoreState<64>>(p, G, grid, warps, stages, pdl, s);
        return launch_splitk_t<64, CudaCoreState<64>>(p, G, grid, warps, stages, pdl, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_merge(const MergeParams &p, bool pdl, cudaStream_t s)
{
    const int64_t segs = (int64_t)p.B * p.Hkv;
    cudaLaunchConfig_t cfg = {};
    const int64_t want = (segs + MERGE_WARPS - 1) / MERGE_WARPS;
    cfg.gridDim = dim3((unsigned)(want < p.max_ctas ? want : p.max_ctas));
    cfg.blockDim = dim3(MERGE_WARPS * 32);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (p.D == 128) return cudaLaunchKernelEx(&cfg, merge_kernel<128>, p);
    if (p.D == 64) return cudaLaunchKernelEx(&cfg, merge_kernel<64>, p);
    return cudaErrorInvalidValue;
}

}  // namespace skv
