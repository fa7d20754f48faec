// "Load + Attn" of Algorithm 2 for one new token per sequence (Eq. (3.1)):
// a split-K flash-decoding pass over the owner layer's pages and a
// log-sum-exp merge of the partial results.
//
// Work decomposition.  All (sequence, kv head, page) blocks of the call form
// one flattened list, b-major; it is cut into W equal contiguous ranges, one
// per WARP (W = grid * warps per CTA).  A warp streams its blocks through a
// private shared-memory ring filled by linear bulk copies (one 2*PAGE*D*2-byte
// copy per block, completion on an mbarrier), keeps a running (max, sum, out)
// per query head of the kv head's group, and writes one fp32 partial per
// (sequence, kv head) segment its range touches, to slot  worker + segment.
// Every warp does the same number of blocks (+-1) whatever the length mix, so
// there is no tail; warps never synchronise with each other after the prologue.
#include "skv_common.cuh"

#include <math.h>

namespace skv {

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;

struct Cursor {        // a position in the flattened (b, h, page) list
    int b, h, pg, pages;
};

__device__ __forceinline__ Cursor locate(const int32_t *prefix, int B, int Hkv, int64_t x)
{
    int lo = 0, hi = B - 1;   // smallest b with prefix[b+1]*Hkv > x
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)prefix[mid + 1] * Hkv > x) hi = mid; else lo = mid + 1;
    }
    Cursor c;
    c.b = lo;
    c.pages = prefix[lo + 1] - prefix[lo];
    const int64_t r = x - (int64_t)prefix[lo] * Hkv;
    c.h = (int)(r / c.pages);
    c.pg = (int)(r - (int64_t)c.h * c.pages);
    return c;
}

// Only called while another position remains, so b never runs past B-1.
__device__ __forceinline__ void advance(Cursor &c, const int32_t *prefix, int Hkv)
{
    if (++c.pg < c.pages) return;
    c.pg = 0;
    if (++c.h < Hkv) return;
    c.h = 0;
    do {
        ++c.b;
        c.pages = prefix[c.b + 1] - prefix[c.b];
    } while (c.pages == 0);
}

// Shared-memory carve-up (dynamic): prefix[B+1] | rings | barriers
__host__ __device__ inline size_t prefix_bytes(int B) { return (((size_t)(B + 1) * 4) + 127) & ~(size_t)127; }

// ---------------------------------------------------------------------------
// Per-warp compute state, tensor-core variant: the G query heads of one kv head
// are rows of a 16-row A operand (rows >= G are zero), one page is 16 key
// columns.  S = Q K^T  (m16 n16 k D) and  O += P V  (m16 n D k16) with
// mma.m16n8k16; softmax runs on the accumulator fragment in fp32.
// ---------------------------------------------------------------------------
template <int D>
struct TensorCoreState {
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

    // one page: sK/sV = shared addresses of the K and V halves, valid = tokens in use (1..16)
    __device__ __forceinline__ void page(uint32_t sK, uint32_t sV, int valid, float scale_log2, int lane)
    {
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
// the 16 slots are combined once per segment.
// ---------------------------------------------------------------------------
template <int D>
struct CudaCoreState {
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

    __device__ __forceinline__ void page(uint32_t sK, uint32_t sV, int valid, float scale_log2, int lane)
    {
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

    __device__ __forceinline__ void finish(const DecodeParams &p, int64_t slot, int /*G*/, int lane)
    {
        const int t = lane & 15, hf = lane >> 4;
        float M = m;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, d));
        const float wgt = (m == -INFINITY) ? 0.f : fast_exp2(m - M);
        float lt = l * wgt;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) lt += __shfl_xor_sync(FULL, lt, d);
#pragma unroll
        for (int i = 0; i < D / 2; ++i) {
            float x = o[i] * wgt;
#pragma unroll
            for (int d = 1; d < 16; d <<= 1) x += __shfl_xor_sync(FULL, x, d);
            o[i] = x;
        }
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
// Where the partials of one segment (sequence b, kv head kvh) live.  A static
// range that meets the segment wrote slot  worker + seg;  a pool chunk that
// meets it wrote slot  W + n_seg + chunk + seg.  Lane k of the calling warp
// gets the k-th partial's slot (or -1); returns how many there are.  A segment
// with more than 32 partials is walked in rounds of 32 (`round`).
// ---------------------------------------------------------------------------
__device__ __forceinline__ int partial_slots(const Plan &pl, int64_t W, int64_t n_seg, int64_t s0, int pages,
                                             int64_t seg, int lane, int round, int64_t &slot)
{
    const int64_t s1 = s0 + pages;
    int n_static = 0;
    int64_t w_first = 0;
    const bool sparse = pl.Ts < W;            // then every non-empty static range is a single block
    if (s0 < pl.Ts) {
        const int64_t e = s1 < pl.Ts ? s1 : pl.Ts;
        if (sparse) {
            n_static = (int)(e - s0);
        } else {
            w_first = worker_of(s0, pl.Ts, W);
            n_static = worker_of(e - 1, pl.Ts, W) - (int)w_first + 1;
        }
    }
    int n_pool = 0;
    int64_t j_first = 0;
    if (s1 > pl.Ts && pl.n_chunks > 0) {
        const int64_t a = s0 > pl.Ts ? s0 : pl.Ts;
        j_first = (a - pl.Ts) / pl.chunk;
        n_pool = (int)((s1 - 1 - pl.Ts) / pl.chunk - j_first) + 1;
    }
    const int k = round * 32 + lane;
    slot = -1;
    if (k < n_static) slot = (sparse ? (int64_t)worker_of(s0 + k, pl.Ts, W) : w_first + k) + seg;
    else if (k < n_static + n_pool) slot = W + n_seg + j_first + (k - n_static) + seg;
    return n_static + n_pool;
}

// Log-sum-exp merge of one segment's partials for its G query heads, by one warp:
// out[b, kvh*G+g, :] = sum_i 2^(m_i - M) o_i / sum_i 2^(m_i - M) l_i,  M = max_i m_i.
template <int D>
__device__ __noinline__ void merge_segment(const float *part_o, const float *part_ml, uint16_t *out,
                                              const Plan &pl, int64_t W, int B, int Hq, int Hkv, int b, int kvh,
                                              int64_t s0, int pages, int lane)
{
    constexpr int PER = D / 32;               // consecutive output dims per lane
    const int G = Hq / Hkv;
    const int64_t seg = (int64_t)b * Hkv + kvh, n_seg = (int64_t)B * Hkv;
    int64_t slot;
    const int n = partial_slots(pl, W, n_seg, s0, pages, seg, lane, 0, slot);
    for (int g = 0; g < G; ++g) {
        float acc[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) acc[i] = 0.f;
        float M = -INFINITY, L = 0.f;
        for (int r = 0; r * 32 < n; ++r) {
            int64_t my = slot;
            if (r > 0) partial_slots(pl, W, n_seg, s0, pages, seg, lane, r, my);
            // this round's (max, sum) pairs, one partial per lane
            float2 ml = make_float2(-INFINITY, 0.f);
            if (my >= 0) ml = __ldcg(reinterpret_cast<const float2 *>(part_ml + (my * G + g) * 2));
            float Mr = ml.x;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) Mr = fmaxf(Mr, __shfl_xor_sync(FULL, Mr, d));
            const float M_new = fmaxf(M, Mr);
            const float keep = exp2f(M - M_new);          // 0 on the first round
            const float wt = (my >= 0) ? exp2f(ml.x - M_new) : 0.f;
            float Lr = wt * ml.y;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) Lr += __shfl_xor_sync(FULL, Lr, d);
            L = L * keep + Lr;
            M = M_new;
#pragma unroll
            for (int i = 0; i < PER; ++i) acc[i] *= keep;
            const int cnt = (n - r * 32) < 32 ? (n - r * 32) : 32;
            for (int i0 = 0; i0 < cnt; i0 += 4) {
                float v[4][PER], wv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = (i0 + u) < cnt ? (i0 + u) : i0;       // clamp: weight 0 below
                    const int64_t sl = __shfl_sync(FULL, my, i);
                    wv[u] = (i0 + u) < cnt ? __shfl_sync(FULL, wt, i) : 0.f;
                    const float *po = part_o + (sl * G + g) * D + lane * PER;
                    if constexpr (PER == 4) {
                        const float4 t = __ldcg(reinterpret_cast<const float4 *>(po));
                        v[u][0] = t.x; v[u][1] = t.y; v[u][2] = t.z; v[u][3] = t.w;
                    } else {
                        const float2 t = __ldcg(reinterpret_cast<const float2 *>(po));
                        v[u][0] = t.x; v[u][1] = t.y;
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int i = 0; i < PER; ++i) acc[i] = fmaf(wv[u], v[u][i], acc[i]);
            }
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        uint16_t *dst = out + ((int64_t)b * Hq + (int64_t)kvh * G + g) * D + lane * PER;
#pragma unroll
        for (int i = 0; i < PER; i += 2)
            *reinterpret_cast<uint32_t *>(dst + i) = pack_bf16x2(acc[i] * inv, acc[i + 1] * inv);
    }
}

// ---------------------------------------------------------------------------
template <int D, class State>
__global__ void decode_splitk_kernel(DecodeParams p, int G, int stages)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = block_bytes(D);
    constexpr int QLEN = 8;                   // per-warp queue of range ids between producer and consumer
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint64_t t_entry = p.trace ? global_timer_ns() : 0;
    uint64_t t_first = 0;

    // carve shared memory: prefix | rings | barriers | range queues  (ring base rounded up to 128 bytes)
    const uint32_t base = smem_u32(smem_raw);
    const uint32_t pad = (128u - (base & 127u)) & 127u;
    int32_t *prefix = reinterpret_cast<int32_t *>(smem_raw + pad);
    const size_t rings_off = pad + prefix_bytes(p.B);
    const uint32_t rings = base + (uint32_t)rings_off;
    const uint32_t ring = rings + (uint32_t)(warp * stages * BLOCK);
    const size_t bars_off = rings_off + (size_t)nwarps * stages * BLOCK;
    const uint32_t bars = base + (uint32_t)bars_off + (uint32_t)(warp * stages * 8);
    int32_t *queue = reinterpret_cast<int32_t *>(smem_raw + bars_off + (size_t)nwarps * stages * 8) + warp * QLEN;

    if (lane == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(bars + 8 * s, 1);
        fence_barrier_init();
    }
    // cumulative page counts of the batch (warp 0), visible to every warp after the barrier
    if (warp == 0) {
        int carry = 0;
        for (int i0 = 0; i0 < p.B; i0 += 32) {
            const int i = i0 + lane;
            int v = 0;
            if (i < p.B) {
                const int n = __ldg(p.seq_lens + i);
                v = n > 0 ? (n + PAGE - 1) / PAGE : 0;
            }
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(FULL, v, d);
                if (lane >= d) v += u;
            }
            if (i < p.B) prefix[i + 1] = carry + v;
            carry += __shfl_sync(FULL, v, 31);
        }
        if (lane == 0) prefix[0] = 0;
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i <= p.B; i += blockDim.x) p.prefix[i] = prefix[i];
        if (p.out) {     // fused merge: rows of empty sequences are zero and belong to nobody else
            const int row_words = p.Hq * D / 2;
            for (int b = 0; b < p.B; ++b)
                if (prefix[b + 1] == prefix[b])
                    for (int i = threadIdx.x; i < row_words; i += blockDim.x)
                        reinterpret_cast<uint32_t *>(p.out)[(int64_t)b * row_words + i] = 0u;
        }
    }

    const int64_t W = (int64_t)gridDim.x * nwarps, w = (int64_t)blockIdx.x * nwarps + warp;
    const int64_t n_seg = (int64_t)p.B * p.Hkv;
    const Plan pl = make_plan((int64_t)prefix[p.B] * p.Hkv, p.bal);
    if (pl.T == 0) return;
    const bool pooled = pl.n_chunks > 0;

    // static range of this worker
    const int64_t x0 = worker_begin(w, pl.Ts, W);
    const int n_static = (int)(worker_begin(w + 1, pl.Ts, W) - x0);
    // first pool claim, requested now and looked at only when the static range has been issued
    int next_j = 0;
    if (pooled && lane == 0) next_j = atomicAdd(p.ctrl, 1);

    // ---- producer: walks ranges (static, then claimed chunks) and keeps the ring full ----
    Cursor prod = {0, 0, 0, 0};
    int prod_left = 0, q_tail = 0, in_flight = 0, p_stage = 0;
    bool static_given = false, prod_done = false;
    int win_b = -1, win_base = 0, win_ids = 0;   // page ids of the current sequence, 32 at a time, one per lane
    auto issue = [&]() -> bool {
        if (prod_done) return false;
        if (prod_left == 0) {
            int id = -1, cnt = 0;
            int64_t begin = 0;
            if (!static_given) {
                static_given = true;
                begin = x0;
                cnt = n_static;
            }
            if (cnt == 0 && pooled) {
                const int j = __shfl_sync(FULL, next_j, 0);
                if (j < pl.n_chunks) {
                    if (lane == 0) next_j = atomicAdd(p.ctrl, 1);
                    id = j;
                    begin = pl.Ts + (int64_t)j * pl.chunk;
                    const int64_t rest = pl.T - begin;
                    cnt = rest < pl.chunk ? (int)rest : pl.chunk;
                }
            }
            if (cnt == 0) {
                prod_done = true;
                return false;
            }
            if (lane == 0) queue[q_tail & (QLEN - 1)] = id;
            ++q_tail;
            prod = locate(prefix, p.B, p.Hkv, begin);
            prod_left = cnt;
        }
        if (prod.b != win_b || prod.pg < win_base || prod.pg >= win_base + 32) {
            win_b = prod.b;
            win_base = prod.pg;
            const int i = prod.pg + lane;
            win_ids = (i < prod.pages) ? __ldg(p.page_table + (int64_t)prod.b * p.pt_stride + i) : 0;
        }
        int id = __shfl_sync(FULL, win_ids, prod.pg - win_base);
        if (lane == 0) {
            if (id < 0 || (int64_t)id >= p.max_pages) {
                atomicOr(p.status, STATUS_BOUNDS);
                id = 0;
            }
            const uint8_t *src = p.layer_base + (int64_t)id * p.page_stride + (int64_t)prod.h * BLOCK;
            const uint32_t bar = bars + 8 * p_stage;
            mbar_expect_tx(bar, BLOCK);
            bulk_copy_g2s(ring + (uint32_t)(p_stage * BLOCK), src, BLOCK, bar);
        }
        if (++p_stage == stages) p_stage = 0;
        ++in_flight;
        if (--prod_left > 0) advance(prod, prefix, p.Hkv);
        return true;
    };
    // the queue holds at most `stages`+1 ranges: a range is queued only when one of its blocks is issued
    while (in_flight < stages && issue()) {}

    // ---- consumer ----
    State st;
    Cursor cons = {0, 0, 0, 0};
    int cons_left = 0, q_head = 0, c_stage = 0, run_pages = 0, n_b = 0;
    int64_t slot_base = 0;
    uint32_t parity = 0;
    bool fresh = true, first = true, failed = false;
    while (in_flight > 0) {
        if (cons_left == 0) {
            __syncwarp();
            const int id = queue[q_head & (QLEN - 1)];
            ++q_head;
            int64_t begin;
            if (id < 0) {
                begin = x0;
                cons_left = n_static;
                slot_base = w;
            } else {
                begin = pl.Ts + (int64_t)id * pl.chunk;
                const int64_t rest = pl.T - begin;
                cons_left = rest < pl.chunk ? (int)rest : pl.chunk;
                slot_base = W + n_seg + id;
            }
            cons = locate(prefix, p.B, p.Hkv, begin);
            fresh = true;
        }
        if (fresh) {
            st.begin(p, cons.b, cons.h, G, lane);
            n_b = __ldg(p.seq_lens + cons.b);
            run_pages = 0;
            fresh = false;
        }
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
        if (p.trace && first) t_first = global_timer_ns();
        first = false;
        const uint32_t sK = ring + (uint32_t)(c_stage * BLOCK);
        const int left = n_b - cons.pg * PAGE;
        st.page(sK, sK + half_bytes(D), left < PAGE ? left : PAGE, p.scale_log2, lane);
        __syncwarp();                       // every lane is done reading this stage
        --in_flight;
        issue();                            // refill it
        if (++c_stage == stages) { c_stage = 0; parity ^= 1u; }
        ++run_pages;
        --cons_left;
        if (cons.pg + 1 == cons.pages || cons_left == 0) {
            // this worker's run inside segment (b, h) ends: publish the partial
            const int64_t seg = (int64_t)cons.b * p.Hkv + cons.h;
            st.finish(p, slot_base + seg, G, lane);
            if (p.out) {
                // the worker that completes the segment's block count merges it
                __threadfence();
                __syncwarp();
                int done = 0;
                if (lane == 0) done = atomicAdd(p.seg_count + seg, run_pages) + run_pages;
                done = __shfl_sync(FULL, done, 0);
                if (done == cons.pages) {
                    __threadfence();
                    const int64_t s0 = (int64_t)prefix[cons.b] * p.Hkv + (int64_t)cons.h * cons.pages;
                    merge_segment<D>(p.part_o, p.part_ml, p.out, pl, W, p.B, p.Hq, p.Hkv, cons.b, cons.h, s0,
                                     cons.pages, lane);
                    if (lane == 0) p.seg_count[seg] = 0;
                }
            }
            fresh = true;
        }
        if (cons_left > 0) advance(cons, prefix, p.Hkv);
    }
    (void)failed;
    // the last worker to leave puts the two counters back to zero for the next launch
    if (pooled && lane == 0) {
        if (atomicAdd(p.ctrl + 1, 1) == (int)W - 1) {
            p.ctrl[0] = 0;
            p.ctrl[1] = 0;
        }
    }
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
template <int D>
__global__ void __launch_bounds__(128) merge_kernel(MergeParams p)
{
    const int lane = threadIdx.x & 31;
    const int64_t seg = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (seg >= (int64_t)p.B * p.Hkv) return;
    const int b = (int)(seg / p.Hkv), kvh = (int)(seg - (int64_t)b * p.Hkv);
    const int pages = p.prefix[b + 1] - p.prefix[b];
    const int G = p.Hq / p.Hkv;
    if (pages == 0) {
        uint32_t *dst = reinterpret_cast<uint32_t *>(p.out + ((int64_t)b * p.Hq + (int64_t)kvh * G) * D);
        for (int i = lane; i < G * D / 2; i += 32) dst[i] = 0u;
        return;
    }
    const Plan pl = make_plan((int64_t)p.prefix[p.B] * p.Hkv, p.bal);
    const int64_t s0 = (int64_t)p.prefix[b] * p.Hkv + (int64_t)kvh * pages;
    merge_segment<D>(p.part_o, p.part_ml, p.out, pl, p.n_workers, p.B, p.Hq, p.Hkv, b, kvh, s0, pages, lane);
}

template <int D, class State>
cudaError_t launch_splitk_t(const DecodeParams &p, int G, int grid, int warps, int stages, cudaStream_t s)
{
    const size_t smem = decode_smem_bytes(D, p.B, warps, stages);
    auto kern = decode_splitk_kernel<D, State>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, warps * 32, smem, s>>>(p, G, stages);
    return cudaGetLastError();
}

}  // namespace

size_t decode_smem_bytes(int D, int B, int warps, int stages)
{
    if (D != 64 && D != 128) return 0;
    // 128 bytes of slack for aligning the ring base; 8 queue entries per warp
    return 128 + prefix_bytes(B) + (size_t)warps * stages * block_bytes(D) + (size_t)warps * stages * 8 +
           (size_t)warps * 8 * 4;
}

cudaError_t launch_decode_splitk(const DecodeParams &p, int D, int G, bool tensor_core, int grid, int warps,
                                 int stages, cudaStream_t s)
{
    if (D == 128) {
        if (tensor_core) return launch_splitk_t<128, TensorCoreState<128>>(p, G, grid, warps, stages, s);
        return launch_splitk_t<128, CudaCoreState<128>>(p, G, grid, warps, stages, s);
    }
    if (D == 64) {
        if (tensor_core) return launch_splitk_t<64, TensorCoreState<64>>(p, G, grid, warps, stages, s);
        return launch_splitk_t<64, CudaCoreState<64>>(p, G, grid, warps, stages, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_merge(const MergeParams &p, cudaStream_t s)
{
    const int64_t segs = (int64_t)p.B * p.Hkv;
    const unsigned blocks = (unsigned)((segs + 3) / 4);
    if (p.D == 128) merge_kernel<128><<<blocks, 128, 0, s>>>(p);
    else if (p.D == 64) merge_kernel<64><<<blocks, 128, 0, s>>>(p);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace skv
