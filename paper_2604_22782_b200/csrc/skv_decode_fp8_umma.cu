// Decode attention ("Load + Attn" of Algorithm 2, Eq. (3.1)) over FP8 pages on the 5th-generation
// tensor cores: both contractions are tcgen05 instructions of kind f8f6f4 that read the stored E4M3
// codes straight from shared memory, so no code is ever converted.  Same split-K scheme and the same
// partial format as skv_decode.cu (the merge kernel is shared); here a worker is a CTA and the unit
// of work is a TILE: pages [8i, 8i+8) (128 tokens) of one (sequence, kv head) segment.  The list
// that is cut into equal contiguous ranges is the list of tiles.
//
// Per tile, with the tokens as the M dimension (TMEM lanes):
//   S^T[128 tokens x 16]  = Kc[128 x D] . Q'^T[D x 16]          4 instructions (K = 32 dims each)
//   O^T[D dims x 16]     += Vc^T[D x 32 tokens] . P'^T[32 x 16]  1 instruction per 2 pages
// The other operand must be E4M3 too, so it is split into a leading E4M3 term and an E4M3 remainder,
// and the two terms take the 16 columns: column h = leading term of head h, column 8 + h =
// remainder of head h (h < G <= 8); the softmax adds the two columns.
//   Q' = Q 2^k, the power of two that brings the row's maximum into [128, 256): a bf16 number times
//        a power of two has 8 significant bits, which 4 + 4 hold exactly (but for the smallest elements);
//   P' = 32 p vscale / 2^ref, leading term rounded to 4 significant bits, remainder times 16.
// The per-token scales stay outside the contractions:  score_t = 2^-k kscale_t (S_h + S_{8+h}).
// The reference of head h follows  e_t = score_t + log2(vscale_t), the size of the token's term in
// the output, and only moves when the maximum of e has grown by more than 2^3.5: P' <= 362 fits E4M3
// whatever the spread of the V scales, O^T is rescaled (through registers) rarely, and the partial
// (reference, sum of 2^(score - reference), O^T / 32) is in the merge kernel's usual form.
//
// Six warps:
//   warps 0-3  softmax: thread t owns token t of the tile (TMEM lane t); at the end of a run thread
//              d owns dim d of O^T
//   warp 4     lane 0 issues the tensor-core instructions
//   warp 5     walks the worker's tiles, prepares Q' of every new segment, issues the copies
// Shared memory: a K ring and a V ring of two stages each.  A K stage holds the K parts of the
// tile's pages side by side (page j at j * 2048: [8-token group][16-dim chunk][8 tokens][16 B], the
// K-major core-matrix layout the pages are stored in, so the 128 tokens form ONE A operand with a
// uniform group stride) and is given back by the tile's score instructions; a V stage holds the
// V-and-scales parts (page j at j * 2176: [dim][16 tokens] = K-major core matrices of V^T, then the
// K and V scales) and is given back by the tile's value instructions.  Two P' operands (N-major:
// a token's 16 bytes are one row), one Q' operand.  Tensor memory (64 columns): two S^T buffers, O^T.
// Waiting threads are suspended (try_wait with a time hint), not polling.  Every wait is bounded;
// after a timeout the roles leave through the common exit, where copies in flight get their
// (bounded) wait and the tensor memory is freed.
#include "skv_common.cuh"
#include "skv_tcgen05.cuh"
#include "skv_walk.cuh"

#include <math.h>

namespace skv {

namespace {

using namespace tc5;

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int TP = 8;                  // pages per tile: 128 tokens, the height of the instructions
constexpr int NST = 2;                 // stages of the K ring and of the V ring
constexpr int THREADS = 192;
constexpr int COL_O = 32;              // S^T buffers at columns 0 and 16
constexpr int TMEM_COLS = 64;
constexpr float RESCALE_STEP = 3.5f;    // p <= 2^3.5 between moves of the reference: P' = 32 p vscale / c <= 362 fits E4M3 (max 448)
constexpr float P_SCALE = 32.f, REM_SCALE = 16.f;
constexpr int CTAS_PER_SM = 3;

constexpr int TILE_FIRST = 1, TILE_LAST = 2, TILE_END = 4;
struct alignas(16) TileMeta {
    int n_pages;        // 1..8
    int short_slot;     // page slot whose page is the sequence's last, partly filled one (-1: none)
    int short_valid;    // tokens in use in that page
    int flags;          // TILE_FIRST / TILE_LAST of a run inside a segment, TILE_END of the worker
    int b, h;           // the segment
    int qbuf;           // which of the two sets of query scales belongs to the segment
    int pad;
};

// a tile's description as its consumers read it (after their wait on the stage's barrier)
__device__ __forceinline__ TileMeta load_meta(const TileMeta *m)
{
    TileMeta r;
    const uint32_t a = smem_u32(m);
    asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(r.n_pages), "=r"(r.short_slot), "=r"(r.short_valid), "=r"(r.flags) : "r"(a) : "memory");
    asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(r.b), "=r"(r.h), "=r"(r.qbuf), "=r"(r.pad) : "r"(a + 16) : "memory");
    return r;
}

__device__ __forceinline__ void f16x2_to_f32(uint32_t w, float &lo, float &hi)
{
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}"
        : "=f"(lo), "=f"(hi) : "r"(w));
}

// four fp32 -> one word of E4M3 codes (round to nearest even, saturating) and the values of the codes
__device__ __forceinline__ uint32_t e4m3x4_round(const float (&x)[4], float (&back)[4])
{
    const uint32_t w = pack_e4m3x2(x[0], x[1]) | (pack_e4m3x2(x[2], x[3]) << 16);
    uint32_t h01, h23;
    e4m3x4_to_f16x2(w, h01, h23);
    f16x2_to_f32(h01, back[0], back[1]);
    f16x2_to_f32(h23, back[2], back[3]);
    return w;
}

// order-preserving map float <-> signed int (its own inverse)
__device__ __forceinline__ int float_key(float f)
{
    const int i = __float_as_int(f);
    return i ^ ((i >> 31) & 0x7FFFFFFF);
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k ^ ((k >> 31) & 0x7FFFFFFF)); }

__device__ __forceinline__ int warp_max_s32(int v)
{
    int r;
    asm volatile("redux.sync.max.s32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
}

// barrier over the 128 softmax threads
__device__ __forceinline__ void softmax_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// ... that also tells whether every one of them passed `ok`
__device__ __forceinline__ bool softmax_all(bool ok)
{
    int r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbar.red.and.pred q, 1, 128, p;\n\tselp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((int)ok) : "memory");
    return r != 0;
}

// Waits that leave the issue slots to the warps that have work: the thread is suspended until the phase
// completes or `ns` nanoseconds have passed (a plain try_wait comes back at once, and six waiting warps
// per CTA polling in a loop slowed the softmax warps down several times).
__device__ __forceinline__ bool try_wait_for(uint32_t bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// bounded (about two seconds), suspended while waiting
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity)
{
    if (try_wait_for(bar, parity, 2000u)) return true;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        __nanosleep(64);
        if (try_wait_for(bar, parity, 10000u)) return true;
        if (global_timer_ns() - t0 > 2000000000ull) return false;
    }
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int D, int GP>   // GP: the group size rounded up to a power of two (the softmax loops run over GP heads)
// (bounds as for four CTAs per SM = 80 registers: shared memory admits three, and the registers left over let
// a CTA of the merge kernel become resident beside them, which the launch chain needs to move on)
__global__ void __launch_bounds__(THREADS, CTAS_PER_SM + 1) decode_fp8_umma_kernel(DecodeParams p, int G)
{
    static_assert(D == 128, "the tile shapes below are those of head_dim 128");
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = fp8_block_bytes(D);          // 4224: K codes | V codes | K scales | V scales
    constexpr int K_PAGE = PAGE * D;                   // 2048
    constexpr int V_PAGE = BLOCK - K_PAGE;             // 2176
    constexpr int K_STAGE = TP * K_PAGE, V_STAGE = TP * V_PAGE;
    constexpr int Q_BYTES = 16 * D;                    // the Q' operand: 16 rows (8 leading, 8 remainder) x D
    constexpr int P_BYTES = 16 * TP * PAGE;            // one P' operand: 16 rows x 128 tokens
    constexpr uint32_t IDESC = instr_desc_e4m3(128, 16);
    constexpr uint32_t IDESC_PV = IDESC | (1u << 16);   // P' is N-major: a token's 16 bytes (the N index) are contiguous

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    int32_t *prefix = reinterpret_cast<int32_t *>(base);
    int32_t *lens = prefix + p.B + 1;
    uint8_t *at = base + table_bytes(p.B);
    const uint32_t k_ring = smem_u32(at);              at += NST * K_STAGE;
    const uint32_t v_ring = smem_u32(at);
    const uint8_t *v_ring_ptr = at;                    at += NST * V_STAGE;
    const uint32_t p_sm = smem_u32(at);
                                                       at += 2 * P_BYTES;
    const uint32_t q_sm = smem_u32(at);                at += Q_BYTES;
    TileMeta *meta = reinterpret_cast<TileMeta *>(at); at += 4 * sizeof(TileMeta);
    float *qscale = reinterpret_cast<float *>(at);     at += 2 * 8 * 4;
    int *red = reinterpret_cast<int *>(at);            at += 2 * 64 * 4;      // two sets of [8 head maxima, 1 vscale maximum][4 softmax warps]
    float *red_l = reinterpret_cast<float *>(at);      at += 4 * 8 * 4;
    const uint32_t bars = smem_u32(at);                at += 16 * 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(at);
    int *gave_up = reinterpret_cast<int *>(at + 4);
    const uint32_t k_full = bars, k_empty = bars + 16, v_full = bars + 32, v_empty = bars + 48, s_ready = bars + 64,
                   p_ready = bars + 80, pv_done = bars + 96, q_full = bars + 112;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(k_full + 8 * i, 1);
            mbar_init(k_empty + 8 * i, 1);
            mbar_init(v_full + 8 * i, 1);
            mbar_init(v_empty + 8 * i, 1);
            mbar_init(s_ready + 8 * i, 1);
            mbar_init(p_ready + 8 * i, 4);
            mbar_init(pv_done + 8 * i, 1);
        }
        mbar_init(q_full, 1);
        *gave_up = 0;
        fence_barrier_init();
    }
    if (warp == 4) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    const bool late_wait = (p.flags & DECODE_LATE_WAIT) != 0;
    const bool reverse = (p.flags & DECODE_REVERSE) != 0;
    if (!late_wait) pdl_wait();            // anything read below may come from the kernel before this one
    const unsigned long long t_entry = p.trace ? global_timer_ns() : 0ull;

    // Sequence lengths and cumulative TILE counts of the batch (warp 0), visible to all after the barrier.  The
    // flattened list that is cut into equal ranges is the list of (sequence, kv head, tile) here, a tile
    // being pages [8i, 8i+8) of the sequence: equal ranges are then equal numbers of tiles, which is what a
    // CTA's time goes with.  The merge kernel is told the same counts, so it finds the partials as usual.
    if (warp == 0) scan_lengths(p.seq_lens, p.B, TP * PAGE, (int64_t)p.pt_stride * PAGE, p.status, prefix, lens, lane);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (blockIdx.x == 0)       // the merge kernel reads the counts from global memory
        for (int i = tid; i <= p.B; i += THREADS) p.prefix[i] = prefix[i];

    const int64_t W = gridDim.x, w = blockIdx.x;
    const int64_t T = (int64_t)prefix[p.B] * p.Hkv;
    int64_t x0 = 0;
    int n = 0;
    if (T > 0) {
        x0 = worker_begin(w, T, W);
        n = (int)(worker_begin(w + 1, T, W) - x0);
    }
    const int64_t x_first = reverse ? x0 + n - 1 : x0;
    int tiles_issued = 0;                  // producer's count, used at the exit

    if (warp == 5) {
        // ================= producer =================
        const uint64_t pol_stream = make_policy_evict_first(), pol_keep = make_policy_evict_normal();
        const int keep_from = (p.keep_pct > 0 && T * TP <= p.l2_fit_blocks) ? 0 : n - (int)(((int64_t)n * p.keep_pct) / 100);
        // Where the launch after this one may be scheduled (and, in a chain of calls, where this one waits for
        // the launch before it): at 7/8 of the range, not at the middle as the warp-per-worker kernel does --
        // the CTAs of this kernel are one wave, and CTAs of the next launch that got in early would only sit
        // on their wait.
        const int trigger_at = n - n / 8;
        bool triggered = false;
        Cursor cur = {0, 0, 0, 1};
        if (n > 0) cur = locate(prefix, p.B, p.Hkv, x_first);
        int left = n, k = 0, runs = 0;
        auto give_up = [&]() { if (lane == 0) { atomicOr(p.status, STATUS_TIMEOUT); *gave_up = 1; } };
        while (left > 0) {
            if (!triggered && k >= trigger_at) {
                triggered = true;
                if (lane == 0) {
                    if (late_wait) pdl_wait();
                    pdl_trigger();
                }
                __syncwarp();
            }
            const int s = k & 1;
            // tile cur.pg of segment (cur.b, cur.h): pages [8 cur.pg, 8 cur.pg + np)
            const int b = cur.b, h = cur.h, n_b = lens[b], pages = (n_b + PAGE - 1) / PAGE, pg0 = TP * cur.pg;
            const int np = pages - pg0 < TP ? pages - pg0 : TP;
            const bool first = (k == 0) || (reverse ? cur.pg == cur.pages - 1 : cur.pg == 0);
            const bool last = (left == 1) || (reverse ? cur.pg == 0 : cur.pg == cur.pages - 1);
            // page ids of the tile (lane j < np), fetched before the waits for the stages
            int id = 0;
            if (lane < np) {
                id = __ldg(p.page_table + (int64_t)b * p.pt_stride + pg0 + lane);
                if (id < 0 || (int64_t)id >= p.max_pages) {
                    atomicOr(p.status, STATUS_BOUNDS);
                    id = 0;
                }
            }
            const uint8_t *src = p.layer_base + (int64_t)id * p.page_stride + (int64_t)h * BLOCK;
            const uint64_t pol = (k >= keep_from) ? pol_keep : pol_stream;
            // K part: its stage comes back as soon as the scores of the tile two before this one are done
            if (k >= 2 && !__all_sync(FULL, wait_bounded(k_empty + 8 * s, (uint32_t)((k / 2 - 1) & 1)))) { give_up(); break; }
            if (lane == 0) {
                TileMeta m;
                m.n_pages = np;
                const int short_valid = n_b - (pages - 1) * PAGE;      // 1..16 tokens in the sequence's last page
                const int last_pg_slot = (pages - 1) - pg0;             // its slot, if it is in this tile
                m.short_slot = (short_valid < PAGE && last_pg_slot < np) ? last_pg_slot : -1;
                m.short_valid = short_valid;
                m.flags = (first ? TILE_FIRST : 0) | (last ? TILE_LAST : 0) | (left == 1 ? TILE_END : 0);
                m.b = b;
                m.h = h;
                m.qbuf = (first ? runs : runs - 1) & 1;                // which set of query scales
                m.pad = 0;
                meta[k & 3] = m;       // (four slots: a slot's last readers finished before the tile two back gave its V stage back)
                mbar_expect_tx(k_full + 8 * s, (uint32_t)(np * K_PAGE));
            }
            __syncwarp();
            if (lane < np) bulk_copy_g2s_hint(k_ring + (uint32_t)(s * K_STAGE + lane * K_PAGE), src, K_PAGE, k_full + 8 * s, pol);
            // V part and scales: that stage is held until the tile's value instructions are done
            if (k >= 2 && !__all_sync(FULL, wait_bounded(v_empty + 8 * s, (uint32_t)((k / 2 - 1) & 1)))) { give_up(); break; }
            if (lane == 0) mbar_expect_tx(v_full + 8 * s, (uint32_t)(np * V_PAGE));
            __syncwarp();
            if (lane < np) bulk_copy_g2s_hint(v_ring + (uint32_t)(s * V_STAGE + lane * V_PAGE), src + K_PAGE, V_PAGE, v_full + 8 * s, pol);
            if (first) {
                // Q' of the new segment: lane = (head g, quarter of the dims); rows g >= G are zero.  The single
                // buffer is free once the scores of the previous tile (the last one of the previous run) are done;
                // the two sets of scales alternate (the set's last reader finished before the V stage came back).
                if (k >= 1 && !__all_sync(FULL, wait_bounded(k_empty + 8 * ((k - 1) & 1), (uint32_t)(((k - 1) / 2) & 1)))) { give_up(); break; }
                const int qset = runs & 1;
                const int g = lane >> 2, qd = lane & 3;
                float q[32];
                float amax = 0.f;
                if (g < G) {
                    const uint4 *qsrc = reinterpret_cast<const uint4 *>(p.Q + ((int64_t)b * p.Hq + (int64_t)h * G + g) * D + 32 * qd);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint4 wq = __ldg(qsrc + c);
                        q[8 * c + 0] = bf16_lo(wq.x); q[8 * c + 1] = bf16_hi(wq.x);
                        q[8 * c + 2] = bf16_lo(wq.y); q[8 * c + 3] = bf16_hi(wq.y);
                        q[8 * c + 4] = bf16_lo(wq.z); q[8 * c + 5] = bf16_hi(wq.z);
                        q[8 * c + 6] = bf16_lo(wq.w); q[8 * c + 7] = bf16_hi(wq.w);
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(q[i]));
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) q[i] = 0.f;
                }
                amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 1));
                amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 2));
                // scaled by the power of two that brings the row's maximum into [128, 256): a bf16 number times a
                // power of two has 8 significant bits, which the two E4M3 terms (4 + 4) hold exactly
                const uint32_t be = __float_as_uint(amax) >> 23;          // biased exponent (amax >= 0)
                const bool tiny = be < 8u;                                // zero (or next to it): the row counts as zero
                const float inv = tiny ? 0.f : __uint_as_float((261u - be) << 23);      // 2^(7 - e)
                const float back_q = tiny ? 0.f : __uint_as_float((be - 7u) << 23);     // 2^(e - 7)
                const uint32_t qdst = q_sm + (uint32_t)(g * 16);
#pragma unroll
                for (int c = 0; c < 2; ++c) {               // 16-dim chunk 2 qd + c
                    uint32_t lead[4], rem[4];
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        float x[4], back[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) x[i] = q[16 * c + 4 * v4 + i] * inv;
                        lead[v4] = e4m3x4_round(x, back);
#pragma unroll
                        for (int i = 0; i < 4; ++i) x[i] -= back[i];
                        rem[v4] = e4m3x4_round(x, back);
                    }
                    const uint32_t a = qdst + (uint32_t)((2 * qd + c) * 128);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(lead[0]), "r"(lead[1]), "r"(lead[2]), "r"(lead[3]) : "memory");
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a + 1024u), "r"(rem[0]), "r"(rem[1]), "r"(rem[2]), "r"(rem[3]) : "memory");
                }
                if (qd == 0) qscale[qset * 8 + g] = back_q * p.scale_log2;
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(q_full);
                ++runs;
            }
            ++k;
            tiles_issued = k;
            if (--left > 0) step(cur, prefix, p.Hkv, reverse);
        }
        if (!triggered && lane == 0) {
            if (late_wait) pdl_wait();
            pdl_trigger();
        }
    } else if (warp == 4) {
        // ================= tensor-core issue =================
        // Per tile k: the scores need the tile's K stage (and Q' of a new segment), the values of tile k-1 need
        // its probabilities; whichever is ready first is issued first, so that neither a late copy nor a busy
        // softmax holds the other up.  A K stage is given back by the tile's scores, a V stage by its values.
        if (lane == 0 && n > 0) {
            int prev_np = 0, prev_first = 0, runs = 0;
            bool ok = true;
            auto issue_pv = [&](int j, int np_j, int first_j) -> bool {
                const int sj = j & 1;
                if (!wait_bounded(v_full + 8 * sj, (uint32_t)((j >> 1) & 1))) return false;   // long over: the softmax read the scales
                tc_fence_after();
                const uint32_t vbase = v_ring + (uint32_t)(sj * V_STAGE), pbase = p_sm + (uint32_t)(sj * P_BYTES);
                const int nks = (np_j + 1) >> 1;
                for (int ks = 0; ks < nks; ++ks)
                    umma_ss_f8(tmem + COL_O, smem_desc(vbase + (uint32_t)(ks * 2 * V_PAGE), V_PAGE, 128),
                               smem_desc(pbase + (uint32_t)(ks * 512), 128, 128), IDESC_PV, (first_j && ks == 0) ? 0u : 1u);
                tc_commit(pv_done + 8 * sj);
                tc_commit(v_empty + 8 * sj);
                return true;
            };
            for (int k = 0; ok; ++k) {
                const int s = k & 1;
                bool qk_issued = false, pv_issued = (k == 0);
                TileMeta m = {};
                const uint64_t t0 = global_timer_ns();
                for (int spin = 0; ok && !(qk_issued && pv_issued); ++spin) {
                    if (!pv_issued && try_wait_for(p_ready + 8 * ((k - 1) & 1), (uint32_t)(((k - 1) >> 1) & 1), qk_issued ? 2000u : 200u)) {
                        ok = issue_pv(k - 1, prev_np, prev_first);
                        pv_issued = true;
                    }
                    if (ok && !qk_issued && try_wait_for(k_full + 8 * s, (uint32_t)((k >> 1) & 1), pv_issued ? 2000u : 200u)) {
                        m = load_meta(&meta[k & 3]);
                        if (m.flags & TILE_FIRST) {
                            ok = wait_bounded(q_full, (uint32_t)(runs & 1));
                            if (!ok) break;
                            ++runs;
                        }
                        tc_fence_after();
                        const uint32_t kbase = k_ring + (uint32_t)(s * K_STAGE);
#pragma unroll
                        for (int ks = 0; ks < D / 32; ++ks)
                            umma_ss_f8(tmem + (uint32_t)(16 * s), smem_desc(kbase + (uint32_t)(ks * 256), 128, 1024),
                                       smem_desc(q_sm + (uint32_t)(ks * 256), 128, 1024), IDESC, ks > 0 ? 1u : 0u);
                        tc_commit(s_ready + 8 * s);
                        tc_commit(k_empty + 8 * s);
                        qk_issued = true;
                    }
                    if (!(qk_issued && pv_issued)) __nanosleep(32);
                    if ((spin & 63) == 63 && global_timer_ns() - t0 > 2000000000ull) ok = false;
                }
                if (!ok) break;
                prev_np = m.n_pages;
                prev_first = (m.flags & TILE_FIRST) != 0;
                if (m.flags & TILE_END) {
                    ok = wait_bounded(p_ready + 8 * s, (uint32_t)((k >> 1) & 1));
                    if (ok) ok = issue_pv(k, prev_np, prev_first);
                    break;
                }
            }
            if (!ok) { atomicOr(p.status, STATUS_TIMEOUT); *gave_up = 1; }
        }
        __syncwarp();
    } else if (n > 0) {
        // ================= softmax (warps 0-3) =================
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const int j = tid >> 4, tt = tid & 15;           // page slot and token-in-page of this thread's token
        float m_ref[GP], l_sum[GP], qs[GP];
#pragma unroll
        for (int h = 0; h < GP; ++h) { m_ref[h] = -INFINITY; l_sum[h] = 0.f; qs[h] = 0.f; }
        bool ok = true;
        for (int k = 0; ok; ++k) {
            const int s = k & 1;
            // (after a timeout the thread goes on with whatever it finds, up to the barrier below, where all leave)
            ok = wait_bounded(v_full + 8 * s, (uint32_t)((k >> 1) & 1));          // the scales
            ok = ok && wait_bounded(s_ready + 8 * s, (uint32_t)((k >> 1) & 1));  // the scores
            tc_fence_after();
            const TileMeta m = load_meta(&meta[k & 3]);
            const bool first = (m.flags & TILE_FIRST) != 0;
            if (first) {
                // (the query scales were written before Q' was announced, which the issuing thread saw before it
                // issued these scores; no wait on that barrier here -- it may be two phases on by now, which a
                // parity wait cannot tell from none)
#pragma unroll
                for (int h = 0; h < GP; ++h) {
                    m_ref[h] = -INFINITY;
                    l_sum[h] = 0.f;
                    qs[h] = reinterpret_cast<volatile float *>(qscale)[m.qbuf * 8 + h];
                }
            }
            uint32_t sv[16];
            tmem_ld16(lane_base + (uint32_t)(16 * s), sv);
            tmem_wait_ld();
            const bool valid = j < m.n_pages && (j != m.short_slot || tt < m.short_valid);
            const uint8_t *vpage = v_ring_ptr + s * V_STAGE + j * V_PAGE;
            float ksc = 0.f, vsc = 0.f;
            if (valid) {
                ksc = *reinterpret_cast<const float *>(vpage + K_PAGE + 4 * tt);
                vsc = *reinterpret_cast<const float *>(vpage + K_PAGE + 4 * PAGE + 4 * tt);
            }
            // The reference of head h follows  e = score + log2(vscale), the size of the token's term in the
            // output, not the score alone: P' = 32 * 2^(e - ref) then stays in E4M3's range whatever the spread
            // of the V scales (a huge V row with a negligible probability does not push the others out of it).
            float lv;
            asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lv) : "f"(vsc));
            lv = fmaxf(lv, -60.f);         // an all-zero V row (scale 0) counts as a very small one
            float sc[GP];                  // (heads G..GP-1 have zero queries: their scores are 0, their results unused)
#pragma unroll
            for (int h = 0; h < GP; ++h)
                sc[h] = valid ? (__uint_as_float(sv[h]) + __uint_as_float(sv[8 + h])) * (ksc * qs[h]) : -INFINITY;
            // maxima of e over the tile's 128 tokens, per head
#pragma unroll
            for (int h = 0; h < GP; ++h) {
                const int mk = warp_max_s32(float_key(sc[h] + lv));
                if (lane == 0) red[s * 64 + h * 4 + warp] = mk;
            }
            ok = softmax_all(ok);          // the maxima are in place; and has every thread's wait ended normally?
            if (!ok) break;
            bool changed = false;
            float m_new[GP];
#pragma unroll
            for (int h = 0; h < GP; ++h) {
                const int4 r = *reinterpret_cast<const int4 *>(red + s * 64 + h * 4);      // the four warps' maxima
                const float mx = key_float(max(max(r.x, r.y), max(r.z, r.w)));           // finite: every tile has a valid token
                m_new[h] = mx > m_ref[h] + RESCALE_STEP ? mx : m_ref[h];
                changed = changed || (m_new[h] != m_ref[h]);
            }
            if (changed) {
                // the sums (and, unless the run starts here, O^T of the run so far) move to the new references
                float alpha[GP];
#pragma unroll
                for (int h = 0; h < GP; ++h) {
                    alpha[h] = fast_exp2(m_ref[h] - m_new[h]);
                    l_sum[h] *= alpha[h];
                    m_ref[h] = m_new[h];
                }
                if (!first) {
                    // the values of the tile before this one must be done (that barrier's phase before that one is over
                    // because this tile's scores were issued after it, and its next phase needs the probabilities
                    // written below)
                    ok = wait_bounded(pv_done + 8 * ((k - 1) & 1), (uint32_t)(((k - 1) >> 1) & 1));
                    ok = softmax_all(ok);
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t ov[16];
                    tmem_ld16(lane_base + COL_O, ov);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        if ((c & 7) < GP) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha[(c & 7) % GP]);
                    tmem_st16(lane_base + COL_O, ov);
                    tmem_wait_st();
                }
            }
            // probabilities, split into two E4M3 terms: the token's 16 bytes [leading terms of heads 0..7 |
            // remainders of heads 0..7] (heads >= GP zero) are one row of the N-major P' operand
            {
                float lead[8], rem[8];
#pragma unroll
                for (int h = 0; h < 8; ++h) { lead[h] = 0.f; rem[h] = 0.f; }
#pragma unroll
                for (int h = 0; h < GP; ++h) {
                    const float pr = fast_exp2(sc[h] - m_ref[h]);       // 0 for a token that is not in use; its share of the sum
                    const float pp = pr * (vsc * P_SCALE);               // = 32 * 2^(e - ref) <= 362
                    lead[h] = __uint_as_float((__float_as_uint(pp) + 0x00080000u) & 0xFFF00000u);   // rounded to E4M3's three mantissa bits
                    rem[h] = (pp - lead[h]) * REM_SCALE;                              // |.| <= 16 * 16 at the top binade
                    l_sum[h] += pr;
                }
                const uint32_t w0 = pack_e4m3x2(lead[0], lead[1]) | (pack_e4m3x2(lead[2], lead[3]) << 16);
                const uint32_t w1 = GP > 4 ? pack_e4m3x2(lead[4], lead[5]) | (pack_e4m3x2(lead[6], lead[7]) << 16) : 0u;
                const uint32_t w2 = pack_e4m3x2(rem[0], rem[1]) | (pack_e4m3x2(rem[2], rem[3]) << 16);
                const uint32_t w3 = GP > 4 ? pack_e4m3x2(rem[4], rem[5]) | (pack_e4m3x2(rem[6], rem[7]) << 16) : 0u;
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(p_sm + (uint32_t)(s * P_BYTES + tid * 16)), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
            }
            // V codes the tensor core will read but that belong to no token in use must be finite too: the
            // unused slots of the sequence's last page may hold anything, and an odd tile reads one page
            // slot beyond its last.  Thread d owns the 16 tokens of dim d.
            if (m.short_slot >= 0) {
                const uint32_t a = v_ring + (uint32_t)(s * V_STAGE + m.short_slot * V_PAGE + tid * 16);
                uint32_t w0, w1, w2, w3;
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(a));
                const int keep = m.short_valid;          // leading bytes to keep, 1..15
                auto mask_word = [&](uint32_t wv, int first_byte) -> uint32_t {
                    const int kb = keep - first_byte;
                    return kb >= 4 ? wv : kb <= 0 ? 0u : (wv & (0xFFFFFFFFu >> (8 * (4 - kb))));
                };
                w0 = mask_word(w0, 0); w1 = mask_word(w1, 4); w2 = mask_word(w2, 8); w3 = mask_word(w3, 12);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
            }
            if (m.n_pages & 1)
                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(v_ring + (uint32_t)(s * V_STAGE + m.n_pages * V_PAGE + tid * 16)), "r"(0u) : "memory");
            fence_proxy_async();           // the tensor core reads P' (and the V bytes just cleared) through the async proxy
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_ready + 8 * s);

            if (m.flags & TILE_LAST) {
                // the run's partial: O^T (thread d = dim d), the references and the sums
                ok = wait_bounded(pv_done + 8 * s, (uint32_t)((k >> 1) & 1));
                ok = softmax_all(ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t ov[16];
                tmem_ld16(lane_base + COL_O, ov);
                tmem_wait_ld();
#pragma unroll
                for (int h = 0; h < GP; ++h) {
                    float v = l_sum[h];
#pragma unroll
                    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(FULL, v, d);
                    if (lane == 0) red_l[warp * 8 + h] = v;
                }
                softmax_sync();
                const int64_t seg = (int64_t)m.b * p.Hkv + m.h;
                const int64_t slot = partial_slot(T, W, w, x0, seg);
                const float back = 1.f / P_SCALE;
#pragma unroll
                for (int h = 0; h < GP; ++h)
                    if (h < G)
                        p.part_o[(slot * G + h) * D + tid] = (__uint_as_float(ov[h]) + __uint_as_float(ov[8 + h]) * (1.f / REM_SCALE)) * back;
                if (tid < G) {
                    const volatile float *r = red_l + tid;
                    float mine = m_ref[0];
#pragma unroll
                    for (int h = 1; h < GP; ++h) mine = tid == h ? m_ref[h] : mine;
                    *reinterpret_cast<float2 *>(p.part_ml + (slot * G + tid) * 2) = make_float2(mine, (r[0] + r[8]) + (r[16] + r[24]));
                }
                tc_fence_before();
            }
            if (m.flags & TILE_END) break;
        }
        if (!ok && tid == 0) { atomicOr(p.status, STATUS_TIMEOUT); *gave_up = 1; }
    }

    // ---- common exit ----
    pdl_trigger();
    tc_fence_before();
    __syncthreads();
    if (warp == 5 && lane == 0 && *reinterpret_cast<volatile int *>(gave_up)) {
        // after a timeout copies may still be in flight: give them their (bounded) wait before the shared memory goes away
        for (int k = (tiles_issued > 2 ? tiles_issued - 2 : 0); k < tiles_issued; ++k) {
            mbar_wait_bounded(k_full + 8 * (k & 1), (uint32_t)((k >> 1) & 1));
            mbar_wait_bounded(v_full + 8 * (k & 1), (uint32_t)((k >> 1) & 1));
        }
    }
    if (p.trace && tid == 0) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        unsigned long long *t = p.trace + 4 * w;
        t[0] = smid; t[1] = t_entry; t[2] = t_entry; t[3] = global_timer_ns();
    }
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

}  // namespace

bool decode_fp8_umma_supported(int D, int G) { return D == 128 && G >= 1 && G <= 8; }

int decode_fp8_umma_ctas_per_sm() { return CTAS_PER_SM; }
int decode_fp8_umma_tile_tokens() { return TP * PAGE; }

size_t decode_fp8_umma_smem_bytes(int D, int B)
{
    const int block = fp8_block_bytes(D);
    // alignment | tables | K and V rings | two P' | Q' | tile descriptions | query scales | maxima | sums | barriers | two words
    return 128 + table_bytes(B) + (size_t)NST * TP * block + 2 * 16 * (size_t)(TP * PAGE) + 16 * (size_t)D + 4 * sizeof(TileMeta) +
           64 + 512 + 128 + 16 * 8 + 16;
}

cudaError_t launch_decode_fp8_umma(const DecodeParams &p, int D, int G, int grid, bool pdl, cudaStream_t s)
{
    if (!decode_fp8_umma_supported(D, G)) return cudaErrorInvalidValue;
    const size_t smem = decode_fp8_umma_smem_bytes(D, p.B);
    auto kern = G <= 1 ? decode_fp8_umma_kernel<128, 1> : G <= 2 ? decode_fp8_umma_kernel<128, 2>
              : G <= 4 ? decode_fp8_umma_kernel<128, 4> : decode_fp8_umma_kernel<128, 8>;
    cudaError_t e = ensure_dynamic_smem(kern, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p, G);
}

}  // namespace skv
