// Pre-fill attention on the 5th-generation tensor cores (tcgen05): the same computation as
// skv_prefill.cu with both contractions issued as UMMA instructions and their accumulators in
// tensor memory.
//
// One CTA (2 per SM) owns 128 query rows: 128/G tokens x the G query heads of one kv head, row
// r = token r/G, head r%G.  Eight warps:
//   warps 0-3  softmax: thread r owns row r (= TMEM lane r)
//   warp 4     lane 0 issues the UMMA instructions
//   warps 5, 6 copy K of the even / odd key blocks into the K ring (a warp waits for its own copies to land
//              before it hands the stage over, so one warp doing every block made the landing time of a
//              block's K the period of the whole pipeline: 2730 cycles per block with the softmax switched off)
//   warp 7     copies V into the V ring
// Shared memory
//   Q tile   K-major core-matrix layout [D/8 chunks][128 rows][16 B]
//   K ring   2 stages of 64 keys, [D/8 chunks][64 keys][16 B]: a page's K half is
//            [chunk][16 keys][16 B]; a copy warp moves it with 16-byte cp.async copies that interleave
//            the four pages of a stage by chunk, which makes the 64 keys ONE N=64 operand
//   V ring   2 stages of 4 pages, each page's V half copied as it is (4 KB): read as the B operand
//            of P V it is the MN-major core-matrix layout
// Tensor memory (256 columns)
//   [0,64), [64,128)   two score buffers: S = Q K^T of a key block (fp32), overwritten in place by
//                      its P (bf16 pairs, 32 columns), the A operand of P V
//   [128,128+D)        O += P V
// Per key block kb: Q K^T(kb+1) is issued before the softmax of block kb has finished, so the
// tensor core works on the next scores (and on P V of the block before) while the softmax warps
// are busy.  Softmax state (running max, sum) lives in the row's thread.  O is rescaled lazily:
// the max used for the exponentials only moves when the true max has grown by more than 8 (in
// log2 units), so most key blocks cost no pass over O; the final division uses the same max, so
// the result is the exact softmax.
// Barriers are all per stage / per score buffer (two of each): a parity wait only means "phase k is
// over" if the waiter knows phase k-1 of that barrier is over and phase k+1 cannot have happened,
// and with a period of two key blocks per barrier every waiter here can show both (a single
// barrier counting every block let a fast softmax warp pass the final wait one phase early).
// Every wait is bounded; on a timeout the warp flags the status word and goes to the common exit,
// where copies are given time to land and the tensor memory is freed.
#include "skv_common.cuh"
#include "skv_tcgen05.cuh"

#include <math.h>

namespace skv {

namespace {

using namespace tc5;

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int ROWS = 128;
constexpr int KB = 4;                 // pages per key block
constexpr int KEYS = KB * PAGE;       // 64
constexpr int NSTAGE = 2;
constexpr int COL_O = 128;            // score buffers at columns 0 and 64
constexpr int TMEM_COLS = 256;
constexpr float RESCALE_STEP = 8.f;
// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major)
{
    return (1u << 4) /* D fp32 */ | (1u << 7) /* A bf16 */ | (1u << 10) /* B bf16 */ |
           ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

constexpr int THREADS = 256;

template <int D>
__global__ void __launch_bounds__(THREADS, 2) prefill_umma_kernel(PrefillParams p, int G)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = block_bytes(D), HALF = half_bytes(D), CH = D / 8;
    constexpr int Q_BYTES = ROWS * D * 2;
    constexpr int K_STAGE = KEYS * D * 2, V_STAGE = KB * HALF;
    constexpr uint32_t IDESC_QK = instr_desc(ROWS, KEYS, false), IDESC_PV = instr_desc(ROWS, D, true);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.z, h = blockIdx.y;
    const int TQ = ROWS / G;

    const uint32_t base = smem_u32(smem_raw);
    const uint32_t pad = (128u - (base & 127u)) & 127u;
    const uint32_t q_smem = base + pad;
    const uint32_t k_ring = q_smem + Q_BYTES;
    const uint32_t v_ring = k_ring + NSTAGE * K_STAGE;
    const uint32_t bars = v_ring + NSTAGE * V_STAGE;
    const uint32_t full_k = bars, full_v = bars + 16, s_ready = bars + 32, p_ready = bars + 48, pv_done = bars + 64;
    const uint32_t slot = bars + 80;
    volatile uint32_t *slot_ptr =
        reinterpret_cast<volatile uint32_t *>(smem_raw + pad + Q_BYTES + NSTAGE * K_STAGE + NSTAGE * V_STAGE + 80);
    volatile uint32_t *gave_up = slot_ptr + 1;     // set by a warp whose wait ran out

    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(full_k + 8 * s, 1);
            mbar_init(full_v + 8 * s, 1);
            mbar_init(s_ready + 8 * s, 1);
            mbar_init(p_ready + 8 * s, ROWS);
            mbar_init(pv_done + 8 * s, 1);
        }
        *gave_up = 0;
        fence_barrier_init();
    }
    pdl_wait();
    const int q_begin = __ldg(p.cu_q + b), q_len = __ldg(p.cu_q + b + 1) - q_begin;
    const int n_b = __ldg(p.seq_lens + b);
    const bool too_long = (int64_t)n_b > (int64_t)p.pt_stride * PAGE;     // more pages than a page-table row holds
    const int n_tiles = (q_len + TQ - 1) / TQ;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;
    if (blockIdx.x == 0 && tid == 0 && (q_len < 0 || q_len > n_b || too_long || n_tiles > (int)gridDim.x))
        atomicOr(p.status, STATUS_BOUNDS);
    if (q_len <= 0 || q_len > n_b || too_long || qt >= n_tiles) return;    // uniform over the CTA, before any allocation
    const int q0 = qt * TQ;
    const int q_end = (q0 + TQ < q_len) ? q0 + TQ : q_len;
    const int pos0 = n_b - q_len;
    const int n_keys = pos0 + q_end;
    const int n_pages = (n_keys + PAGE - 1) / PAGE;
    const int n_kb = (n_pages + KB - 1) / KB;

    if (warp == 4) {
        tmem_alloc(slot, TMEM_COLS);
        tmem_relinquish();
    }

    // ---- copies (warps 5-7, all lanes).  Lane j < KB carries the id of page j of a block. ----
    auto load_ids = [&](int kb) -> int {
        const int pg = kb * KB + lane;
        int id = 0;
        if (lane < KB && pg < n_pages) {
            id = __ldg(p.page_table + (int64_t)b * p.pt_stride + pg);
            if (id < 0 || (int64_t)id >= p.max_pages) {
                atomicOr(p.status, STATUS_BOUNDS);
                id = 0;
            }
        }
        return id;
    };
    // K of key block kb: 16-byte asynchronous copies, the four pages interleaved by chunk (one cp.async group)
    auto copy_k = [&](int kb, int ids) {
        const int s = kb % NSTAGE, pg0 = kb * KB;
        const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
        for (int j = 0; j < np; ++j) {
            const int id = __shfl_sync(FULL, ids, j);
            const uint8_t *src = p.layer_base + (int64_t)id * p.page_stride + (int64_t)h * BLOCK;
            const uint32_t dst = k_ring + (uint32_t)(s * K_STAGE + j * PAGE * 16);
#pragma unroll
            for (int i = lane; i < CH * PAGE; i += 32) {          // piece i = (chunk i / 16, key i % 16)
                const uint32_t d = dst + (uint32_t)((i / PAGE) * KEYS * 16 + (i % PAGE) * 16);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src + i * 16) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // V of key block kb: one 4 KB bulk copy per page
    auto copy_v = [&](int kb, int ids) {
        const int s = kb % NSTAGE, pg0 = kb * KB;
        const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
        const uint32_t bar = full_v + 8 * s;
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(np * HALF));
        __syncwarp();
        if (lane < np)
            bulk_copy_g2s(v_ring + (uint32_t)(s * V_STAGE + lane * HALF),
                          p.layer_base + (int64_t)ids * p.page_stride + (int64_t)h * BLOCK + HALF, HALF, bar);
    };
    // this warp's copies of K(kb) have landed: make them visible to the tensor core's proxy, tell the MMA warp
    auto publish_k = [&](int kb) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(full_k + 8 * (kb % NSTAGE)) : "memory");
    };
    int v_copies = 0;                              // V blocks issued (warp 7)

    // ---- this thread's row (softmax warps): Q into shared memory in core-matrix layout ----
    const int qi = tid / G, g = tid - qi * G;
    const bool row_ok = warp < 4 && q0 + qi < q_end;
    const int pos = row_ok ? pos0 + q0 + qi : 0x7FFFFFFF;
    const int64_t row_off = ((int64_t)(q_begin + q0 + qi) * p.Hq + (int64_t)h * G + g) * D;
    if (warp < 4) {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.Q + row_off);
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const uint4 v = row_ok ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(q_smem + (uint32_t)(c * ROWS * 16 + tid * 16)),
                         "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
        fence_proxy_async();           // the tensor core reads Q through the async proxy
    }
    tc_fence_before();
    __syncthreads();                   // Q tile complete, TMEM address published
    tc_fence_after();
    const uint32_t tmem = *slot_ptr;

    if (warp == 5 || warp == 6) {
        // =================== K copy warps: warp 5 the even key blocks (stage 0), warp 6 the odd ones ===================
        const int par = warp - 5;
        bool ok = true;
        if (par < n_kb) {
            int ids = load_ids(par);
            copy_k(par, ids);
            ids = load_ids(par + 2);                           // fetched ahead of its use
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            publish_k(par);
            for (int kb = par; kb + 2 < n_kb; kb += 2) {
                // Q K^T(kb) complete (its scores are ready): the stage takes K(kb+2).  The barrier's next completion
                // needs the very copy issued after this wait, so the warp can never fall a whole phase behind.
                if (lane == 0) ok = mbar_wait_bounded(s_ready + 8 * par, (uint32_t)((kb / NSTAGE) & 1));
                ok = __shfl_sync(FULL, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                copy_k(kb + 2, ids);
                ids = load_ids(kb + 4);
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                publish_k(kb + 2);
            }
        }
        if (!ok && lane == 0) {
            atomicOr(p.status, STATUS_TIMEOUT);
            *gave_up = 1;
        }
    } else if (warp == 7) {
        // =================== V copy warp ===================
        bool ok = true;
        int ids = load_ids(0);
        copy_v(0, ids);
        v_copies = 1;
        if (n_kb > 1) {
            ids = load_ids(1);
            copy_v(1, ids);
            v_copies = 2;
        }
        ids = load_ids(2);
        for (int kb = 0; kb + 2 < n_kb; ++kb) {
            // P V of block kb complete: its V stage takes V(kb+2)
            if (lane == 0) ok = mbar_wait_bounded(pv_done + 8 * (kb % NSTAGE), (uint32_t)((kb / NSTAGE) & 1));
            ok = __shfl_sync(FULL, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            copy_v(kb + 2, ids);
            v_copies = kb + 3;
            ids = load_ids(kb + 3);
        }
        if (!ok && lane == 0) {
            atomicOr(p.status, STATUS_TIMEOUT);
            *gave_up = 1;
        }
    } else if (warp == 4) {
        // =================== MMA warp: lane 0 issues ===================
        if (lane == 0) {
            // S(kb) = Q K^T: D/16 instructions M128 N64 K16 into score buffer kb % 2
            auto issue_qk = [&](int kb) {
                const int s = kb % NSTAGE;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint64_t a = smem_desc(q_smem + (uint32_t)(ks * 2 * ROWS * 16), ROWS * 16, 128);
                    const uint64_t bd = smem_desc(k_ring + (uint32_t)(s * K_STAGE + ks * 2 * KEYS * 16), KEYS * 16, 128);
                    umma_ss(tmem + (uint32_t)(s * KEYS), a, bd, IDESC_QK, ks > 0);
                }
                tc_commit(s_ready + 8 * s);
            };
            // O += P V: one instruction M128 N=D K16 per present page
            auto issue_pv = [&](int kb) {
                const int s = kb % NSTAGE, pg0 = kb * KB;
                const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
                for (int j = 0; j < np; ++j) {
                    const uint64_t bd = smem_desc(v_ring + (uint32_t)(s * V_STAGE + j * HALF), 128, PAGE * 16);
                    umma_ts(tmem + COL_O, tmem + (uint32_t)(s * KEYS + 8 * j), bd, IDESC_PV, (kb > 0 || j > 0) ? 1u : 0u);
                }
                tc_commit(pv_done + 8 * s);
            };
            bool ok = mbar_wait_bounded(full_k, 0);
            if (ok) { tc_fence_after(); issue_qk(0); }
            for (int kb = 0; ok && kb < n_kb; ++kb) {
                if (kb + 1 < n_kb) {
                    // K(kb+1) in shared memory; score buffer of block kb+1 free (P V of block kb-1 complete)
                    ok = mbar_wait_bounded(full_k + 8 * ((kb + 1) % NSTAGE), (uint32_t)(((kb + 1) / NSTAGE) & 1));
                    if (ok && kb >= 1) ok = mbar_wait_bounded(pv_done + 8 * ((kb - 1) % NSTAGE), (uint32_t)(((kb - 1) / NSTAGE) & 1));
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(kb + 1);
                }
                ok = mbar_wait_bounded(p_ready + 8 * (kb % NSTAGE), (uint32_t)((kb / NSTAGE) & 1)) &&
                     mbar_wait_bounded(full_v + 8 * (kb % NSTAGE), (uint32_t)((kb / NSTAGE) & 1));
                if (!ok) break;
                tc_fence_after();
                issue_pv(kb);
            }
            if (!ok) {
                atomicOr(p.status, STATUS_TIMEOUT);
                *gave_up = 1;
            }
        }
        __syncwarp();
    } else {
        // =================== softmax warps ===================
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        float m_used = -INFINITY, l_sum = 0.f;
        bool ok = true;
        for (int kb = 0; kb < n_kb; ++kb) {
            const int s = kb % NSTAGE, pg0 = kb * KB;
            const int np = (n_pages - pg0) < KB ? (n_pages - pg0) : KB;
            ok = mbar_wait_bounded(s_ready + 8 * s, (uint32_t)((kb / NSTAGE) & 1));
            if (!__all_sync(FULL, ok)) { ok = false; break; }
            tc_fence_after();
            uint32_t raw[2][32];
            tmem_ld32(lane_base + (uint32_t)(s * KEYS), raw[0]);
            tmem_ld32(lane_base + (uint32_t)(s * KEYS + 32), raw[1]);
            tmem_wait_ld();
            const int t_base = pg0 * PAGE, n_there = np * PAGE;
            // causal mask (and absent pages of the last block) on the raw scores; most blocks are fully visible
            float mx = -INFINITY;
            if (n_there == KEYS && t_base + KEYS - 1 <= pos) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(raw[hh][c]));
            } else {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const int col = hh * 32 + c;
                        if (!(col < n_there && t_base + col <= pos)) raw[hh][c] = 0xFF800000u;   // -inf
                        mx = fmaxf(mx, __uint_as_float(raw[hh][c]));
                    }
            }
            mx *= p.scale_log2;                                // the scale is positive
            // lazy rescaling: move the reference max only when the true max has run away from it
            float alpha = 1.f;
            const bool move = mx > m_used + RESCALE_STEP;      // also true for the first block with a visible key
            if (move) {
                alpha = fast_exp2(m_used - mx);                // 0 when m_used = -inf
                m_used = mx;
            }
            if (kb > 0 && __any_sync(FULL, move)) {
                // O must hold every block up to kb-1 before it is scaled
                ok = mbar_wait_bounded(pv_done + 8 * ((kb - 1) % NSTAGE), (uint32_t)(((kb - 1) / NSTAGE) & 1));
                if (!__all_sync(FULL, ok)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int q4 = 0; q4 < D / 16; ++q4) {
                    uint32_t ov[16];
                    tmem_ld16(lane_base + COL_O + 16 * q4, ov);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
                    tmem_st16(lane_base + COL_O + 16 * q4, ov);
                }
            }
            l_sum *= alpha;
            uint32_t pk[32];
            float sum = 0.f;
            const float neg_m = -m_used;
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                const int hh = c >> 4, cc = (2 * c) & 31;
                const float x0 = fmaf(__uint_as_float(raw[hh][cc]), p.scale_log2, neg_m);
                const float x1 = fmaf(__uint_as_float(raw[hh][cc + 1]), p.scale_log2, neg_m);
                const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                sum += p0 + p1;
                pk[c] = pack_bf16x2(p0, p1);
            }
            l_sum += sum;
            tmem_st32(lane_base + (uint32_t)(s * KEYS), pk);    // P over the first half of its own scores
            // slots of the sequence's last page that were never written may hold anything: zero their V rows
            const int last_valid = n_b - (pg0 + np - 1) * PAGE;
            if (last_valid < PAGE) {
                ok = mbar_wait_bounded(full_v + 8 * s, (uint32_t)((kb / NSTAGE) & 1));
                if (!__all_sync(FULL, ok)) { ok = false; break; }
                const uint32_t sV = v_ring + (uint32_t)(s * V_STAGE + (np - 1) * HALF);
                for (int i = tid; i < CH * PAGE; i += ROWS)
                    if ((i & (PAGE - 1)) >= last_valid)
                        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(sV + (uint32_t)(i * 16)), "r"(0u) : "memory");
                fence_proxy_async();
            }
            tmem_wait_st();
            tc_fence_before();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(p_ready + 8 * s) : "memory");
        }
        if (ok) {
            // the last P V (the phase before it on this barrier, block n_kb-3, is known to be over)
            ok = mbar_wait_bounded(pv_done + 8 * ((n_kb - 1) % NSTAGE), (uint32_t)(((n_kb - 1) / NSTAGE) & 1));
            ok = __all_sync(FULL, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l_sum;
            uint16_t *dst = p.out + row_off;
#pragma unroll
            for (int q4 = 0; q4 < D / 32; ++q4) {
                uint32_t ov[32];
                tmem_ld32(lane_base + COL_O + 32 * q4, ov);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(ov[c]) * inv, __uint_as_float(ov[c + 1]) * inv);
                        w.y = pack_bf16x2(__uint_as_float(ov[c + 2]) * inv, __uint_as_float(ov[c + 3]) * inv);
                        w.z = pack_bf16x2(__uint_as_float(ov[c + 4]) * inv, __uint_as_float(ov[c + 5]) * inv);
                        w.w = pack_bf16x2(__uint_as_float(ov[c + 6]) * inv, __uint_as_float(ov[c + 7]) * inv);
                        *reinterpret_cast<uint4 *>(dst + 32 * q4 + c) = w;
                    }
                }
            }
        } else if (lane == 0) {
            atomicOr(p.status, STATUS_TIMEOUT);
            *gave_up = 1;
        }
    }
    // ---- common exit ----
    pdl_trigger();
    tc_fence_before();
    __syncthreads();
    if (warp == 5 || warp == 6) asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (warp == 7) {
        // after a timeout the last copies issued may still be in flight: give them their (bounded) wait
        // before the shared memory goes away
        if (lane == 0 && *gave_up)
            for (int kb = (v_copies > NSTAGE ? v_copies - NSTAGE : 0); kb < v_copies; ++kb)
                mbar_wait_bounded(full_v + 8 * (kb % NSTAGE), (uint32_t)((kb / NSTAGE) & 1));
    }
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

}  // namespace

size_t prefill_umma_smem_bytes(int D)
{
    if (D != 128) return 0;
    return 128 + (size_t)ROWS * D * 2 + (size_t)NSTAGE * KB * block_bytes(D) + 96 + 16;
}

bool prefill_umma_supported(int D, int G) { return D == 128 && G >= 1 && G <= 8 && ROWS % G == 0; }

int prefill_umma_tile_tokens(int G) { return ROWS / G; }

cudaError_t launch_prefill_umma(const PrefillParams &p, int D, int G, int q_tiles, bool pdl, cudaStream_t s)
{
    const size_t smem = prefill_umma_smem_bytes(D);
    if (smem == 0 || q_tiles <= 0 || !prefill_umma_supported(D, G)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)q_tiles, (unsigned)p.Hkv, (unsigned)p.B);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaError_t e = ensure_dynamic_smem(prefill_umma_kernel<128>, smem);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&cfg, prefill_umma_kernel<128>, p, G);
}

}  // namespace skv
