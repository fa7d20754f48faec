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
#include "skv_decode_states.cuh"
#include "skv_walk.cuh"

#include <math.h>

namespace skv {

namespace {

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
    const bool early_fetch = (p.flags & DECODE_EARLY_FETCH) != 0 && !late_wait;
    const bool reverse = (p.flags & DECODE_REVERSE) != 0;
    if (!late_wait && !early_fetch) pdl_wait();   // anything read below may come from the kernel before this one

    // sequence lengths and cumulative page counts of the batch (warp 0), visible to all after the barrier
    if (warp == 0) scan_lengths(p.seq_lens, p.B, PAGE, (int64_t)p.pt_stride * PAGE, p.status, prefix, lens, lane);
    __syncthreads();
    // the merge kernel reads the page counts from global memory (written after the wait on the previous
    // kernel: the merge of an earlier call may still be reading this buffer)
    auto publish_prefix = [&]() {
        if (blockIdx.x == 0)
            for (int i = threadIdx.x; i <= p.B; i += blockDim.x) p.prefix[i] = prefix[i];
    };
    if (!early_fetch) publish_prefix();

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
    const int keep_from = (p.keep_pct > 0 && T <= p.l2_fit_blocks) ? 0 : n - (int)(((int64_t)n * p.keep_pct) / 100);
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
    if (early_fetch) {
        // The lengths, the page table and every cached token except each sequence's newest one are older
        // than the kernel before this one (the caller's promise behind DECODE_EARLY_FETCH): the ring is
        // filled with such blocks while that kernel is still running.  A sequence's last page may be
        // receiving its newest token right now, so the fill stops in front of it; the queries are read
        // only after the wait (State::begin below).
        while (in_flight < stages && prod_left > 0 && prod.pg + 1 != prod.pages && issue()) {}
        pdl_wait();
        publish_prefix();
    }
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
            if (!failed) st.finish(p.part_o, p.part_ml, partial_slot(T, W, w, x0, seg), G, lane);
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

// this warp's share of the segments: seg0, seg0 + stride, ...  (prefix: [B+1] cumulative unit counts)
template <int D, int E2MAX, int NB>
__device__ __forceinline__ void merge_loop(const MergeParams &p, const int32_t *prefix, int64_t seg0, int64_t stride, int lane)
{
    const int64_t n_seg = (int64_t)p.B * p.Hkv;
    const int G = p.Hq / p.Hkv;
    const int64_t T = (int64_t)prefix[p.B] * p.Hkv;
    for (int64_t seg = seg0; seg < n_seg; seg += stride) {
        const int b = (int)(seg / p.Hkv), kvh = (int)(seg - (int64_t)b * p.Hkv);
        const int pages = prefix[b + 1] - prefix[b];
        uint16_t *out_seg = p.out + ((int64_t)b * p.Hq + (int64_t)kvh * G) * D;
        if (pages == 0) {
            uint32_t *dst = reinterpret_cast<uint32_t *>(out_seg);
            for (int i = lane; i < G * D / 2; i += 32) dst[i] = 0u;
            continue;
        }
        const int64_t s0 = (int64_t)prefix[b] * p.Hkv + (int64_t)kvh * pages;
        int slot0, n_part;
        segment_partials(T, p.n_workers, seg, s0, pages, slot0, n_part);
        if (n_part == 1 && p.skip_single) continue;     // finished by the split-K launch
        merge_rows<D, E2MAX, NB>(p.part_o, p.part_ml, out_seg, G, slot0, n_part, lane);
    }
}

// One warp per (sequence, kv head) segment, a grid of at most one CTA per SM walking the segments:
// every CTA must be resident (waiting for the split-K launch to end) before the launch after this
// one may be scheduled, so the grid has to fit beside the split-K CTAs in one wave.
// Given the sequence lengths, the kernel counts the pages itself while the split-K launch is still
// running, so that only the partials remain to be fetched once that launch has ended.
template <int D>
__global__ void __launch_bounds__(MERGE_WARPS * 32) merge_kernel(MergeParams p)
{
    extern __shared__ int32_t merge_smem[];          // prefix [B+1], lens [B] when the lengths are given
    pdl_trigger();        // nothing after this kernel in the stream needs to wait for its start
    const int lane = threadIdx.x & 31;
    const int32_t *prefix = p.prefix;
    if (p.seq_lens) {
        if (threadIdx.x < 32)        // (over-long sequences were flagged by the split-K launch: no status word here)
            scan_lengths(p.seq_lens, p.B, p.unit_tokens, p.max_tokens, nullptr, merge_smem, merge_smem + p.B + 1, lane);
        __syncthreads();
        prefix = merge_smem;
    }
    pdl_wait();           // the partials come from the kernel before this one
    const int64_t seg0 = (int64_t)blockIdx.x * MERGE_WARPS + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * MERGE_WARPS;
    const int G = p.Hq / p.Hkv;
    const int E2 = (G <= 1 ? 1 : G <= 2 ? 2 : G <= 4 ? 4 : 8) * D / 64;   // float2 per lane, see merge_rows
    constexpr int P = SKV_MERGE_PAYLOAD;
    if (E2 <= 2) merge_loop<D, 2, (P / 2 > 16 ? 16 : P / 2)>(p, prefix, seg0, stride, lane);
    else if (E2 <= 4) merge_loop<D, 4, (P / 4 > 16 ? 16 : P / 4)>(p, prefix, seg0, stride, lane);
    else if (E2 <= 8) merge_loop<D, 8, P / 8>(p, prefix, seg0, stride, lane);
    else merge_loop<D, 16, P / 16>(p, prefix, seg0, stride, lane);
}

template <int D, class State>
cudaError_t launch_splitk_t(const DecodeParams &p, int G, int grid, int warps, int stages, bool pdl, cudaStream_t s)
{
    const size_t smem = 128 + table_bytes(p.B) + (size_t)warps * stages * State::BLOCK + (size_t)warps * stages * 8 + 16;
    auto kern = decode_splitk_kernel<D, State>;
    cudaError_t e = ensure_dynamic_smem(kern, smem);
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
    cfg.dynamicSmemBytes = p.seq_lens ? (size_t)(2 * p.B + 1) * sizeof(int32_t) : 0;
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
