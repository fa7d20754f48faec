// "Load + Attn" of Algorithm 2 for one new token per sequence (Eq. (3.1)), the form used for stand-alone
// attention calls: the worker of the split-K pass is a whole CTA (one per SM) instead of a warp.
//
// The flattened (sequence, kv head, page) block list of the call is cut into one contiguous range per CTA.
// One producer warp streams the CTA's blocks, in order, through ONE shared ring of 8 KB stages (a linear
// bulk copy per block, completion on the stage's mbarrier); the consumer warps take the blocks of the ring
// in turn (consumer c takes blocks c, c + C, ...: the same sum order every time, so results repeat bit for
// bit) or, as an option, claim them from a shared counter (whoever is free takes the next block), each
// keeping a running (max, sum, out) of its own for the (sequence, kv head) segment the blocks belong to.
// At the end of every run of the range inside one segment the consumers put their states side by side in
// shared memory and combine them:
//   - a segment that lies wholly inside the CTA's range is finished on the spot: normalised, rounded to
//     bf16 and written to `out`;
//   - a segment that continues in a neighbouring CTA leaves one fp32 partial at slot  cta + segment  for the
//     merge kernel, which only has those segments left to do.
// Compared with a warp per range this evens out the consumers of an SM block by block (a warp with two
// copies of its own in flight advances at the pace of its own latencies, and the slowest of 1184 sets the
// end of the launch), leaves a fifth of the partials, and keeps more bytes in flight per SM.
#include "skv_common.cuh"
#include "skv_decode_states.cuh"
#include "skv_walk.cuh"

namespace skv {

namespace {

constexpr int MAX_CONSUMERS = 8;      // (+ the producer: 288 threads, which the register budget is set for)

// floats of one consumer's state in the scratch: out [G][D], then (max, sum) [G][2], rounded up to 16 bytes
// (the states are written with 16-byte stores)
__host__ __device__ constexpr int cta_part_floats(int G, int D) { return G * D + ((2 * G + 3) & ~3); }

// One try with the thread suspended until the phase completes or `ns` nanoseconds have passed (a plain
// try_wait comes back at once, and a warp that polls in a loop takes issue slots from the warps that work).
__device__ __forceinline__ bool mbar_try_wait_for(uint32_t bar, uint32_t parity, uint32_t ns)
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

// A look at the barrier that never suspends the thread.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// wait with a time limit that also gives up soon after another warp of the CTA has
__device__ __forceinline__ bool wait_or_quit(uint32_t bar, uint32_t parity, volatile int *gave_up)
{
    if (mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (;;) {
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait_for(bar, parity, 4000u)) return true;
        if (*gave_up) return false;
        const uint64_t now = global_timer_ns();
        if (t0 == 0) t0 = now;
        else if (now - t0 > 2000000000ull) return false;
    }
}

// try_wait until an absolute time (for the exit path, where one limit covers every copy still in flight)
__device__ __forceinline__ bool wait_until(uint32_t bar, uint32_t parity, uint64_t deadline_ns)
{
    for (;;) {
        for (int i = 0; i < 128; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() > deadline_ns) return false;
    }
}

// Block index a stage's barrier has last been armed for: written by the producer right after arming (and
// before the copy goes out), read by the consumer that claimed the block before it waits on the barrier.  A
// parity wait only means "the copy of block k has landed" to a waiter who knows that the barrier is in
// block k's phase; a consumer that visits the stages in no fixed order does not know, so it is told.
// Plain volatile accesses: shared-memory operations of one thread reach the SM's memory in program order,
// and a fence here would make the producer wait for its copies.
__device__ __forceinline__ void publish_issued(uint32_t addr, int k)
{
    asm volatile("st.volatile.shared::cta.s32 [%0], %1;" ::"r"(addr), "r"(k) : "memory");
}

__device__ __forceinline__ bool wait_issued(uint32_t addr, int k, volatile int *gave_up, int lane)
{
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i) {
            int v = 0;
            if (lane == 0) asm volatile("ld.volatile.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
            if (__shfl_sync(0xFFFFFFFFu, v, 0) == k) return true;
            __nanosleep(32);
        }
        if (*gave_up) return false;
        if (global_timer_ns() - t0 > 2000000000ull) return false;
    }
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Shared memory: tables (prefix, lens) | ring [S][BLOCK] | scratch [2][C] x ([G][D] fp32 out + [G][2] (max, sum))
//                | query rows [2][G][D] bf16 | full[S], empty[S], run_done[2], q_full[2] mbarriers
//                | gave_up word, claim counter, q_taken[2] | issued[S] | scratch_free[2] mbarriers
// A RUN is the part of the CTA's range inside one (sequence, kv head) segment.  What a run costs beyond its
// blocks is kept off the consumers' path, because a range holds two to five of them and the slowest CTA sets
// the end of the launch:
//   - the run's query rows are brought into shared memory by the producer, ahead of the run's first block
//     (two buffers by run parity; q_full: the rows have landed; q_taken: how many consumers have taken their
//     copy of a buffer's rows so far, a plain count that runs on, because the producer lanes that refill the
//     buffer do not see every phase a barrier would go through);
//   - at the end of run r a consumer writes its state to scratch buffer r&1 and goes straight on with run
//     r+1; the states of a run are combined by a warp of their own (warp C + 1), which gives the buffer
//     back through the scratch_free barrier of its parity (a consumer waits for that of run r-2 before it
//     writes run r's state).  Combining on the consumers cost 0.45 us per run: they all stop at the same
//     blocks, and with them the SM's copies.  Only the range's last run is combined by the consumers, all
//     together, because they have nothing else left to do then and one warp alone would make the CTA end later.
// Where the registers leave no room for the extra warp (one query head per kv head at head_dim 128) the
// consumers combine: the states of run r at the end of run r+1, when they have long been complete; order
// at the end of run r: wait for run r-1 to be complete and combine it, THEN write the state of run r and
// arrive for run r, so that a consumer that writes scratch buffer r&1 has passed the barrier of run r-1,
// which every consumer arrives at only after it has combined run r-2, the last reader of that buffer.
// INMERGE: the instance that finishes cut segments itself (DECODE_MERGE_IN_KERNEL).  It is a kernel of its own
// because it may use more registers: no CTA of the merge kernel has to fit on the SM beside it.
template <int D, class State, bool INMERGE>
__global__ void __launch_bounds__((State::MAX_CTA_CONSUMERS + (State::CTA_COMBINER ? 2 : 1)) * 32, 1)
__maxnreg__(INMERGE ? 200 : State::CTA_MAX_REGS) decode_cta_kernel(DecodeParams p, int G, int S)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BLOCK = State::BLOCK;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr bool COMBINER = State::CTA_COMBINER;     // warp C + 1 combines the runs' states; else the consumers do
    const int C = (int)(blockDim.x >> 5) - (COMBINER ? 2 : 1);   // consumer warps; warp C is the producer
    const uint64_t t_entry = p.trace ? global_timer_ns() : 0;

    const uint32_t base = smem_u32(smem_raw);
    const uint32_t pad = (128u - (base & 127u)) & 127u;
    int32_t *prefix = reinterpret_cast<int32_t *>(smem_raw + pad);
    int32_t *lens = prefix + p.B + 1;
    const size_t ring_off = pad + table_bytes(p.B);
    const uint32_t ring = base + (uint32_t)ring_off;
    const size_t scratch_off = ring_off + (size_t)S * BLOCK;
    const int part_floats = cta_part_floats(G, D);     // one consumer's state: out [G][D], then (max, sum) [G][2]
    float *scratch = reinterpret_cast<float *>(smem_raw + scratch_off);
    const int CS = C + 1;                              // states per scratch buffer: the consumers' and one from the next range
    const size_t q_off = scratch_off + (((size_t)2 * CS * part_floats * 4 + 15) & ~(size_t)15);
    const int q_bytes = G * D * 2;                     // the query rows of one kv head: a multiple of 128 bytes
    const uint16_t *q_rows = reinterpret_cast<const uint16_t *>(smem_raw + q_off);
    const size_t bars_off = q_off + 2 * (size_t)q_bytes;
    const uint32_t full = base + (uint32_t)bars_off, empty = full + 8u * S, run_done = empty + 8u * S;
    const uint32_t q_full = run_done + 16;
    volatile int *gave_up = reinterpret_cast<volatile int *>(smem_raw + bars_off + 16 * (size_t)S + 32);
    int *next_claim = const_cast<int *>(gave_up) + 1;
    volatile int *q_taken = gave_up + 2;                // [2]: consumers that have taken their copy of a buffer's rows, ever
    const uint32_t issued_at = q_full + 16 + 16;        // int [S]
    const uint32_t scratch_free = (issued_at + 4u * (uint32_t)S + 7u) & ~7u;   // two: scratch buffer r&1 has been combined
    const uint32_t nb_ready = scratch_free + 16;        // the neighbouring range's partial is in the scratch (in-kernel merging)

    {   // the layout above must fit the shared memory the launch was given (else: flag it and do nothing)
        uint32_t given;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(given));
        if (nb_ready - base + 8u > given) {
            if (threadIdx.x == 0) atomicOr(p.status, STATUS_BOUNDS);
            return;
        }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(run_done + 8 * i, C);
            mbar_init(q_full + 8 * i, 1);
            mbar_init(scratch_free + 8 * i, 1);
            q_taken[i] = 0;
        }
        mbar_init(nb_ready, 1);
        gave_up[0] = 0;
        *next_claim = 0;
        for (int s = 0; s < S; ++s) publish_issued(issued_at + 4 * s, -1);
        fence_barrier_init();
    }
    const bool early_fetch = (p.flags & DECODE_EARLY_FETCH) != 0;
    const bool reverse = (p.flags & DECODE_REVERSE) != 0;
    if (!early_fetch) pdl_wait();                      // anything read below may come from the kernel before this one
    if (warp == 0) scan_lengths(p.seq_lens, p.B, PAGE, (int64_t)p.pt_stride * PAGE, p.status, prefix, lens, lane);
    __syncthreads();

    // Merging inside the kernel: a CTA may wait for the partial of the range after its own (forward walks) or
    // before it (backward walks); the ranges are dealt so that this is always a CTA with a lower index, which
    // the hardware has started no later than this one.
    constexpr bool inmerge = INMERGE && COMBINER;
    const int64_t W = gridDim.x, w = (inmerge && !reverse) ? (int64_t)gridDim.x - 1 - blockIdx.x : blockIdx.x;
    const int64_t T = (int64_t)prefix[p.B] * p.Hkv;
    int64_t x0 = 0;
    int n = 0;
    if (T > 0) {
        x0 = worker_begin(w, T, W);
        n = (int)(worker_begin(w + 1, T, W) - x0);
    }
    const int64_t x_first = reverse ? x0 + n - 1 : x0;
    // A run that is only a piece of its segment (the range ends cut it).  Without in-kernel merging its partial
    // goes to `slot` for the merge kernel.  With it, partials travel along the block list against the walk: the
    // piece its CTA reaches first (the SOURCE: the segment's last piece in forward walks, its first in backward
    // walks) only leaves its partial; every other piece is the last run of its CTA, takes the partial at
    // `src_slot` (its neighbour's, which already holds everything beyond), adds its own and either leaves the sum
    // at `slot` or, as the FINAL piece, writes the segment's rows.  a = the run's lowest position in the list.
    struct Piece { bool crossing, source, final; int slot, src_slot; };
    auto piece_of = [&](int b, int h, int pages, int64_t a, int len) -> Piece {
        Piece q;
        const int64_t seg = (int64_t)b * p.Hkv + h, s0 = (int64_t)prefix[b] * p.Hkv + (int64_t)h * pages;
        const bool below = a > s0, above = a + len < s0 + pages;      // the segment has blocks before / after this run
        q.crossing = len != pages;
        q.source = reverse ? !below : !above;
        q.final = reverse ? !above : !below;
        q.slot = partial_slot(T, W, w, a, seg);
        q.src_slot = q.slot + (reverse ? -1 : 1);
        return q;
    };
    const int64_t n_slots = W + (int64_t)p.B * p.Hkv;

    if (warp == C) {
        // ================= producer =================
        // The range is walked in groups of 32 blocks, lane L of the warp owning block 32g + L: it finds the
        // block's place in the list and reads its page id one group AHEAD of the copies (the id is a trip to
        // L2 that must not sit between two batches of copies), then issues the block's copy itself.  Within
        // a group the copies go out PB lanes at a time, in order (one thread alone cannot issue bulk copies
        // fast enough for an SM's share of the bandwidth; and never two blocks of one batch in one stage).
        // The lane whose block opens a run first sends for the run's query rows.
        const int PB = S < 8 ? S : 8;
        const uint64_t pol_stream = make_policy_evict_first(), pol_keep = make_policy_evict_normal();
        const int keep_from = (p.keep_pct > 0 && T <= p.l2_fit_blocks) ? 0 : n - (int)(((int64_t)n * p.keep_pct) / 100);
        bool waited = !early_fetch, triggered = false, quit = false;
        // This lane's block of a group: sequence and kv head, raw page id (checked and turned into an address
        // only when the group's copies go out, so that the load stays in flight meanwhile; -1 past the end of
        // the range), whether the block is the last page of its sequence, whether it opens a run.
        struct Look { int id, b, h; bool last_page, opens; };
        auto look_up = [&](int kk) -> Look {
            Look r = {-1, 0, 0, false, false};
            if (kk >= n) return r;
            const Cursor cur = locate(prefix, p.B, p.Hkv, reverse ? x_first - kk : x_first + kk);
            r.id = __ldg(p.page_table + (int64_t)cur.b * p.pt_stride + cur.pg);
            r.b = cur.b;
            r.h = cur.h;
            r.last_page = cur.pg + 1 == cur.pages;
            r.opens = kk == 0 || (reverse ? cur.pg + 1 == cur.pages : cur.pg == 0);
            return r;
        };
        // The first run's query rows go out before anything else (unless early fetch holds them back until the
        // wait): the consumers start on them while this warp is still looking up its first page ids.
        Look cur = look_up(lane), nxt;                  // (the page ids first: they are the longest chain to the first block)
        bool first_rows_sent = false;
        if (n > 0 && waited) {
            if (lane == 0) {
                mbar_expect_tx(q_full, (uint32_t)q_bytes);
                bulk_copy_g2s(base + (uint32_t)q_off, p.Q + ((int64_t)cur.b * p.Hq + (int64_t)cur.h * G) * D, (uint32_t)q_bytes, q_full);
            }
            first_rows_sent = true;
        }
        int runs_before = 0;                            // runs opened in earlier groups
        int k = 0;                                      // first block of the current group
        for (; k < n && !quit; k += 32) {
            const int kk = k + lane;
            int id = cur.id;
            if (kk < n && (id < 0 || (int64_t)id >= p.max_pages)) {
                atomicOr(p.status, STATUS_BOUNDS);
                id = 0;
            }
            const uint8_t *src = p.layer_base + (int64_t)id * p.page_stride + (int64_t)cur.h * BLOCK;
            const unsigned openers = __ballot_sync(FULL, cur.opens);
            const int my_run = runs_before + __popc(openers & ((2u << lane) - 1u)) - 1;     // (for a lane that opens one)
            bool q_pending = false;                      // this lane's block opened a run whose query rows are not sent for yet
            auto send_for_rows = [&]() {
                // The rows of run r go into buffer r&1 once every consumer has taken its copy of run r-2's (C times
                // r/2 copies of that buffer taken in all).  All lanes stay in this loop together and each sends
                // when its turn has come: a lane that left early would stand between a later lane and its turn.
                if (!__any_sync(FULL, q_pending)) return true;
                const int qb = my_run & 1, need = C * (my_run / 2);
                const uint64_t t0 = global_timer_ns();
                bool ok = true;
                while (__any_sync(FULL, q_pending)) {
                    if (q_pending && q_taken[qb] >= need) {
                        mbar_expect_tx(q_full + 8 * qb, (uint32_t)q_bytes);
                        bulk_copy_g2s(base + (uint32_t)q_off + (uint32_t)(qb * q_bytes),
                                      p.Q + ((int64_t)cur.b * p.Hq + (int64_t)cur.h * G) * D, (uint32_t)q_bytes, q_full + 8 * qb);
                        q_pending = false;
                    }
                    if (!__any_sync(FULL, q_pending)) break;
                    if (gave_up[0] || global_timer_ns() - t0 > 2000000000ull) {
                        ok = false;
                        break;
                    }
                }
                return ok;
            };
            for (int j0 = 0; j0 < 32 && k + j0 < n && !quit; j0 += PB) {
                const bool active = lane >= j0 && lane < j0 + PB && kk < n;
                // With early fetch the ring is filled before the wait on the kernel before this one, but
                // never with a sequence's last page (its newest token may be on its way), and the wait is
                // taken at the latest when the ring has been filled once.  Query rows are sent for after it.
                bool ok = true;
                if (!waited && (k + j0 + PB > S || k + j0 >= n / 2 || __any_sync(FULL, active && cur.last_page))) {
                    pdl_wait();
                    waited = true;
                    ok = send_for_rows();              // the rows held back so far, before any copy below waits for a stage
                }
                if (!triggered && k + j0 >= n / 2) {   // the merge kernel may move in from here on
                    triggered = true;
                    pdl_trigger();
                }
                if (ok && active) {
                    const int s = kk % S;
                    if (kk >= S) ok = wait_or_quit(empty + 8 * s, (uint32_t)((kk / S - 1) & 1), gave_up);
                    if (ok) {
                        mbar_expect_tx(full + 8 * s, BLOCK);
                        publish_issued(issued_at + 4 * s, kk);
                        bulk_copy_g2s_hint(ring + (uint32_t)(s * BLOCK), src, BLOCK, full + 8 * s, kk >= keep_from ? pol_keep : pol_stream);
                    }
                    if (cur.opens && !(kk == 0 && first_rows_sent)) q_pending = true;
                }
                if (j0 == 0) nxt = look_up(k + 32 + lane);   // (after the group's first copies have gone out)
                ok = __all_sync(FULL, ok);
                if (ok && waited) ok = send_for_rows();  // (all of the group's blocks so far are out: nobody waits for one of them)
                if (!ok) {
                    if (lane == 0) { atomicOr(p.status, STATUS_TIMEOUT); gave_up[0] = 1; }
                    quit = true;
                }
            }
            if (!quit && __any_sync(FULL, q_pending)) {   // rows held back by early fetch: the range ends inside the first ring fill
                if (!waited) { pdl_wait(); waited = true; }
                if (!send_for_rows()) {
                    if (lane == 0) { atomicOr(p.status, STATUS_TIMEOUT); gave_up[0] = 1; }
                    quit = true;
                }
            }
            runs_before += __popc(openers);
            cur = nxt;
        }
        if (!waited) pdl_wait();
        if (!triggered) pdl_trigger();
        // Leave only when every copy that was issued has landed: the ring must not be written after the CTA
        // is gone.  (Normally the consumers have seen them all long ago; after a failure they may not have.)
        const int issued = k < n ? k : n;
        const uint64_t deadline = global_timer_ns() + 2000000000ull;
        for (int j = issued > S ? issued - S : 0; j < issued; ++j)
            if (!wait_until(full + 8 * (j % S), (uint32_t)((j / S) & 1), deadline)) break;
        for (int r = runs_before > 2 ? runs_before - 2 : 0; r < runs_before; ++r)
            if (!wait_until(q_full + 8 * (r & 1), (uint32_t)((r / 2) & 1), deadline)) break;
        return;
    }

    // ================= consumers =================
    // The page counts go to global memory for the merge kernel (after the wait on the kernel before this
    // one: the merge of an earlier call may still be reading this buffer).
    if (early_fetch) pdl_wait();
    if (blockIdx.x == 0 && warp < C)
        for (int i = threadIdx.x; i <= p.B; i += C * 32) p.prefix[i] = prefix[i];

    // Dynamic: whoever is free takes the next block (the consumers of an SM end together, but which blocks a
    // consumer sums, and with that the last bits of the result, vary from run to run).  In turn: block j
    // goes to consumer j mod C (reproducible bit for bit).
    const bool in_turn = (p.flags & DECODE_CLAIM_IN_TURN) != 0;
    // With blocks taken in turn and the ring a whole number of rounds deep, a stage always serves the same
    // consumer, who then sees every phase of its barrier in order and needs no telling.
    const bool ask_issued = !in_turn || S % C != 0;
    int my_next = warp;
    auto claim = [&]() -> int {
        if (in_turn) {
            const int j = my_next;
            my_next += C;
            return j;
        }
        int j = 0;
        if (lane == 0) j = atomicAdd(next_claim, 1);
        return __shfl_sync(FULL, j, 0);
    };
    // the states of run `r` (all consumers', in scratch buffer r&1) -> the segment's rows, or its partial at `slot`
    // the states of run `r` (all consumers', in scratch buffer r&1) -> the segment's rows, or its partial at `slot`;
    // by the threads first, first + step, ... of a group of `step` threads, one pair of outputs at a time
    // (n_states: the consumers' C, or C + 1 with the neighbouring range's partial behind them; rows: write the
    // segment's rows, normalised, instead of a partial)
    auto combine = [&](int r, int b, int h, bool rows, int slot, int n_states, int first, int step) {
        const float *buf = scratch + (size_t)(r & 1) * CS * part_floats;
        for (int e2 = first; e2 < G * D / 2; e2 += step) {
            const int g = (2 * e2) / D;
            // every consumer's (max, sum) of the head and its pair of outputs: all loads first
            float m_c[MAX_CONSUMERS + 1], l_c[MAX_CONSUMERS + 1];
            float2 v_c[MAX_CONSUMERS + 1];
#pragma unroll
            for (int c = 0; c < MAX_CONSUMERS + 1; ++c) {
                m_c[c] = -INFINITY;
                l_c[c] = 0.f;
                v_c[c] = make_float2(0.f, 0.f);
                if (c < n_states) {
                    const float *sc = buf + c * part_floats;
                    m_c[c] = sc[G * D + 2 * g];
                    l_c[c] = sc[G * D + 2 * g + 1];
                    v_c[c] = *reinterpret_cast<const float2 *>(sc + 2 * e2);
                }
            }
            float M = -INFINITY;
#pragma unroll
            for (int c = 0; c < MAX_CONSUMERS + 1; ++c) M = fmaxf(M, m_c[c]);
            float L = 0.f, a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int c = 0; c < MAX_CONSUMERS + 1; ++c) {
                if (m_c[c] == -INFINITY) continue;      // this consumer had no block in the run (or is not there)
                const float wt = fast_exp2(m_c[c] - M);
                L = fmaf(wt, l_c[c], L);
                a0 = fmaf(wt, v_c[c].x, a0);
                a1 = fmaf(wt, v_c[c].y, a1);
            }
            if (rows) {
                const float inv = L > 0.f ? 1.f / L : 0.f;
                uint32_t *dst = reinterpret_cast<uint32_t *>(p.out + ((int64_t)b * p.Hq + (int64_t)h * G) * D);
                dst[e2] = pack_bf16x2(a0 * inv, a1 * inv);
            } else {
                *reinterpret_cast<float2 *>(p.part_o + (int64_t)slot * G * D + 2 * e2) = make_float2(a0, a1);
                if ((2 * e2) % D == 0) *reinterpret_cast<float2 *>(p.part_ml + ((int64_t)slot * G + g) * 2) = make_float2(M, L);
            }
        }
    };

    if (COMBINER && warp == C + 1) {
        // ================= combiner =================
        // Walks the range run by run like the consumers; when all of them have handed in their state of a run
        // it combines them (the segment's rows, or its partial) and gives the scratch buffer back.  The
        // consumers never stop for it: they would all stop at the same blocks, and with them the SM's copies.
        if (inmerge && blockIdx.x == 0)                // rows of empty sequences: zeros (no merge kernel will write them)
            for (int b = 0; b < p.B; ++b)
                if (lens[b] == 0) {
                    uint32_t *dst = reinterpret_cast<uint32_t *>(p.out + (int64_t)b * p.Hq * D);
                    for (int i = lane; i < p.Hq * D / 2; i += 32) dst[i] = 0u;
                }
        // In-kernel merging: the range's last run may take its neighbour's partial.  Which run that is, and from
        // which slot, is known before the walk begins, and the neighbour reached that piece FIRST, so its partial
        // is usually there long before this CTA comes to its last run.  The warp looks at the slot's tag whenever
        // it waits for the consumers anyway and brings the partial into the scratch, behind the consumers' states
        // (of both run parities: which one the last run has is not known yet), as soon as the tag says that it is
        // complete.  Left to the last run itself, the tag's and the partial's round trips to L2 were in the open
        // whenever that run was only a few blocks long (+2 to +4 us for such a CTA, and the launch ends with them).
        Piece lastq = {false, false, false, 0, 0};
        bool takes_last = false, fetched = false;
        if (inmerge && n > 0) {
            const Cursor lc = locate(prefix, p.B, p.Hkv, reverse ? x0 : x0 + n - 1);
            const int64_t s0 = (int64_t)prefix[lc.b] * p.Hkv + (int64_t)lc.h * lc.pages;
            const int64_t a = s0 > x0 ? s0 : x0, e = s0 + lc.pages < x0 + n ? s0 + lc.pages : x0 + n;
            lastq = piece_of(lc.b, lc.h, lc.pages, a, (int)(e - a));
            takes_last = lastq.crossing && !lastq.source;
            if (takes_last && (lastq.src_slot < 0 || lastq.src_slot >= n_slots)) {
                if (lane == 0) { atomicOr(p.status, STATUS_BOUNDS); gave_up[0] = 1; }
                return;
            }
        }
        // one look at the tag; the partial, if it is there
        auto try_fetch = [&]() -> bool {
            unsigned long long tag;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(tag) : "l"(p.tags + lastq.src_slot) : "memory");
            if (!__all_sync(FULL, tag == p.epoch)) return false;
            float *dst0 = scratch + (size_t)C * part_floats, *dst1 = dst0 + (size_t)CS * part_floats;
            const float *so = p.part_o + (int64_t)lastq.src_slot * G * D, *sm = p.part_ml + (int64_t)lastq.src_slot * G * 2;
            for (int i = lane * 4; i < G * D; i += 128) {
                const float4 v = __ldcg(reinterpret_cast<const float4 *>(so + i));
                *reinterpret_cast<float4 *>(dst0 + i) = v;
                *reinterpret_cast<float4 *>(dst1 + i) = v;
            }
            for (int i = lane; i < 2 * G; i += 32) {
                const float v = __ldcg(sm + i);
                dst0[G * D + i] = v;
                dst1[G * D + i] = v;
            }
            __syncwarp();
            if (lane == 0) {
                // The tag has done its work: clear it.  A launch that is replayed from a CUDA graph carries the
                // same epoch every time, so a tag left standing would pass for this launch's in the next replay.
                // (Every tag has exactly one reader, this one; the slot is not written again before the kernel ends.)
                asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p.tags + lastq.src_slot), "l"(0ull) : "memory");
                mbar_arrive(nb_ready);
            }
            return true;
        };
        // ... until it is there (bounded)
        auto fetch_neighbour = [&]() -> bool {
            uint64_t t0 = 0;
            for (int it = 0;; ++it) {
                if (try_fetch()) return true;
                __nanosleep(64);
                if ((it & 255) == 255) {
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    const bool quit = gave_up[0] || now - t0 > 2000000000ull;
                    if (__any_sync(FULL, quit)) return false;
                }
            }
        };
        // The wait for a run's states.  This warp polls (a look that never suspends, then a short sleep) instead
        // of letting the hardware suspend it: a suspended wait with a hint of 1 us came back only every 5 to 8 us,
        // too rarely for the looks at the tag in between.  One warp per SM that looks about once a microsecond
        // takes nothing from the consumers.
        auto wait_run = [&](uint32_t bar, uint32_t parity) -> bool {
            uint64_t t0 = 0;
            for (int it = 1;; ++it) {
                const bool done = mbar_test_wait(bar, parity);
                if (__all_sync(FULL, done)) return true;
                if (takes_last && !fetched && (it & 1) == 0) fetched = try_fetch();
                __nanosleep(400);
                if ((it & 255) == 0) {
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    const bool quit = gave_up[0] || now - t0 > 2000000000ull;
                    if (__any_sync(FULL, quit)) return false;
                }
            }
        };
        Cursor cc = {0, 0, 0, 1};
        if (n > 0) cc = locate(prefix, p.B, p.Hkv, x_first);
        bool ok = true;
        for (int k = 0, run = 0; k < n && ok; ++run) {
            const int b = cc.b, h = cc.h, pages = cc.pages;
            const int to_edge = reverse ? cc.pg + 1 : pages - cc.pg;
            const int len = to_edge < n - k ? to_edge : n - k;
            const Piece q = piece_of(b, h, pages, reverse ? x0 + n - k - len : x0 + k, len);
            const bool publish = inmerge && q.crossing && !q.final;      // somebody waits for this run's partial
            const bool takes = inmerge && q.crossing && !q.source;       // (only the range's last run can)
            // the range's last run is combined by the consumers, all together, unless its partial has to be handed on
            // (rare: a range that holds a middle piece of a long segment), which one warp does more simply
            if (k + len >= n && !publish) {
                if (takes && !fetched) ok = fetched = fetch_neighbour();   // (takes: this is the last run, q is lastq)
                break;
            }
            ok = wait_run(run_done + 8 * (run & 1), (uint32_t)((run >> 1) & 1));
            if (ok && takes && !fetched) ok = fetched = fetch_neighbour();
            if (!ok) break;
            if (takes_last && !fetched) fetched = try_fetch();       // (before the work below, if it has come meanwhile)
            const int n_states = takes ? C + 1 : C;
            combine(run, b, h, !q.crossing, q.slot, n_states, lane, 32);
            __syncwarp();
            if (lane == 0) mbar_arrive(scratch_free + 8 * (run & 1));   // (first: the fence below takes microseconds while the SM streams)
            if (publish && lane == 0) {
                __threadfence();                        // the partial before its tag, for whoever reads the tag
                asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.tags + q.slot), "l"(p.epoch) : "memory");
            }
            k += len;
            if (k < n) {
                cc.pg = reverse ? cc.pg - (len - 1) : cc.pg + (len - 1);
                step(cc, prefix, p.Hkv, reverse);
            }
        }
        if (!ok && lane == 0 && !gave_up[0]) { atomicOr(p.status, STATUS_TIMEOUT); gave_up[0] = 1; }
        return;
    }

    Cursor cons = {0, 0, 0, 1};
    if (n > 0) cons = locate(prefix, p.B, p.Hkv, x_first);
    uint64_t t_first = 0;
    int k = 0, run = 0;
    int held = -1;                                     // a block of the range this consumer has claimed and not done yet
    int prev_b = 0, prev_h = 0, prev_slot = 0, prev_states = C;   // the run before this one, not yet combined
    bool prev_rows = false, prev_skip = false, failed = false;
    auto fail = [&]() {
        if (lane == 0 && !gave_up[0]) { atomicOr(p.status, STATUS_TIMEOUT); gave_up[0] = 1; }
        failed = true;
    };
    while (k < n && !failed) {
        // one run: blocks [k, k + len) of the range, all of segment (b, h)
        const int b = cons.b, h = cons.h, pages = cons.pages, n_b = lens[b];
        const int to_edge = reverse ? cons.pg + 1 : pages - cons.pg;           // blocks left in this segment
        const int len = to_edge < n - k ? to_edge : n - k;
        const int qb = run & 1;
        float *mine = scratch + ((size_t)qb * CS + warp) * part_floats;
        if (held < 0) held = claim();
        const bool has_blocks = held < k + len;
        {
            State st;
            if (has_blocks) {
                if (!wait_or_quit(q_full + 8 * qb, (uint32_t)((run >> 1) & 1), gave_up)) { fail(); break; }
                st.begin_rows(q_rows + (size_t)qb * G * D, G, lane);
            }
            __syncwarp();
            if (lane == 0) atomicAdd(const_cast<int *>(q_taken) + qb, 1);       // (with or without a copy taken)
            while (has_blocks && held < k + len) {
                const int j = held, s = j % S;
                if ((ask_issued && !wait_issued(issued_at + 4 * s, j, gave_up, lane)) ||
                    !wait_or_quit(full + 8 * s, (uint32_t)((j / S) & 1), gave_up)) {
                    fail();
                    break;
                }
                if (p.trace && t_first == 0) t_first = global_timer_ns();
                const int pg = reverse ? cons.pg - (j - k) : cons.pg + (j - k);
                const int left = n_b - pg * PAGE;
                st.page(ring + (uint32_t)(s * BLOCK), left < PAGE ? left : PAGE, p.scale_log2, lane);
                __syncwarp();                           // every lane is done reading this stage
                if (lane == 0) mbar_arrive(empty + 8 * s);
                held = claim();
            }
            if (failed) break;
            // Nobody goes on to run r+1 before everybody has handed in run r-1 (long the case, normally).  The
            // consumers must stay within a run of each other: one without a block in a run neither waits for that
            // run's query rows nor sees that phase of their barrier, and the count of rows taken, by which the
            // producer refills a buffer, is only right while nobody counts two runs ahead.
            if (run > 0) {
                if (!wait_or_quit(run_done + 8 * (qb ^ 1), (uint32_t)(((run - 1) >> 1) & 1), gave_up)) { fail(); break; }
                if (!COMBINER) combine(run - 1, prev_b, prev_h, prev_rows, prev_slot, C, (int)threadIdx.x, C * 32);    // ... and combine it here
            }
            // with a combining warp: the scratch buffer of this run's parity is free once run - 2 has been combined
            if (COMBINER && run >= 2 && !wait_or_quit(scratch_free + 8 * qb, (uint32_t)(((run >> 1) - 1) & 1), gave_up)) { fail(); break; }
            if (has_blocks) st.finish(mine, mine + G * D, 0, G, lane);
            else if (lane < G) mine[G * D + 2 * lane] = -INFINITY;             // no block of this run: nothing to contribute
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(run_done + 8 * qb);
        const Piece q = piece_of(b, h, pages, reverse ? x0 + n - k - len : x0 + k, len);
        prev_b = b;
        prev_h = h;
        prev_slot = q.slot;
        prev_rows = !q.crossing || (inmerge && q.final);                       // the segment's rows come out of this run
        prev_states = (inmerge && q.crossing && !q.source) ? C + 1 : C;        // ... with the neighbouring range's partial
        prev_skip = inmerge && q.crossing && !q.final;                         // (a partial to hand on: the combining warp's)
        k += len;
        ++run;
        if (k < n) {                                   // first block of the next run
            cons.pg = reverse ? cons.pg - (len - 1) : cons.pg + (len - 1);
            step(cons, prefix, p.Hkv, reverse);
        }
    }
    if (!failed && run > 0 && !prev_skip) {            // the last run: every consumer has nothing else left to do
        if (wait_or_quit(run_done + 8 * ((run - 1) & 1), (uint32_t)(((run - 1) >> 1) & 1), gave_up) &&
            (prev_states == C || wait_or_quit(nb_ready, 0u, gave_up)))
            combine(run - 1, prev_b, prev_h, prev_rows, prev_slot, prev_states, (int)threadIdx.x, C * 32);
        else
            fail();
    }
    if (p.trace && lane == 0) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        unsigned long long *t = p.trace + 4 * (w * C + warp);
        t[0] = smid; t[1] = t_entry; t[2] = t_first; t[3] = global_timer_ns();
    }
}

template <int D, class State>
cudaError_t launch_cta_t(const DecodeParams &p, int G, int grid, int consumers, int stages, bool pdl, cudaStream_t s)
{
    if (consumers > State::MAX_CTA_CONSUMERS) consumers = State::MAX_CTA_CONSUMERS;      // (what its registers allow)
    const size_t smem = decode_cta_smem_bytes(D, p.B, G, consumers, stages, State::BLOCK != block_bytes(D));
    const bool inmerge = State::CTA_COMBINER && (p.flags & DECODE_MERGE_IN_KERNEL) != 0;
    auto kern = inmerge ? decode_cta_kernel<D, State, State::CTA_COMBINER> : decode_cta_kernel<D, State, false>;
    cudaError_t e = ensure_dynamic_smem(kern, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)((consumers + (State::CTA_COMBINER ? 2 : 1)) * 32));
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

bool decode_cta_can_merge(int D, int kernel)
{
    if (D == 128) return kernel == 2 ? Fp8State<128>::CTA_COMBINER : kernel == 1 ? TensorCoreState<128>::CTA_COMBINER : CudaCoreState<128>::CTA_COMBINER;
    if (D == 64) return kernel == 2 ? Fp8State<64>::CTA_COMBINER : kernel == 1 ? TensorCoreState<64>::CTA_COMBINER : CudaCoreState<64>::CTA_COMBINER;
    return false;
}

size_t decode_cta_smem_bytes(int D, int B, int G, int consumers, int stages, bool fp8)
{
    if (D != 64 && D != 128) return 0;
    if (consumers < 1 || consumers > MAX_CONSUMERS || stages < 2) return 0;
    const size_t blk = fp8 ? fp8_block_bytes(D) : block_bytes(D);
    const size_t scratch = (((size_t)2 * (consumers + 1) * cta_part_floats(G, D) * 4) + 15) & ~(size_t)15;
    // 128 bytes of slack for aligning the ring base; barriers: full, empty per stage, two run barriers; two words
    // ... the query rows of two runs, their barriers, and the issued-block word of every stage
    return 128 + table_bytes(B) + (size_t)stages * blk + scratch + 2 * (size_t)G * D * 2 + 16 * (size_t)stages + 32 + 16 +
           4 * (size_t)stages + 16 + 8 + 16 + 8;       // (... the two scratch-free barriers behind them, 8-byte aligned, and
                                                       // the barrier of the neighbouring range's partial)
}

cudaError_t launch_decode_cta(const DecodeParams &p, int D, int G, int kernel, int grid, int consumers, int stages,
                              bool pdl, cudaStream_t s)
{
    if (D == 128) {
        if (kernel == 2) return launch_cta_t<128, Fp8State<128>>(p, G, grid, consumers, stages, pdl, s);
        if (kernel == 1) return launch_cta_t<128, TensorCoreState<128>>(p, G, grid, consumers, stages, pdl, s);
        return launch_cta_t<128, CudaCoreState<128>>(p, G, grid, consumers, stages, pdl, s);
    }
    if (D == 64) {
        if (kernel == 2) return launch_cta_t<64, Fp8State<64>>(p, G, grid, consumers, stages, pdl, s);
        if (kernel == 1) return launch_cta_t<64, TensorCoreState<64>>(p, G, grid, consumers, stages, pdl, s);
        return launch_cta_t<64, CudaCoreState<64>>(p, G, grid, consumers, stages, pdl, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace skv
