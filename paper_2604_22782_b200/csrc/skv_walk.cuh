// Walking the flattened (sequence, kv head, page) block list of a decode call, shared by the split-K
// kernels.
#pragma once
#include "skv_common.cuh"

namespace skv {

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

// One position forward (or backward).  Only called while another position remains in that
// direction, so b stays inside [0, B).
__device__ __forceinline__ void step(Cursor &c, const int32_t *prefix, int Hkv, bool reverse)
{
    if (!reverse) {
        if (++c.pg < c.pages) return;
        c.pg = 0;
        if (++c.h < Hkv) return;
        c.h = 0;
        do {
            ++c.b;
            c.pages = prefix[c.b + 1] - prefix[c.b];
        } while (c.pages == 0);
    } else {
        if (--c.pg >= 0) return;
        if (--c.h < 0) {
            c.h = Hkv - 1;
            do {
                --c.b;
                c.pages = prefix[c.b + 1] - prefix[c.b];
            } while (c.pages == 0);
        }
        c.pg = c.pages - 1;
    }
}

// By one warp: lens[i] = max(seq_lens[i], 0) and prefix[i] = number of units (pages, or tiles of several
// pages: `unit_tokens` tokens each, the last one of a sequence possibly short) of the sequences before i,
// per kv head; prefix[B] = all of them.  A length that needs more pages than a page-table row holds
// (max_tokens = pt_stride * PAGE) is cut to what the row holds and flagged in the status word, so that no
// page id is ever read past the end of a row.
__device__ __forceinline__ void scan_lengths(const int32_t *seq_lens, int B, int unit_tokens, int64_t max_tokens,
                                             int *status, int32_t *prefix, int32_t *lens, int lane)
{
    int carry = 0;
    for (int i0 = 0; i0 < B; i0 += 32) {
        const int i = i0 + lane;
        int n = 0, v = 0;
        if (i < B) {
            n = __ldg(seq_lens + i);
            n = n > 0 ? n : 0;
            if ((int64_t)n > max_tokens) {
                n = (int)max_tokens;
                if (status) atomicOr(status, STATUS_BOUNDS);
            }
            v = (n + unit_tokens - 1) / unit_tokens;
            lens[i] = n;
        }
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int u = __shfl_up_sync(0xFFFFFFFFu, v, d);
            if (lane >= d) v += u;
        }
        if (i < B) prefix[i + 1] = carry + v;
        carry += __shfl_sync(0xFFFFFFFFu, v, 31);
    }
    if (lane == 0) prefix[0] = 0;
}

// Shared-memory carve-up (dynamic): prefix[B+1] | lens[B] | rings | barriers | CTA arrival word
__host__ __device__ inline size_t table_bytes(int B) { return (((size_t)(2 * B + 1) * 4) + 127) & ~(size_t)127; }

// ---------------------------------------------------------------------------
// Where the partials of a segment live.  The segment's blocks are [s0, s0 + pages) of the flattened
// list.  Normally worker w writes the partial of its run inside segment seg to slot  w + seg, so a
// segment's partials sit in consecutive slots.  When there are fewer blocks than workers every
// non-empty range is a single block x, and its partial goes to slot  x + seg  (consecutive again).
// ---------------------------------------------------------------------------
__device__ __forceinline__ int partial_slot(int64_t T, int64_t W, int64_t w, int64_t x_any, int64_t seg)
{
    return (int)((T < W ? x_any : w) + seg);
}

}  // namespace skv
