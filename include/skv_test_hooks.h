/*
 * skv_test_hooks.h -- entry points that exist only in a library built with
 * -DSKV_TEST_HOOKS (the test suite builds one beside the product library; the
 * product library does not export them).  No counterpart in the paper: they
 * exercise the library's own failure reporting.
 */
#ifndef SKV_TEST_HOOKS_H
#define SKV_TEST_HOOKS_H

#include "skv.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Makes one of the library's bounded device waits run out, without a fault and
 * without anything left in flight: a one-thread kernel arms a shared-memory
 * barrier for bytes that no copy delivers, waits for them through the same
 * bounded-wait routine the attention kernels use, with a limit of limit_ms
 * (1..1000) milliseconds, and on expiry sets the timeout bit in the status word
 * exactly as those kernels do.
 *   device_status_word  device: the handle's status word, i.e. the first 4 bytes
 *                       of the pool given to skv_cache_create
 * Afterwards skv_get_status reports SKV_ERR_TIMEOUT once (reading clears it) and
 * the handle, the stream and the context are as usable as before.
 * Errors: SKV_ERR_ARG, SKV_ERR_CUDA. */
int skv_test_wait_expires(void *device_status_word, int limit_ms, void *stream);

/* A stand-in for the kernel of the caller's that computes a layer's query from the
 * layer before it ("Compute Query Q_l" of Algorithm 2; not part of the library's
 * path): q_out[i] = bf16(q_in[i] + 0 * prev_out[i]) in fp32, so that q_out cannot
 * be had before prev_out is final.  It is launched with the programmatic
 * stream-serialisation attribute, releases its dependents as its first
 * instruction and waits for the end of the kernel before it as its second: the
 * way a decoder's own kernels must behave for skv_append and skv_decode_attn of
 * the next layer to be brought forward into the end of the attention kernel of
 * this one (skv_set_decode_early_fetch).  A kernel without the attribute between
 * two attention calls keeps them apart.
 *   q_in, prev_out, q_out   device, bf16, n_elems elements each, 16-byte aligned;
 *                           n_elems a multiple of 8
 * Errors: SKV_ERR_ARG, SKV_ERR_CUDA. */
int skv_test_query_kernel(const void *q_in, const void *prev_out, void *q_out, long long n_elems, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SKV_TEST_HOOKS_H */
