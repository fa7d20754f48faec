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

#ifdef __cplusplus
}
#endif
#endif /* SKV_TEST_HOOKS_H */
