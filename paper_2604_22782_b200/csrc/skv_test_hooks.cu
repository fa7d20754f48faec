// Test hooks of the skv library (see include/skv_test_hooks.h).  Compiled to nothing unless SKV_TEST_HOOKS is
// defined: the product library does not contain them.
#ifdef SKV_TEST_HOOKS
#include "../../include/skv_test_hooks.h"
#include "skv_common.cuh"

namespace {

// One CTA, one thread: arms a barrier for bytes that nobody sends, waits for them through the kernels' own
// bounded wait with a short limit, reports the expiry in the status word as the kernels do, and returns.
// No copy is in flight and nothing else is touched, so the context stays usable.
__global__ void wait_expires_kernel(int *status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    const uint32_t bar = skv::smem_u32(&bar_storage);
    skv::mbar_init(bar, 1);
    skv::fence_barrier_init();
    skv::mbar_expect_tx(bar, 4096);                       // phase 0 now needs 4096 bytes that never arrive
    if (!skv::mbar_wait_limited(bar, 0, limit_ns)) atomicOr(status, skv::STATUS_TIMEOUT);
}

}  // namespace

extern "C" int skv_test_wait_expires(void *device_status_word, int limit_ms, void *stream)
{
    if (!device_status_word || limit_ms < 1 || limit_ms > 1000) return SKV_ERR_ARG;
    wait_expires_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int *>(device_status_word),
                                                                     (unsigned long long)limit_ms * 1000000ull);
    if (cudaGetLastError() != cudaSuccess) return SKV_ERR_CUDA;
    return SKV_OK;
}
#endif  // SKV_TEST_HOOKS
