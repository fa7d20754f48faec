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

// Stands for a decoder's own kernel between two attention calls: q_out = q_in + 0 * prev_out, element by element in
// fp32, rounded to bf16 (what the value is does not matter; that it cannot be had before prev_out is final does).
// Unlike a kernel that knows nothing of programmatic launches it releases its dependents at once and only then
// waits for the kernel before it, so that the launches after it can be brought forward to its start.
__global__ void __launch_bounds__(256) query_kernel(const uint4 *q_in, const uint4 *prev_out, uint4 *q_out, long long n16)
{
    skv::pdl_trigger();
    skv::pdl_wait();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n16) return;
    const uint4 a = __ldg(q_in + i), b = __ldcg(prev_out + i);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    uint32_t r[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float a0 = __uint_as_float(aw[k] << 16), a1 = __uint_as_float(aw[k] & 0xFFFF0000u);
        const float b0 = __uint_as_float(bw[k] << 16), b1 = __uint_as_float(bw[k] & 0xFFFF0000u);
        r[k] = skv::pack_bf16x2(fmaf(0.f, b0, a0), fmaf(0.f, b1, a1));
    }
    q_out[i] = make_uint4(r[0], r[1], r[2], r[3]);
}

}  // namespace

extern "C" int skv_test_query_kernel(const void *q_in, const void *prev_out, void *q_out, long long n_elems, void *stream)
{
    if (!q_in || !prev_out || !q_out || n_elems < 0 || n_elems % 8 != 0) return SKV_ERR_ARG;
    if (((uintptr_t)q_in | (uintptr_t)prev_out | (uintptr_t)q_out) & 15) return SKV_ERR_ARG;
    if (n_elems == 0) return SKV_OK;
    const long long n16 = n_elems / 8, blocks = (n16 + 255) / 256;
    if (blocks > 0x7FFFFFFFll) return SKV_ERR_ARG;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, query_kernel, static_cast<const uint4 *>(q_in), static_cast<const uint4 *>(prev_out),
                           static_cast<uint4 *>(q_out), n16) != cudaSuccess) {
        (void)cudaGetLastError();
        return SKV_ERR_CUDA;
    }
    return SKV_OK;
}

extern "C" int skv_test_wait_expires(void *device_status_word, int limit_ms, void *stream)
{
    if (!device_status_word || limit_ms < 1 || limit_ms > 1000) return SKV_ERR_ARG;
    wait_expires_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int *>(device_status_word),
                                                                     (unsigned long long)limit_ms * 1000000ull);
    if (cudaGetLastError() != cudaSuccess) return SKV_ERR_CUDA;
    return SKV_OK;
}
#endif  // SKV_TEST_HOOKS
