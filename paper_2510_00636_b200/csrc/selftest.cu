// ea_selftest_wait_timeout: exercises, on a healthy GPU, the route by which a bounded device-side
// wait that gives up reaches the host.  One CTA, one thread: it initialises an mbarrier that
// nothing ever arrives at, waits on it with the library's own bounded wait and a short limit, and
// on giving up raises the context's status word exactly as the production kernels' teardown does.
// No asynchronous copy is outstanding and no tensor memory is held, so the kernel simply returns.
#include "ea_internal.h"
#include "ptx_sm100.cuh"

namespace {

__global__ void wait_timeout_kernel(unsigned long long limit_ns, int* status) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x != 0) return;
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_mbar_init();
    const bool ok = ptx::mbar_wait_limited<8>(ptx::smem_u32(&bar), 0u, &abort_flag, limit_ns);
    if (!ok && abort_flag) *status = (int)EA_ERR_DEVICE_TIMEOUT;
}

}  // namespace

extern "C" ea_status ea_selftest_wait_timeout(ea_ctx* ctx, int32_t limit_us, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    if (limit_us < 1 || limit_us > 1000) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        (unsigned long long)limit_us * 1000ull, ctx->status_dev);
    ea_count_launches(ctx, 1);
    const ea_status st = EA_CHECK_LAUNCH();
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}
