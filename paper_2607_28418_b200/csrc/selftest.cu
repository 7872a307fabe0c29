// Self-test of the bounded-wait failure path.  Every device-side wait of the library gives up after
// the context's wait bound, sets the status word and lets its kernel return; this kernel makes that
// happen on purpose, without faulting or hanging anything: one CTA waits on an mbarrier whose
// phase needs two arrivals and gets one.
#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

__global__ void __launch_bounds__(64) selftest_wait_kernel(int* __restrict__ status, unsigned long long wait_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 2);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_arrive(smem_u32(&bar));   // one of the two arrivals: the phase never completes
    const bool ok = mbar_wait(smem_u32(&bar), 0, wait_ns, &abort_flag);
    if (!ok && (threadIdx.x & 31) == 0) atomicExch(status, WIDE_ERR_TIMEOUT);
}

}  // namespace

extern "C" int wide_selftest_wait(wide_ctx* ctx, void* stream) {
    if (!ctx) return WIDE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    WideLaunch l(ctx, s, "selftest_wait");
    selftest_wait_kernel<<<1, 64, 0, s>>>(ctx->d_status, ctx->wait_ns);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}
