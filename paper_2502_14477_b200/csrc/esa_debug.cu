// Diagnostic kernel for the bounded device-side waits (esa_debug_wait_timeout).
#include "esa_internal.h"
#include "esa_umma.cuh"

namespace esa {

namespace {

// One thread initialises an mbarrier that expects one arrival, and waits for a phase that nobody
// will ever complete.  mbar_wait gives up after `limit` cycles, records ESA_ERR_TIMEOUT in the
// status word and returns; the kernel then simply ends.
__global__ void debug_wait_kernel(int* status, long long limit) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        mbar_init_fence();
        WaitCtx wc{&abort_flag, status, limit};
        mbar_wait(smem_u32(&bar), 0, wc);
    }
}

}  // namespace

cudaError_t launch_debug_wait(esa_ctx* ctx, int64_t limit_cycles, cudaStream_t st) {
    debug_wait_kernel<<<1, 32, 0, st>>>(ctx->status, (long long)limit_cycles);
    ctx->launches += 1;
    return cudaGetLastError();
}

}  // namespace esa
