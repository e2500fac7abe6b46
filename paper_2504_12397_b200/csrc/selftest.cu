// Self-test of the bounded wait that every tensor-core kernel of the library relies on: one block waits on an
// mbarrier that nobody arrives at, with a caller-given cycle limit.  The wait must give up, the block records
// ALORA_ERR_TIMEOUT in the context's status word and returns through its normal exit; nothing is left waiting.
#include "alora_internal.h"
#include "tc_common.cuh"

namespace alora {

__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(long long limit_cycles, int32_t *status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(tc::smem_u32(&bar), 1);
        tc::fence_barrier_init();
    }
    __syncthreads();
    // phase 0 of a barrier with one expected arrival and no arriver never completes
    const bool done = tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && (!done || abort_flag)) report(status, ALORA_ERR_TIMEOUT);
}

}  // namespace alora

extern "C" alora_status alora_selftest_wait_timeout(alora_ctx *ctx, int64_t limit_cycles, void *stream) {
    if (!ctx) return ALORA_ERR_INVALID_ARG;
    // at most about a tenth of a second at 2 GHz: this is a check of the give-up path, not a way to stall a GPU
    if (limit_cycles < 1 || limit_cycles > 200000000LL) return ALORA_ERR_INVALID_ARG;
    ALORA_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    alora::wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles, ctx->d_status);
    ALORA_CUDA(ctx, cudaGetLastError());
    ctx->launches += 1;
    return ALORA_OK;
}
