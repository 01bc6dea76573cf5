// Self-test of the bounded wait every pipeline kernel of the library relies on: a barrier that nothing ever
// completes, waited on with a short limit.  The wait must give up, report SBP_ERR_TIMEOUT through the status
// word and let the kernel return normally, so that the stream and the context stay usable - the library
// never spins without a limit, traps or faults on a GPU it shares.
#include "tc_ptx.cuh"

namespace sbp {
namespace {

__global__ void bounded_wait_selftest_kernel(uint64_t limit_ns, int32_t* status_word, int32_t* completed) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    // phase 0 of a barrier expecting one arrival that never comes
    const bool ok = ptx::mbar_wait(ptx::smem_addr(&bar), 0u, &abort_flag, status_word, limit_ns);
    if (threadIdx.x == 0) *completed = ok ? 1 : 0;
}

}  // namespace
}  // namespace sbp

extern "C" sbp_status sbp_selftest_bounded_wait(double limit_ms, int32_t* status_word, int32_t* completed, void* stream) {
    if (status_word == nullptr || completed == nullptr) return SBP_ERR_INVALID_ARG;
    if (!(limit_ms > 0.0) || limit_ms > 2000.0) return SBP_ERR_INVALID_ARG;
    sbp::bounded_wait_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>((uint64_t)(limit_ms * 1e6), status_word, completed);
    return cudaGetLastError() == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}
