// Bias gradient for callers that cannot allocate device memory.
//
// sbp_linear_backward needs a caller-supplied workspace for its split reductions.  Some callers
// have no way to get one: plugins and operator callbacks that are handed only their input and
// output tensors, code running under a memory pool that another framework owns and has locked
// after start-up, and services with a fixed memory budget where a late cudaMalloc may fail or
// stall every stream of the device.  For them this file offers the bias gradient with its scratch
// in a fixed device array that lives in the library image itself.
//
// The array is shared by every call on a device: it keeps whatever the last call left in it,
// and two calls whose kernels overlap on the GPU (different streams) race on it.
#include <mutex>

#include "sbp_common.cuh"

namespace {

constexpr int kStaticMaxCols = 4096;          // largest C_out this entry point accepts
constexpr int kStaticSplits = 64;             // row splits the bias kernels may use
constexpr size_t kStaticScratchFloats = (size_t)kStaticSplits * kStaticMaxCols;   // 1 MiB per device

// Partial column sums [splits, C_out].  Every GPU that loads the library holds this 1 MiB until
// the process exits.  In host code this name is only a handle for cudaGetSymbolAddress.
static __device__ __align__(256) float g_db_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device, resolved once per device.
cudaError_t scratch_address(float** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        float* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_db_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" sbp_status sbp_bias_grad_static(sbp_dtype dt, const void* dY, const int32_t* keep_rows,
                                           const int32_t* M_keep_dev, int64_t M, int64_t M_keep_cap,
                                           int64_t C_out, float* db, uint32_t flags, void* stream) {
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (dY == nullptr || keep_rows == nullptr || db == nullptr) return SBP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dY) & 15u) || (reinterpret_cast<uintptr_t>(db) & 15u) ||
        (reinterpret_cast<uintptr_t>(keep_rows) & 3u))
        return SBP_ERR_INVALID_ARG;
    if (M <= 0 || M >= (1ll << 31) || M_keep_cap < 0 || M_keep_cap > M || C_out <= 0) return SBP_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)SBP_FLAG_ACCUMULATE) return SBP_ERR_INVALID_ARG;
    if (C_out % ((dt == SBP_BF16) ? 8 : 4) != 0) return SBP_ERR_UNSUPPORTED;
    // the built-in scratch is sized for kStaticMaxCols columns; wider layers need sbp_linear_backward
    if (C_out > kStaticMaxCols) return SBP_ERR_WORKSPACE;
    if (sbp::db_workspace_bytes(dt, M_keep_cap, C_out, kStaticSplits) > kStaticScratchFloats * sizeof(float))
        return SBP_ERR_WORKSPACE;

    float* scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return SBP_ERR_CUDA;
    // Nothing in the scratch has to start at zero: the first kernel writes every partial the second reads.
    const cudaError_t e = sbp::launch_db(dt, dY, keep_rows, M_keep_dev, M_keep_cap, C_out, db,
                                         (flags & SBP_FLAG_ACCUMULATE) != 0, scratch, kStaticSplits, nullptr,
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}
