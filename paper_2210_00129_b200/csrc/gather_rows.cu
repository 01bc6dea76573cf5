// Forward cache (Algorithm 1: only inputs[keep] is retained): a compacting row gather,
// X_keep[m, :] = X[keep_rows[m], :], moved as 16-byte vectors.  HBM-bound: it reads and writes
// M_keep * row_bytes bytes each and never touches a dropped row.  Rows in [M_keep, M_keep_cap)
// of the destination are cleared so that later products over the padded capacity see zeros.
// Also holds the optional device-side check of the index list.
#include "sbp_common.cuh"

namespace sbp {
namespace {

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kGatherThreads)
gather_rows_kernel(const uint4* __restrict__ X, uint32_t vec_per_row, const int32_t* __restrict__ keep_rows,
                   const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap, uint4* __restrict__ X_keep) {
    pdl_wait();
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const int64_t total = M_keep_cap * (int64_t)vec_per_row;
    const int64_t valid = M_keep * (int64_t)vec_per_row;
    const int64_t stride = (int64_t)gridDim.x * kGatherThreads;
    for (int64_t base = (int64_t)blockIdx.x * kGatherThreads + threadIdx.x; base < total;
         base += stride * kGatherUnroll) {
        uint4 v[kGatherUnroll];
        int64_t src[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int64_t i = base + u * stride;
            src[u] = -1;
            if (i < valid) {
                const int64_t m = i / vec_per_row;
                const uint32_t c = (uint32_t)(i - m * vec_per_row);
                src[u] = (int64_t)__ldg(keep_rows + m) * vec_per_row + c;
            }
        }
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u)
            v[u] = (src[u] >= 0) ? ld_stream(X + src[u]) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int64_t i = base + u * stride;
            if (i < total) X_keep[i] = v[u];
        }
    }
    // Only now may the next kernel's blocks take their places: the usual successor (the backward kernel) needs
    // a whole SM per block, and resident early it would push this kernel's remaining blocks off the SMs.
    pdl_launch_dependents();
}

__global__ void validate_keep_rows_kernel(const int32_t* __restrict__ keep_rows,
                                          const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap,
                                          int64_t M, int32_t* status_word) {
    pdl_launch_dependents();
    pdl_wait();
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    if (M_keep_dev != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
        const int64_t raw = (int64_t)__ldg(M_keep_dev);
        if (raw < 0 || raw > M_keep_cap) report_device_error(status_word, SBP_ERR_BAD_INDICES);
    }
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t m = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; m < M_keep; m += stride) {
        const int64_t r = keep_rows[m];
        const int64_t prev = (m > 0) ? (int64_t)keep_rows[m - 1] : -1;
        if (r < 0 || r >= M || r <= prev) report_device_error(status_word, SBP_ERR_BAD_INDICES);
    }
}

}  // namespace

cudaError_t launch_gather_rows(const void* X, int64_t row_bytes, const int32_t* keep_rows,
                               const int32_t* M_keep_dev, int64_t M_keep_cap, void* X_keep,
                               cudaStream_t stream) {
    const int64_t vec_per_row = row_bytes / 16;
    const int64_t total = M_keep_cap * vec_per_row;
    if (total == 0) return cudaSuccess;
    const int64_t per_block = (int64_t)kGatherThreads * kGatherUnroll;
    int64_t blocks = (total + per_block - 1) / per_block;
    const int64_t max_blocks = (int64_t)kNumSMs * 16;
    if (blocks > max_blocks) blocks = max_blocks;
    return launch_pdl(gather_rows_kernel, dim3((unsigned)blocks), dim3(kGatherThreads), 0, stream,
                      (const uint4*)X, (uint32_t)vec_per_row, keep_rows, M_keep_dev, M_keep_cap, (uint4*)X_keep);
}

cudaError_t launch_validate_keep_rows(const int32_t* keep_rows, const int32_t* M_keep_dev,
                                      int64_t M_keep_cap, int64_t M, int32_t* status_word,
                                      cudaStream_t stream) {
    int64_t blocks = (M_keep_cap + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
    return launch_pdl(validate_keep_rows_kernel, dim3((unsigned)blocks), dim3(256), 0, stream,
                      keep_rows, M_keep_dev, M_keep_cap, M, status_word);
}

}  // namespace sbp
