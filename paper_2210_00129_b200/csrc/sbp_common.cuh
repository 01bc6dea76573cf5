// Shared device/host helpers of the SBP library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <mutex>

#include "../../include/sbp.h"

namespace sbp {

constexpr int kNumSMs = 148;            // B200: 2 dies x 74 SMs; grids are sized in multiples of this

// Status codes are shared with the C header; device code writes them to the caller's status word.
__device__ __forceinline__ void report_device_error(int32_t* status_word, int32_t code) {
    if (status_word != nullptr) atomicCAS(status_word, 0, code);
}

// Programmatic dependent launch: every kernel of the library lets its successor start launching
// right away and itself waits for its predecessor's results before touching global memory, so
// launch latency and block scheduling overlap with the tail of the previous kernel.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// Opt a kernel in to more than 48 KB of dynamic shared memory.  The attribute belongs to the (kernel, device) pair,
// so it is set once per device a process launches the kernel on, not once per process.
constexpr int kMaxDevices = 64;
template <auto Kernel>
inline cudaError_t opt_in_dynamic_smem(int bytes) {
    static std::mutex mu;
    static bool done[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    std::lock_guard<std::mutex> lock(mu);
    if (!done[dev]) {
        e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    return cudaSuccess;
}
// the same with thread-block clusters of `cluster_x` CTAs along x
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster_x,
                                      cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Row map of the backward kernels: keep_rows[m], or m itself when the tensor is already compact (Sec. 3.3.1:
// with the same keep set on consecutive layers the kept rows can stay packed between them).
__device__ __forceinline__ int32_t mapped_row(const int32_t* rows, int64_t m) {
    return rows != nullptr ? __ldg(rows + m) : (int32_t)m;
}

// Number of valid kept rows: the device-side count when given, else the host capacity.
__device__ __forceinline__ int64_t load_m_keep(const int32_t* M_keep_dev, int64_t M_keep_cap) {
    if (M_keep_dev == nullptr) return M_keep_cap;
    int64_t v = (int64_t)__ldg(M_keep_dev);
    if (v < 0) v = 0;
    return v < M_keep_cap ? v : M_keep_cap;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies with a Weyl key
// schedule.  Device-side implementation used by the keep-index sampler.
// ---------------------------------------------------------------------------------------------
struct PhiloxWords { uint32_t w[4]; };

__device__ __forceinline__ PhiloxWords philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                     uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t lo0 = 0xD2511F53u * c0;
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0);
        const uint32_t lo1 = 0xCD9E8D57u * c2;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2);
        const uint32_t t0 = hi1 ^ c1 ^ k0;
        const uint32_t t2 = hi0 ^ c3 ^ k1;
        c0 = t0; c1 = lo1; c2 = t2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    PhiloxWords out;
    out.w[0] = c0; out.w[1] = c1; out.w[2] = c2; out.w[3] = c3;
    return out;
}

// ---------------------------------------------------------------------------------------------
// Launch entry points of the individual kernels (defined in their own .cu files).
// None synchronises.
// ---------------------------------------------------------------------------------------------
uint32_t sample_keep_max_frames();      // most frames a whole-frame (temporal) mask can choose among
cudaError_t launch_sample_keep(int mode, int grid_family, int64_t B, int64_t H, int64_t W, int64_t K,
                               uint64_t seed, uint32_t step, uint32_t first_sample, bool share_mask,
                               int32_t* keep_rows, int32_t* keep_offsets, cudaStream_t stream);

cudaError_t launch_gather_rows(const void* X, int64_t row_bytes, const int32_t* keep_rows,
                               const int32_t* M_keep_dev, int64_t M_keep_cap, void* X_keep,
                               cudaStream_t stream);

cudaError_t launch_validate_keep_rows(const int32_t* keep_rows, const int32_t* M_keep_dev,
                                      int64_t M_keep_cap, int64_t M, int32_t* status_word,
                                      cudaStream_t stream);

// partial column sums of the kept rows of dY -> db (deterministic two-pass reduction)
// max_splits bounds the number of row splits (and so the scratch: splits * C_out floats)
constexpr int kDbMaxSplits = 512;
size_t db_workspace_bytes(sbp_dtype dt, int64_t M_keep_cap, int64_t C_out, int max_splits);
cudaError_t launch_db(sbp_dtype dt, const void* dY, const int32_t* keep_rows, const int32_t* M_keep_dev,
                      int64_t M_keep_cap, int64_t C_out, float* db, bool accumulate, float* workspace,
                      int max_splits, const int32_t* status_word, cudaStream_t stream);

// out[i] = (accumulate ? out[i] : 0) + sum_s partials[s*n + i], summed in ascending s
cudaError_t launch_reduce_partials(const float* partials, int splits, int64_t n, float* out,
                                   bool accumulate, const int32_t* status_word, cudaStream_t stream);

// two such reductions in one launch (both with the same accumulate setting)
cudaError_t launch_reduce_partials_pair(const float* partials_a, int splits_a, int64_t n_a, float* out_a,
                                        const float* partials_b, int splits_b, int64_t n_b, float* out_b,
                                        bool accumulate, const int32_t* status_word, cudaStream_t stream);

// plain-FMA (CUDA-core) products for fp32 and for bf16 shapes the tensor-core kernels do not take
size_t simt_dw_workspace_bytes(int64_t M_keep_cap, int64_t C_in, int64_t C_out);
int    simt_dw_kernel_count(int64_t M_keep_cap, int64_t C_in, int64_t C_out);
cudaError_t launch_simt_dw(sbp_dtype dt, const void* X_keep, const void* dY, const int32_t* keep_rows,
                           const int32_t* M_keep_dev, int64_t M_keep_cap, int64_t C_in, int64_t C_out,
                           float* dW, bool accumulate, float* workspace, const int32_t* status_word,
                           cudaStream_t stream);
// dy_rows / dx_rows: row m of the product reads row dy_rows[m] of dY and writes row dx_rows[m] of dX
// (nullptr = m itself); M = rows of dX
cudaError_t launch_simt_dx(sbp_dtype dt, const void* dY, const void* W, const int32_t* dy_rows,
                           const int32_t* dx_rows, const int32_t* M_keep_dev, int64_t M, int64_t M_keep_cap,
                           int64_t C_in, int64_t C_out, void* dX, const int32_t* status_word, cudaStream_t stream);

// transposes for weights in the [C_out, C_in] layout
cudaError_t launch_transpose(int elem_bytes, const void* in, void* out, int64_t rows, int64_t cols,
                             const int32_t* status_word, cudaStream_t stream);
cudaError_t launch_transpose_add_f32(const float* in, float* out, int64_t rows, int64_t cols, bool accumulate,
                                     const int32_t* status_word, cudaStream_t stream);

// forward of the layer, Y = X W + bias (bias nullable)
// w_out_in: W is stored [C_out, C_in] instead of [C_in, C_out]
cudaError_t launch_simt_forward(sbp_dtype dt, const void* X, const void* W, bool w_out_in, const float* bias, int64_t M,
                                int64_t C_in, int64_t C_out, void* Y, const int32_t* status_word, cudaStream_t stream);
bool   tc_forward_supported(int64_t M, int64_t C_in, int64_t C_out);
// bf16 forward on the tensor cores; when X_keep is given the same kernel also writes the forward cache
sbp_status launch_tc_forward(const void* X, const void* W, bool w_out_in, const float* bias, int64_t M, int64_t C_in, int64_t C_out,
                             void* Y, const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap,
                             void* X_keep, int32_t* status_word, cudaStream_t stream);

// dZ = dH * gelu'(Z_keep) on packed kept rows (element-wise)
cudaError_t launch_act_backward(sbp_dtype dt, const void* Z, const void* dH, void* dZ, int64_t row_bytes, const int32_t* M_keep_dev,
                                int64_t M_keep_cap, const int32_t* status_word, cudaStream_t stream);

// stride >= kernel convolutions as linear layers on patch rows: gather of the kept patches, scatter of their gradients
cudaError_t launch_patch_gather(const void* X, int64_t H, int64_t W, int64_t pos_bytes, int64_t k, int64_t s,
                                const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap, void* X_keep,
                                cudaStream_t stream);
cudaError_t launch_patch_scatter(const void* dXp, int64_t B, int64_t H, int64_t W, int64_t pos_bytes, int64_t k, int64_t s,
                                 const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap, void* dX,
                                 int32_t* slot, const int32_t* status_word, cudaStream_t stream);

// SBP attention backward on token subsets (bf16, head dimension 64, at most attention_max_tokens() kept tokens per sample
// and side); null row lists mean every token of the sample
bool    attention_supported(sbp_dtype dt, int64_t head_dim);
int64_t attention_max_tokens();
cudaError_t launch_attention_backward(const void* Q, const void* K, const void* V, int64_t ld_qkv, const void* dA, int64_t ld_da,
                                      const int32_t* q_rows, const int32_t* q_offs, const int32_t* k_rows, const int32_t* k_offs,
                                      int64_t B, int64_t N, int64_t heads, int64_t most_tokens, void* dQ, void* dK, void* dV,
                                      int64_t ld_out, bool zero_other_rows, int32_t* status_word, cudaStream_t stream);

// tcgen05 / TMEM bf16 products
bool   tc_shapes_supported(int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out);
size_t tc_dw_workspace_bytes(int64_t M_keep_cap, int64_t C_in, int64_t C_out);
int64_t tc_plan_searches();              // split-plan searches run so far in this process
int    tc_backward_kernel_count(int64_t M_keep_cap, int64_t C_in, int64_t C_out, bool want_dw, bool want_dx,
                                bool want_db, bool dy_packed);
// dW (nullable) and dX (nullable) of one layer in a single persistent kernel (+ the split reduce); when db is
// given its column sums ride along in the same kernel (db_workspace: kNumSMs * C_out floats) + one reduce
// (dy_rows / dx_rows as for launch_simt_dx)
sbp_status launch_tc_backward(const void* X_keep, const void* dY, const void* W, const int32_t* dy_rows,
                              const int32_t* dx_rows, const int32_t* M_keep_dev, int64_t M, int64_t M_keep_cap, int64_t C_in,
                              int64_t C_out, float* dW, bool accumulate, void* dX, float* db, float* workspace,
                              float* db_workspace, int32_t* status_word, cudaStream_t stream);

}  // namespace sbp
