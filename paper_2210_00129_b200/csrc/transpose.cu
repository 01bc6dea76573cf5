// Matrix transposes for weights kept in the [C_out, C_in] layout (SBP_FLAG_W_OUT_IN): the backward kernels work
// on W [C_in, C_out] (the paper's convention, Sec. 3.2.1), so such a W is transposed into the workspace before
// them and dW is transposed (or transpose-added) out of the workspace after them.  32 x 32 tiles through
// shared memory, both sides coalesced; HBM-bound and small next to the products.
#include "sbp_common.cuh"

namespace sbp {
namespace {

template <typename T, bool kAdd>
__global__ void __launch_bounds__(256)
transpose_kernel(const T* __restrict__ in, T* __restrict__ out, int rows, int cols, int accumulate,
                 const int32_t* __restrict__ status_word) {
    __shared__ T tile[32][33];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *status_word != 0) return;
    const int col_tiles = (cols + 31) / 32;                             // tiles are numbered row tile by row tile
    const int c0 = (int)(blockIdx.x % col_tiles) * 32, r0 = (int)(blockIdx.x / col_tiles) * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;           // 32 x 8 threads, four passes
#pragma unroll
    for (int k = 0; k < 32; k += 8) {
        const int r = r0 + ty + k, c = c0 + tx;
        if (r < rows && c < cols) tile[ty + k][tx] = in[(int64_t)r * cols + c];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 32; k += 8) {
        const int c = c0 + ty + k, r = r0 + tx;                       // out is [cols, rows]
        if (c < cols && r < rows) {
            T v = tile[tx][ty + k];
            if constexpr (kAdd) {
                if (accumulate) v += out[(int64_t)c * rows + r];
            }
            out[(int64_t)c * rows + r] = v;
        }
    }
}

}  // namespace

// out[c, r] = in[r, c] for a [rows, cols] matrix of 2- or 4-byte elements
cudaError_t launch_transpose(int elem_bytes, const void* in, void* out, int64_t rows, int64_t cols,
                             const int32_t* status_word, cudaStream_t stream) {
    const dim3 grid((unsigned)(((cols + 31) / 32) * ((rows + 31) / 32)));
    if (elem_bytes == 2)
        return launch_pdl(transpose_kernel<uint16_t, false>, grid, dim3(256), 0, stream, (const uint16_t*)in, (uint16_t*)out,
                          (int)rows, (int)cols, 0, status_word);
    return launch_pdl(transpose_kernel<uint32_t, false>, grid, dim3(256), 0, stream, (const uint32_t*)in, (uint32_t*)out,
                      (int)rows, (int)cols, 0, status_word);
}

// out[c, r] = (accumulate ? out[c, r] : 0) + in[r, c], fp32
cudaError_t launch_transpose_add_f32(const float* in, float* out, int64_t rows, int64_t cols, bool accumulate,
                                     const int32_t* status_word, cudaStream_t stream) {
    const dim3 grid((unsigned)(((cols + 31) / 32) * ((rows + 31) / 32)));
    return launch_pdl(transpose_kernel<float, true>, grid, dim3(256), 0, stream, in, out, (int)rows, (int)cols,
                      accumulate ? 1 : 0, status_word);
}

}  // namespace sbp
