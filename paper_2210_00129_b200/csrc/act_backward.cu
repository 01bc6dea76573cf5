// Backward of a position-wise activation on packed kept rows (Sec. 3.3.1: a position-wise operation maps kept positions
// to kept positions, so between two SBP layers that share a keep set - the two linear layers of a transformer MLP or
// of a ConvNeXt block with their GELU in between - the gradient stays packed):
//     dZ[m, c] = dH[m, c] * act'(Z_keep[m, c])      m < M_keep;  rows [M_keep, M_keep_cap) of dZ = 0
// with Z_keep the cached pre-activation rows of the kept positions.  GELU in its exact form:
//     gelu(z) = z Phi(z),   gelu'(z) = Phi(z) + z phi(z) = (1 + erf(z / sqrt 2)) / 2 + z exp(-z^2 / 2) / sqrt(2 pi)
// Element-wise and HBM-bound: 16-byte vectors, two reads and one write per element; arithmetic in fp32.
#include <math.h>

#include "sbp_common.cuh"

namespace sbp {
namespace {

__device__ __forceinline__ float gelu_grad(float z) {
    return 0.5f * (1.0f + erff(z * 0.70710678118654752f)) + z * 0.3989422804014327f * expf(-0.5f * z * z);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <bool kBf16>
__global__ void __launch_bounds__(256)
act_backward_kernel(const uint4* __restrict__ Z, const uint4* __restrict__ dH, uint4* __restrict__ dZ, int64_t vec_per_row,
                    const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap, const int32_t* status_word) {
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *reinterpret_cast<const volatile int32_t*>(status_word) != 0) return;
    const int64_t valid = load_m_keep(M_keep_dev, M_keep_cap) * vec_per_row, total = M_keep_cap * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
        uint4 o = make_uint4(0u, 0u, 0u, 0u);
        if (i < valid) {
            const uint4 z = __ldg(Z + i), g = __ldg(dH + i);
            const uint32_t zw[4] = {z.x, z.y, z.z, z.w}, gw[4] = {g.x, g.y, g.z, g.w};
            uint32_t ow[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if constexpr (kBf16) {
                    ow[e] = pack_bf16x2(bf16_lo(gw[e]) * gelu_grad(bf16_lo(zw[e])), bf16_hi(gw[e]) * gelu_grad(bf16_hi(zw[e])));
                } else {
                    ow[e] = __float_as_uint(__uint_as_float(gw[e]) * gelu_grad(__uint_as_float(zw[e])));
                }
            }
            o = make_uint4(ow[0], ow[1], ow[2], ow[3]);
        }
        dZ[i] = o;
    }
}

}  // namespace

cudaError_t launch_act_backward(sbp_dtype dt, const void* Z, const void* dH, void* dZ, int64_t row_bytes, const int32_t* M_keep_dev,
                                int64_t M_keep_cap, const int32_t* status_word, cudaStream_t stream) {
    const int64_t vec_per_row = row_bytes / 16, total = M_keep_cap * vec_per_row;
    if (total == 0) return cudaSuccess;
    int64_t blocks = (total + 256 * 4 - 1) / (256 * 4);
    if (blocks > (int64_t)kNumSMs * 16) blocks = (int64_t)kNumSMs * 16;
    if (dt == SBP_BF16)
        return launch_pdl(act_backward_kernel<true>, dim3((unsigned)blocks), dim3(256), 0, stream, (const uint4*)Z, (const uint4*)dH,
                          (uint4*)dZ, vec_per_row, M_keep_dev, M_keep_cap, status_word);
    return launch_pdl(act_backward_kernel<false>, dim3((unsigned)blocks), dim3(256), 0, stream, (const uint4*)Z, (const uint4*)dH, (uint4*)dZ,
                      vec_per_row, M_keep_dev, M_keep_cap, status_word);
}

}  // namespace sbp
