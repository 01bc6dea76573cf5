// Bias gradient db[j] = sum over kept rows of dY[keep_rows[m], j] (the bias term follows the
// same masking of dY as Eq. 5), and the deterministic reduction of split partial results.
//
// db: each block owns a strip of 32 16-byte column vectors and a contiguous share of the kept
// rows; a warp reads one gathered row strip as 32 x 16-byte vectors (coalesced), the eight warps
// of a block take different rows, partial sums are combined through shared memory and written
// to a [splits, C_out] scratch that a second kernel adds up in a fixed order.  HBM-bound: one
// read of the kept rows of dY.
#include "sbp_common.cuh"

namespace sbp {
namespace {

constexpr int kDbThreads = 256;
constexpr int kDbWarps = kDbThreads / 32;
constexpr int kDbUnroll = 4;
constexpr int kDbMaxSplits = 64;

template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int kElems = 4;
    __device__ static void accumulate(const uint4& v, float* acc) {
        acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
        acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void accumulate(const uint4& v, float* acc) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc[2 * i] += __uint_as_float(w[i] << 16);
            acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

inline int db_splits(int64_t M_keep_cap, int64_t col_vecs) {
    const int64_t strips = (col_vecs + 31) / 32;
    int64_t s = (2 * (int64_t)kNumSMs + strips - 1) / strips;
    const int64_t by_rows = (M_keep_cap + 63) / 64;
    if (s > by_rows) s = by_rows;
    if (s > kDbMaxSplits) s = kDbMaxSplits;
    if (s < 1) s = 1;
    return (int)s;
}

template <typename T>
__global__ void __launch_bounds__(kDbThreads)
db_partial_kernel(const uint4* __restrict__ dY, uint32_t col_vecs, const int32_t* __restrict__ keep_rows,
                  const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap, float* __restrict__ partials,
                  const int32_t* __restrict__ status_word) {
    constexpr int E = Vec16<T>::kElems;
    __shared__ float red[kDbWarps][32 * E];
    if (status_word != nullptr && *status_word != 0) return;
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t cv = blockIdx.x * 32 + lane;               // 16-byte column vector of this lane
    const int splits = gridDim.y;
    const int64_t rows_per = (M_keep + splits - 1) / splits;
    const int64_t m_begin = rows_per * blockIdx.y;
    const int64_t m_end = (m_begin + rows_per < M_keep) ? m_begin + rows_per : M_keep;

    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    if (cv < col_vecs) {
        for (int64_t m = m_begin + warp; m < m_end; m += kDbWarps * kDbUnroll) {
            uint4 v[kDbUnroll];
#pragma unroll
            for (int u = 0; u < kDbUnroll; ++u) {
                const int64_t mm = m + u * kDbWarps;
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (mm < m_end) v[u] = __ldg(dY + (int64_t)__ldg(keep_rows + mm) * col_vecs + cv);
            }
#pragma unroll
            for (int u = 0; u < kDbUnroll; ++u) Vec16<T>::accumulate(v[u], acc);
        }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) red[warp][lane * E + e] = acc[e];
    __syncthreads();
    // 32*E columns of the strip, summed over the warps in a fixed order
    for (int c = threadIdx.x; c < 32 * E; c += kDbThreads) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kDbWarps; ++w) s += red[w][c];
        const int64_t col = (int64_t)blockIdx.x * 32 * E + c;
        if (col < (int64_t)col_vecs * E) partials[(int64_t)blockIdx.y * col_vecs * E + col] = s;
    }
}

__global__ void __launch_bounds__(256)
reduce_partials_kernel(const float4* __restrict__ partials, int splits, int64_t n_vec, float4* __restrict__ out,
                       int accumulate, const int32_t* __restrict__ status_word) {
    if (status_word != nullptr && *status_word != 0) return;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
        float4 s = accumulate ? out[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k = 0; k < splits; ++k) {
            const float4 p = __ldg(partials + (int64_t)k * n_vec + i);
            s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
        }
        out[i] = s;
    }
}

}  // namespace

size_t db_workspace_bytes(int64_t M_keep_cap, int64_t C_out) {
    (void)M_keep_cap;
    return (size_t)kDbMaxSplits * (size_t)C_out * sizeof(float);
}

cudaError_t launch_db(sbp_dtype dt, const void* dY, const int32_t* keep_rows, const int32_t* M_keep_dev,
                      int64_t M_keep_cap, int64_t C_out, float* db, bool accumulate, float* workspace,
                      const int32_t* status_word, cudaStream_t stream) {
    const int64_t elems = (dt == SBP_BF16) ? 8 : 4;
    const int64_t col_vecs = C_out / elems;
    const int splits = db_splits(M_keep_cap, col_vecs);
    const dim3 grid((unsigned)((col_vecs + 31) / 32), (unsigned)splits);
    if (dt == SBP_BF16)
        db_partial_kernel<__nv_bfloat16><<<grid, kDbThreads, 0, stream>>>(
            (const uint4*)dY, (uint32_t)col_vecs, keep_rows, M_keep_dev, M_keep_cap, workspace, status_word);
    else
        db_partial_kernel<float><<<grid, kDbThreads, 0, stream>>>(
            (const uint4*)dY, (uint32_t)col_vecs, keep_rows, M_keep_dev, M_keep_cap, workspace, status_word);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_reduce_partials(workspace, splits, C_out, db, accumulate, status_word, stream);
}

cudaError_t launch_reduce_partials(const float* partials, int splits, int64_t n, float* out,
                                   bool accumulate, const int32_t* status_word, cudaStream_t stream) {
    const int64_t n_vec = n / 4;   // n is a multiple of 4 for every caller
    int64_t blocks = (n_vec + 255) / 256;
    if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
    if (blocks < 1) blocks = 1;
    reduce_partials_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const float4*)partials, splits, n_vec,
                                                                (float4*)out, accumulate ? 1 : 0, status_word);
    return cudaGetLastError();
}

}  // namespace sbp
