// Plain-FMA (CUDA-core) versions of the two SBP products of Eq. 5, used for the fp32 path (whose
// 1e-5 tolerance rules out reduced-precision tensor-core modes) and for bf16 shapes too small or
// too ragged for the tensor-core kernels.  Shared-memory tiled, 64x64 outputs per 256-thread block,
// fp32 accumulation.
//   dW[i, j] = sum_m X_keep[m, i] * dY[keep_rows[m], j]        (split over m, fixed-order reduce)
//   dX[keep_rows[m], i] = sum_j dY[keep_rows[m], j] * W[i, j]; every other row of dX = +0.0
#include "sbp_common.cuh"

namespace sbp {
namespace {

constexpr int kTile = 64;
constexpr int kTileK = 16;
constexpr int kSimtThreads = 256;
constexpr int kSimtMaxSplits = 32;

template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) {
    return __ldg(reinterpret_cast<const float4*>(p));
}
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                       __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
}
template <typename T> __device__ __forceinline__ void store4(T* p, float4 v);
template <> __device__ __forceinline__ void store4<float>(float* p, float4 v) {
    *reinterpret_cast<float4*>(p) = v;
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float4 v) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}

inline int simt_dw_splits(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    const int64_t tiles = ((C_in + kTile - 1) / kTile) * ((C_out + kTile - 1) / kTile);
    int64_t s = (2 * (int64_t)kNumSMs + tiles - 1) / tiles;
    const int64_t by_rows = (M_keep_cap + 255) / 256;
    if (s > by_rows) s = by_rows;
    if (s > kSimtMaxSplits) s = kSimtMaxSplits;
    if (s < 1) s = 1;
    return (int)s;
}

template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
simt_dw_kernel(const T* __restrict__ X_keep, const T* __restrict__ dY, const int32_t* __restrict__ keep_rows,
               const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap, int C_in, int C_out,
               float* __restrict__ out, int64_t split_stride, int accumulate,
               const int32_t* __restrict__ status_word) {
    __shared__ __align__(16) float As[kTileK][kTile];
    __shared__ __align__(16) float Bs[kTileK][kTile];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *status_word != 0) return;
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const int splits = gridDim.z;
    int64_t rows_per = (M_keep + splits - 1) / splits;
    rows_per = (rows_per + kTileK - 1) / kTileK * kTileK;
    const int64_t m_begin = rows_per * blockIdx.z;
    const int64_t m_end = (m_begin + rows_per < M_keep) ? m_begin + rows_per : M_keep;
    const int i0 = blockIdx.y * kTile, j0 = blockIdx.x * kTile;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int lk = threadIdx.x >> 4, lc = (threadIdx.x & 15) * 4;      // loader: row of the k-slab, 4 columns

    float acc[4][4] = {};
    for (int64_t m0 = m_begin; m0 < m_end; m0 += kTileK) {
        const int64_t m = m0 + lk;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (m < m_end) {
            if (i0 + lc < C_in) a = load4<T>(X_keep + m * C_in + i0 + lc);
            if (j0 + lc < C_out) b = load4<T>(dY + (int64_t)mapped_row(keep_rows, m) * C_out + j0 + lc);
        }
        *reinterpret_cast<float4*>(&As[lk][lc]) = a;
        *reinterpret_cast<float4*>(&Bs[lk][lc]) = b;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kTileK; ++k) {
            const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(ar[r], br[c], acc[r][c]);
        }
        __syncthreads();
    }
    float* dst = out + (int64_t)blockIdx.z * split_stride;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r, j = j0 + tx * 4;
        if (i < C_in && j < C_out) {
            float4 v = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            float4* p = reinterpret_cast<float4*>(dst + (int64_t)i * C_out + j);
            if (accumulate) { const float4 o = *p; v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
            *p = v;
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
simt_dx_kernel(const T* __restrict__ dY, const T* __restrict__ W, const int32_t* __restrict__ dy_rows,
               const int32_t* __restrict__ dx_rows, const int32_t* __restrict__ M_keep_dev, int64_t M, int64_t M_keep_cap, int C_in, int C_out,
               T* __restrict__ dX, const int32_t* __restrict__ status_word) {
    __shared__ __align__(16) float As[kTileK][kTile + 4];
    __shared__ __align__(16) float Bs[kTileK][kTile + 4];
    // rows[0] = output row before the tile (or -1), rows[1 + t] = output rows of the tile, M past the last kept
    // row; src[t] = rows of dY the tile reads
    __shared__ int64_t rows[kTile + 2];
    __shared__ int64_t src[kTile];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *status_word != 0) return;
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const int64_t m0 = (int64_t)blockIdx.x * kTile;
    const int i0 = blockIdx.y * kTile;
    const int cols = (C_in - i0 < kTile) ? C_in - i0 : kTile;   // multiple of 4
    const int quads = cols / 4;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

    if (M_keep == 0) {                       // nothing kept: the first row tile clears its column strip
        if (blockIdx.x == 0) {
            for (int64_t t = threadIdx.x; t < M * quads; t += kSimtThreads)
                store4<T>(dX + (t / quads) * C_in + i0 + (int)(t % quads) * 4, zero4);
        }
        return;
    }
    if (m0 >= M_keep) return;
    const int tile_rows = (int)((M_keep - m0 < kTile) ? M_keep - m0 : kTile);
    for (int t = threadIdx.x; t <= kTile + 1; t += kSimtThreads) {
        const int64_t m = m0 + t - 1;
        rows[t] = (m < 0) ? -1 : (m < M_keep ? (int64_t)mapped_row(dx_rows, m) : M);
        if (t >= 1 && t <= kTile) src[t - 1] = (m < M_keep) ? (int64_t)mapped_row(dy_rows, m) : -1;
    }
    __syncthreads();

    // zero the dropped rows that precede each kept row of this tile (and, after the very last
    // kept row, the rest of the matrix): every dropped row is written by exactly one block
    {
        const int last = (m0 + tile_rows == M_keep) ? tile_rows + 1 : tile_rows;
        for (int t = 1; t <= last; ++t) {
            const int64_t lo = rows[t - 1] + 1, hi = rows[t];
            for (int64_t w = threadIdx.x; w < (hi - lo) * quads; w += kSimtThreads)
                store4<T>(dX + (lo + w / quads) * C_in + i0 + (int)(w % quads) * 4, zero4);
        }
    }

    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int lr = threadIdx.x >> 2, lc = (threadIdx.x & 3) * 4;    // loader: tile row, 4 of the 16 k columns
    const int64_t a_row = (lr < tile_rows) ? src[lr] : -1;
    float acc[4][4] = {};
    for (int j0 = 0; j0 < C_out; j0 += kTileK) {
        float4 a = zero4, b = zero4;
        if (j0 + lc < C_out) {
            if (a_row >= 0) a = load4<T>(dY + a_row * C_out + j0 + lc);
            if (i0 + lr < C_in) b = load4<T>(W + (int64_t)(i0 + lr) * C_out + j0 + lc);
        }
        As[lc + 0][lr] = a.x; As[lc + 1][lr] = a.y; As[lc + 2][lr] = a.z; As[lc + 3][lr] = a.w;
        Bs[lc + 0][lr] = b.x; Bs[lc + 1][lr] = b.y; Bs[lc + 2][lr] = b.z; Bs[lc + 3][lr] = b.w;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kTileK; ++k) {
            const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(ar[r], br[c], acc[r][c]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int t = ty * 4 + r, i = i0 + tx * 4;
        if (t < tile_rows && i < C_in)
            store4<T>(dX + rows[1 + t] * C_in + i, make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]));
    }
}


// Forward of the layer, Y[m, j] = sum_i X[m, i] * W[i, j] + bias[j] (Eq. 2): 64 x 64 outputs per block.
// The X tile is loaded along i (its contiguous side) and stored transposed, the W tile along j.
template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
simt_forward_kernel(const T* __restrict__ X, const T* __restrict__ W, int w_out_in, const float* __restrict__ bias,
                    int64_t M, int C_in, int C_out, T* __restrict__ Y, const int32_t* __restrict__ status_word) {
    __shared__ __align__(16) float As[kTileK][kTile + 4];
    __shared__ __align__(16) float Bs[kTileK][kTile];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *status_word != 0) return;
    const int64_t m0 = (int64_t)blockIdx.x * kTile;
    const int j0 = blockIdx.y * kTile;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int ar = threadIdx.x >> 2, ac = (threadIdx.x & 3) * 4;      // X loader: tile row, 4 of the 16 k columns
    const int bk = threadIdx.x >> 4, bc = (threadIdx.x & 15) * 4;     // W loader: k row, 4 of the 64 columns
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float acc[4][4] = {};
    for (int i0 = 0; i0 < C_in; i0 += kTileK) {
        float4 a = zero4, b = zero4;
        if (m0 + ar < M && i0 + ac < C_in) a = load4<T>(X + (m0 + ar) * C_in + i0 + ac);
        As[ac + 0][ar] = a.x; As[ac + 1][ar] = a.y; As[ac + 2][ar] = a.z; As[ac + 3][ar] = a.w;
        if (!w_out_in) {
            if (i0 + bk < C_in && j0 + bc < C_out) b = load4<T>(W + (int64_t)(i0 + bk) * C_out + j0 + bc);
            *reinterpret_cast<float4*>(&Bs[bk][bc]) = b;
        } else {                                                      // W [C_out, C_in]: loaded along i like the X tile
            if (j0 + ar < C_out && i0 + ac < C_in) b = load4<T>(W + (int64_t)(j0 + ar) * C_in + i0 + ac);
            Bs[ac + 0][ar] = b.x; Bs[ac + 1][ar] = b.y; Bs[ac + 2][ar] = b.z; Bs[ac + 3][ar] = b.w;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kTileK; ++k) {
            const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float a4[4] = {av.x, av.y, av.z, av.w}, b4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(a4[r], b4[c], acc[r][c]);
        }
        __syncthreads();
    }
    const int j = j0 + tx * 4;
    if (j < C_out) {
        float4 bv = zero4;
        if (bias != nullptr) bv = __ldg(reinterpret_cast<const float4*>(bias + j));
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int64_t m = m0 + ty * 4 + r;
            if (m < M)
                store4<T>(Y + m * C_out + j, make_float4(acc[r][0] + bv.x, acc[r][1] + bv.y, acc[r][2] + bv.z, acc[r][3] + bv.w));
        }
    }
}

}  // namespace

cudaError_t launch_simt_forward(sbp_dtype dt, const void* X, const void* W, bool w_out_in, const float* bias, int64_t M,
                                int64_t C_in, int64_t C_out, void* Y, const int32_t* status_word, cudaStream_t stream) {
    const dim3 grid((unsigned)((M + kTile - 1) / kTile), (unsigned)((C_out + kTile - 1) / kTile));
    if (dt == SBP_BF16)
        return launch_pdl(simt_forward_kernel<__nv_bfloat16>, grid, dim3(kSimtThreads), 0, stream,
                          (const __nv_bfloat16*)X, (const __nv_bfloat16*)W, w_out_in ? 1 : 0, bias, M, (int)C_in,
                          (int)C_out, (__nv_bfloat16*)Y, status_word);
    return launch_pdl(simt_forward_kernel<float>, grid, dim3(kSimtThreads), 0, stream, (const float*)X, (const float*)W,
                      w_out_in ? 1 : 0, bias, M, (int)C_in, (int)C_out, (float*)Y, status_word);
}

size_t simt_dw_workspace_bytes(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    const int s = simt_dw_splits(M_keep_cap, C_in, C_out);
    return s > 1 ? (size_t)s * (size_t)C_in * (size_t)C_out * sizeof(float) : 0;
}

int simt_dw_kernel_count(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    return simt_dw_splits(M_keep_cap, C_in, C_out) > 1 ? 2 : 1;
}

cudaError_t launch_simt_dw(sbp_dtype dt, const void* X_keep, const void* dY, const int32_t* keep_rows,
                           const int32_t* M_keep_dev, int64_t M_keep_cap, int64_t C_in, int64_t C_out,
                           float* dW, bool accumulate, float* workspace, const int32_t* status_word,
                           cudaStream_t stream) {
    const int splits = simt_dw_splits(M_keep_cap, C_in, C_out);
    const dim3 grid((unsigned)((C_out + kTile - 1) / kTile), (unsigned)((C_in + kTile - 1) / kTile), (unsigned)splits);
    float* out = splits > 1 ? workspace : dW;
    const int acc_in_kernel = (splits == 1 && accumulate) ? 1 : 0;
    const int64_t split_stride = C_in * C_out;
    cudaError_t e;
    if (dt == SBP_BF16)
        e = launch_pdl(simt_dw_kernel<__nv_bfloat16>, grid, dim3(kSimtThreads), 0, stream,
                       (const __nv_bfloat16*)X_keep, (const __nv_bfloat16*)dY, keep_rows, M_keep_dev, M_keep_cap,
                       (int)C_in, (int)C_out, out, split_stride, acc_in_kernel, status_word);
    else
        e = launch_pdl(simt_dw_kernel<float>, grid, dim3(kSimtThreads), 0, stream,
                       (const float*)X_keep, (const float*)dY, keep_rows, M_keep_dev, M_keep_cap,
                       (int)C_in, (int)C_out, out, split_stride, acc_in_kernel, status_word);
    if (e != cudaSuccess || splits == 1) return e;
    return launch_reduce_partials(workspace, splits, C_in * C_out, dW, accumulate, status_word, stream);
}

cudaError_t launch_simt_dx(sbp_dtype dt, const void* dY, const void* W, const int32_t* dy_rows, const int32_t* dx_rows,
                           const int32_t* M_keep_dev, int64_t M, int64_t M_keep_cap, int64_t C_in,
                           int64_t C_out, void* dX, const int32_t* status_word, cudaStream_t stream) {
    int64_t row_tiles = (M_keep_cap + kTile - 1) / kTile;
    if (row_tiles < 1) row_tiles = 1;
    const dim3 grid((unsigned)row_tiles, (unsigned)((C_in + kTile - 1) / kTile));
    if (dt == SBP_BF16)
        return launch_pdl(simt_dx_kernel<__nv_bfloat16>, grid, dim3(kSimtThreads), 0, stream,
                          (const __nv_bfloat16*)dY, (const __nv_bfloat16*)W, dy_rows, dx_rows, M_keep_dev, M, M_keep_cap,
                          (int)C_in, (int)C_out, (__nv_bfloat16*)dX, status_word);
    return launch_pdl(simt_dx_kernel<float>, grid, dim3(kSimtThreads), 0, stream,
                      (const float*)dY, (const float*)W, dy_rows, dx_rows, M_keep_dev, M, M_keep_cap,
                      (int)C_in, (int)C_out, (float*)dX, status_word);
}

}  // namespace sbp
