// Bias gradient db[j] = sum over kept rows of dY[keep_rows[m], j] (the bias term follows the
// same masking of dY as Eq. 5), and the deterministic reduction of split partial results.
//
// db: each block owns a strip of 32 16-byte column vectors and a contiguous share of the kept
// rows; a warp reads one gathered row strip as 32 x 16-byte vectors (coalesced, 512 B), keeps
// eight such loads in flight, the eight warps of a block take different rows, partial sums are
// combined through shared memory in a fixed order and written to a [splits, C_out] scratch that
// a second kernel adds up, again in a fixed order.  HBM-bound: one read of the kept rows of dY.
#include "sbp_common.cuh"

namespace sbp {
namespace {

constexpr int kDbThreads = 256;
constexpr int kDbWarps = kDbThreads / 32;
constexpr int kDbUnroll = 8;
constexpr int kDbTargetBlocks = 4 * kNumSMs;

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

inline int db_splits(int64_t M_keep_cap, int64_t col_vecs, int max_splits) {
    const int64_t strips = (col_vecs + 31) / 32;
    int64_t s = (kDbTargetBlocks + strips - 1) / strips;
    const int64_t by_rows = (M_keep_cap + 63) / 64;        // at least 64 rows per block
    if (s > by_rows) s = by_rows;
    if (s > max_splits) s = max_splits;
    if (s < 1) s = 1;
    return (int)s;
}

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <typename T>
__global__ void __launch_bounds__(kDbThreads)
db_partial_kernel(const uint4* __restrict__ dY, uint32_t col_vecs, const int32_t* __restrict__ keep_rows,
                  const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap, float* __restrict__ partials,
                  const int32_t* __restrict__ status_word) {
    constexpr int E = Vec16<T>::kElems;
    __shared__ float red[kDbWarps][32 * E];
    pdl_launch_dependents();
    pdl_wait();
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
            int64_t row[kDbUnroll];
            uint4 v[kDbUnroll];
#pragma unroll
            for (int u = 0; u < kDbUnroll; ++u) {
                const int64_t mm = m + u * kDbWarps;
                row[u] = (mm < m_end) ? (int64_t)mapped_row(keep_rows, mm) : -1;
            }
#pragma unroll
            for (int u = 0; u < kDbUnroll; ++u)
                v[u] = (row[u] >= 0) ? ld_stream16(dY + row[u] * col_vecs + cv) : make_uint4(0u, 0u, 0u, 0u);
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

// ---- deterministic reduction of [splits, n] partial results ------------------------------------
// One launch serves up to two reductions (the split partials of dW and the per-block partials of
// db of one backward call): the first a.blocks blocks work on job a, the rest on job b.
struct ReduceJob {
    const float4* partials;
    float4* out;
    int64_t n_vec;        // float4 elements per partial
    int splits;
    int accumulate;
    int lanes;            // 1: one thread per float4, partials added in ascending order
                          // Y = 4 or 32: 256/Y float4 columns x Y row lanes per block; lane y adds partials
                          //    y, y+Y, ... in ascending order, the Y lane sums are then added in lane order
    int blocks;
};

__device__ __forceinline__ void add4(float4& s, const float4& p) { s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w; }

__device__ __forceinline__ void run_reduce_job(const ReduceJob& jb, int block, float4* red) {
    if (jb.lanes == 1) {
        const int64_t stride = (int64_t)jb.blocks * blockDim.x;
        for (int64_t i = (int64_t)block * blockDim.x + threadIdx.x; i < jb.n_vec; i += stride) {
            float4 s = jb.accumulate ? jb.out[i] : make_float4(0.f, 0.f, 0.f, 0.f);
            for (int k0 = 0; k0 < jb.splits; k0 += 4) {           // four independent loads in flight
                float4 p[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    p[u] = (k0 + u < jb.splits) ? __ldg(jb.partials + (int64_t)(k0 + u) * jb.n_vec + i)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (k0 + u < jb.splits) add4(s, p[u]);
            }
            jb.out[i] = s;
        }
        return;
    }
    const int Y = jb.lanes, X = 256 / Y;
    const int x = threadIdx.x % X, y = threadIdx.x / X;
    const int64_t i = (int64_t)block * X + x;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < jb.n_vec) {
        for (int k0 = y; k0 < jb.splits; k0 += Y * 4) {
            float4 p[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                p[u] = (k0 + Y * u < jb.splits) ? __ldg(jb.partials + (int64_t)(k0 + Y * u) * jb.n_vec + i)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (k0 + Y * u < jb.splits) add4(s, p[u]);
        }
    }
    red[y * X + x] = s;
    __syncthreads();
    if (y == 0 && i < jb.n_vec) {
        float4 t = jb.accumulate ? jb.out[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        for (int w = 0; w < Y; ++w) add4(t, red[w * X + x]);
        jb.out[i] = t;
    }
}

__global__ void __launch_bounds__(256)
reduce_partials_kernel(const ReduceJob a, const ReduceJob b, const int32_t* __restrict__ status_word) {
    __shared__ float4 red[256];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *status_word != 0) return;
    if ((int)blockIdx.x < a.blocks) run_reduce_job(a, (int)blockIdx.x, red);
    else run_reduce_job(b, (int)blockIdx.x - a.blocks, red);
}

ReduceJob make_reduce_job(const float* partials, int splits, int64_t n, float* out, bool accumulate) {
    ReduceJob jb;
    jb.partials = reinterpret_cast<const float4*>(partials);
    jb.out = reinterpret_cast<float4*>(out);
    jb.n_vec = n / 4;             // n is a multiple of 4 for every caller
    jb.splits = splits;
    jb.accumulate = accumulate ? 1 : 0;
    // few partials: one thread per element; many partials of a short vector (db): 32 lanes per column;
    // many partials of a long one (dW): 4 lanes per column
    jb.lanes = splits <= 8 ? 1 : (jb.n_vec <= 8192 ? 32 : 4);
    int64_t blocks;
    if (jb.lanes > 1) {
        const int64_t cols = 256 / jb.lanes;
        blocks = (jb.n_vec + cols - 1) / cols;
    } else {
        blocks = (jb.n_vec + 255) / 256;
        if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
    }
    jb.blocks = (int)(blocks < 1 ? 1 : blocks);
    return jb;
}

}  // namespace

size_t db_workspace_bytes(sbp_dtype dt, int64_t M_keep_cap, int64_t C_out, int max_splits) {
    const int64_t col_vecs = C_out / ((dt == SBP_BF16) ? 8 : 4);
    return (size_t)db_splits(M_keep_cap, col_vecs, max_splits) * (size_t)C_out * sizeof(float);
}

cudaError_t launch_db(sbp_dtype dt, const void* dY, const int32_t* keep_rows, const int32_t* M_keep_dev,
                      int64_t M_keep_cap, int64_t C_out, float* db, bool accumulate, float* workspace,
                      int max_splits, const int32_t* status_word, cudaStream_t stream) {
    const int64_t elems = (dt == SBP_BF16) ? 8 : 4;
    const int64_t col_vecs = C_out / elems;
    const int splits = db_splits(M_keep_cap, col_vecs, max_splits);
    const dim3 grid((unsigned)((col_vecs + 31) / 32), (unsigned)splits);
    cudaError_t e;
    if (dt == SBP_BF16)
        e = launch_pdl(db_partial_kernel<__nv_bfloat16>, grid, dim3(kDbThreads), 0, stream,
                       (const uint4*)dY, (uint32_t)col_vecs, keep_rows, M_keep_dev, M_keep_cap, workspace, status_word);
    else
        e = launch_pdl(db_partial_kernel<float>, grid, dim3(kDbThreads), 0, stream,
                       (const uint4*)dY, (uint32_t)col_vecs, keep_rows, M_keep_dev, M_keep_cap, workspace, status_word);
    if (e != cudaSuccess) return e;
    return launch_reduce_partials(workspace, splits, C_out, db, accumulate, status_word, stream);
}

cudaError_t launch_reduce_partials(const float* partials, int splits, int64_t n, float* out,
                                   bool accumulate, const int32_t* status_word, cudaStream_t stream) {
    const ReduceJob a = make_reduce_job(partials, splits, n, out, accumulate);
    ReduceJob none = a;
    none.blocks = 0;
    return launch_pdl(reduce_partials_kernel, dim3((unsigned)a.blocks), dim3(256), 0, stream, a, none, status_word);
}

cudaError_t launch_reduce_partials_pair(const float* partials_a, int splits_a, int64_t n_a, float* out_a,
                                        const float* partials_b, int splits_b, int64_t n_b, float* out_b,
                                        bool accumulate, const int32_t* status_word, cudaStream_t stream) {
    const ReduceJob a = make_reduce_job(partials_a, splits_a, n_a, out_a, accumulate);
    const ReduceJob b = make_reduce_job(partials_b, splits_b, n_b, out_b, accumulate);
    return launch_pdl(reduce_partials_kernel, dim3((unsigned)(a.blocks + b.blocks)), dim3(256), 0, stream, a, b,
                      status_word);
}

}  // namespace sbp
