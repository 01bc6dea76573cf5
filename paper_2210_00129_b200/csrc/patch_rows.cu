// Convolutions with stride >= kernel size on the row-gather path (Sec. 3.2.2, the text after Eq. 6: with s >= k the
// neighbour effect disappears and the layer behaves like a point-wise one; ConvNeXt's 2 x 2 / stride 2 down-sampling
// layers are such layers).  Every output position reads its own k x k patch of the channels-last input, so the layer
// is a linear layer on "patch rows" of k * k * C values.  Two index kernels put that in front of and behind the
// linear-layer products:
//   patch cache:   X_keep[m, (dh, dw, c)] = X[b, s ho + dh, s wo + dw, c]   for the kept output positions m = (b, ho, wo):
//                  k contiguous pieces of k * C values per patch row (the forward cache of such a layer, Algorithm 1)
//   patch scatter: the packed input gradient [M_keep, k * k * C] back into dX [B, H, W, C]; every input position
//                  outside the kept patches (dropped positions, positions no patch covers when s > k) gets +0.0
// Both move 16-byte vectors and are HBM-bound.
#include "sbp_common.cuh"

namespace sbp {
namespace {

constexpr int kPatchThreads = 256;

struct PatchGeom {
    int H, W, Ho, Wo, k, s;
    uint32_t vec_c;                 // 16-byte vectors per input position (C * element size / 16)
};

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kPatchThreads)
patch_gather_kernel(const uint4* __restrict__ X, const PatchGeom g, const int32_t* __restrict__ keep_rows,
                    const int32_t* __restrict__ M_keep_dev, int64_t M_keep_cap, uint4* __restrict__ X_keep) {
    pdl_wait();
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const uint32_t vec_seg = (uint32_t)g.k * g.vec_c;                  // one piece: k positions of a row of the patch
    const uint32_t vec_row = (uint32_t)g.k * vec_seg;                  // one patch row
    const int64_t total = M_keep_cap * (int64_t)vec_row;
    const int64_t stride = (int64_t)gridDim.x * kPatchThreads;
    for (int64_t i = (int64_t)blockIdx.x * kPatchThreads + threadIdx.x; i < total; i += stride) {
        const int64_t m = i / vec_row;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);                          // rows past M_keep are cleared
        if (m < M_keep) {
            const uint32_t in_row = (uint32_t)(i - m * vec_row);
            const uint32_t dh = in_row / vec_seg, off = in_row - dh * vec_seg;
            const int64_t pos = __ldg(keep_rows + m);
            const int64_t b = pos / ((int64_t)g.Ho * g.Wo);
            const int rem = (int)(pos - b * (int64_t)g.Ho * g.Wo);
            const int ho = rem / g.Wo, wo = rem - ho * g.Wo;
            const int64_t pix = (b * g.H + (int64_t)g.s * ho + dh) * g.W + (int64_t)g.s * wo;
            v = ld_stream16(X + pix * g.vec_c + off);
        }
        X_keep[i] = v;
    }
    pdl_launch_dependents();
}

// slot[pos] = m for the kept output positions (the slots were set to -1 beforehand)
__global__ void patch_slots_kernel(const int32_t* __restrict__ keep_rows, const int32_t* __restrict__ M_keep_dev,
                                   int64_t M_keep_cap, int32_t* __restrict__ slot, const int32_t* status_word) {
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *reinterpret_cast<const volatile int32_t*>(status_word) != 0) return;
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    for (int64_t m = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; m < M_keep; m += (int64_t)gridDim.x * blockDim.x)
        slot[__ldg(keep_rows + m)] = (int32_t)m;
}

__global__ void __launch_bounds__(kPatchThreads)
patch_scatter_kernel(const uint4* __restrict__ dXp, const PatchGeom g, const int32_t* __restrict__ slot, int64_t positions,
                     uint4* __restrict__ dX, const int32_t* status_word) {
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *reinterpret_cast<const volatile int32_t*>(status_word) != 0) return;
    const int64_t total = positions * (int64_t)g.vec_c;               // every 16-byte vector of dX is written exactly once
    const uint32_t vec_seg = (uint32_t)g.k * g.vec_c, vec_row = (uint32_t)g.k * vec_seg;
    const int64_t stride = (int64_t)gridDim.x * kPatchThreads;
    for (int64_t i = (int64_t)blockIdx.x * kPatchThreads + threadIdx.x; i < total; i += stride) {
        const int64_t pix = i / g.vec_c;
        const uint32_t c = (uint32_t)(i - pix * g.vec_c);
        const int w = (int)(pix % g.W);
        const int64_t bh = pix / g.W;
        const int h = (int)(bh % g.H);
        const int64_t b = bh / g.H;
        const int ho = h / g.s, dh = h - ho * g.s, wo = w / g.s, dw = w - wo * g.s;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (dh < g.k && dw < g.k && ho < g.Ho && wo < g.Wo) {
            const int32_t m = __ldg(slot + (b * g.Ho + ho) * g.Wo + wo);
            if (m >= 0) v = ld_stream16(dXp + (int64_t)m * vec_row + (uint32_t)dh * vec_seg + (uint32_t)dw * g.vec_c + c);
        }
        dX[i] = v;
    }
}

PatchGeom geom(int64_t H, int64_t W, int64_t k, int64_t s, int64_t pos_bytes) {
    PatchGeom g;
    g.H = (int)H; g.W = (int)W; g.k = (int)k; g.s = (int)s;
    g.Ho = (int)((H - k) / s + 1); g.Wo = (int)((W - k) / s + 1);
    g.vec_c = (uint32_t)(pos_bytes / 16);
    return g;
}

unsigned blocks_for(int64_t vectors) {
    int64_t blocks = (vectors + kPatchThreads * 4 - 1) / (kPatchThreads * 4);
    if (blocks < 1) blocks = 1;
    if (blocks > (int64_t)kNumSMs * 16) blocks = (int64_t)kNumSMs * 16;
    return (unsigned)blocks;
}

}  // namespace

cudaError_t launch_patch_gather(const void* X, int64_t H, int64_t W, int64_t pos_bytes, int64_t k, int64_t s,
                                const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap, void* X_keep,
                                cudaStream_t stream) {
    const PatchGeom g = geom(H, W, k, s, pos_bytes);
    const int64_t total = M_keep_cap * k * k * (int64_t)g.vec_c;
    if (total == 0) return cudaSuccess;
    return launch_pdl(patch_gather_kernel, dim3(blocks_for(total)), dim3(kPatchThreads), 0, stream, (const uint4*)X, g, keep_rows,
                      M_keep_dev, M_keep_cap, (uint4*)X_keep);
}

cudaError_t launch_patch_scatter(const void* dXp, int64_t B, int64_t H, int64_t W, int64_t pos_bytes, int64_t k, int64_t s,
                                 const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap, void* dX,
                                 int32_t* slot, const int32_t* status_word, cudaStream_t stream) {
    const PatchGeom g = geom(H, W, k, s, pos_bytes);
    const int64_t outputs = B * (int64_t)g.Ho * g.Wo;
    cudaError_t e = cudaMemsetAsync(slot, 0xFF, (size_t)outputs * sizeof(int32_t), stream);     // every slot -1
    if (e != cudaSuccess) return e;
    int64_t blocks = (M_keep_cap + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > kNumSMs * 8) blocks = kNumSMs * 8;
    e = launch_pdl(patch_slots_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, keep_rows, M_keep_dev, M_keep_cap, slot, status_word);
    if (e != cudaSuccess) return e;
    const int64_t positions = B * H * W;
    return launch_pdl(patch_scatter_kernel, dim3(blocks_for(positions * g.vec_c)), dim3(kPatchThreads), 0, stream, (const uint4*)dXp, g,
                      (const int32_t*)slot, positions, (uint4*)dX, status_word);
}

}  // namespace sbp
