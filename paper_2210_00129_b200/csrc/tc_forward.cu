// bf16 tensor-core (tcgen05 / TMEM) forward of the layer, Y = X W + bias (Eq. 2), with the SBP
// forward cache written by the same kernel (Algorithm 1: every row is computed, only the kept rows of
// the input are retained): X_keep[m, :] = X[keep_rows[m], :].
//
//   tiles:  D[m, j] = sum_i X[m, i] * W[i, j]     A = X tile, K-major (TMA); B = W tile, MN-major (TMA,
//           64 x 64 boxes); the epilogue adds the bias, rounds to bf16 and writes whole rows.
//
// One persistent CTA per SM walks the 128 x BN output tiles (column tile fastest, so neighbouring CTAs
// share their rows of X through L2).  Warp roles: 0-3 epilogue (TMEM lane quadrants), 4 TMA producer,
// 5 MMA issuer and TMEM owner, 6-9 side warps, which copy the kept rows of X into the cache while the
// tensor pipe works - the rows are being streamed by the MMAs at about the same time, so DRAM sees X
// once.  Ring of four 48 KB stages behind full/empty mbarriers, two 256-column fp32 accumulators so
// the epilogue of one tile overlaps the MMAs of the next.  Every wait is bounded and reports through
// the status word.
#include "tc_ptx.cuh"

namespace sbp {
namespace {

constexpr int kFwdSideWarp0 = 6;
constexpr int kFwdSideThreads = 128;
constexpr int kFwdThreads = 32 * kFwdSideWarp0 + kFwdSideThreads;
constexpr int kBM = 128;                 // accumulator rows per tile (= TMEM lanes)
constexpr int kBK = 64;                  // reduction depth per stage: 64 bf16 = one 128-byte swizzle row
constexpr uint32_t kUmmaK = 16;
constexpr uint32_t kRowBytes = 128;
constexpr uint32_t kAtomBytes = 1024;
constexpr uint32_t kBlock64Bytes = 64 * kRowBytes;
constexpr int kStages = 4;
constexpr uint32_t kABytes = kBM * kRowBytes;        // 16 KB
constexpr uint32_t kBBytesMax = 256 * kRowBytes;     // 32 KB
constexpr uint32_t kStageBytes = kABytes + kBBytesMax;
constexpr uint32_t kAccCols = 256;
constexpr int kEpiBarrier = 2;
constexpr uint32_t kEpiBytes = 4 * 4096 + 2 * 256 * 4;   // one 4 KB transpose buffer per epilogue warp + two bias strips
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 256 + kEpiBytes + 1024;

struct FwdControl {
    uint64_t full_bar[kStages];    // 1 arrival carrying the byte count of both TMA operands
    uint64_t empty_bar[kStages];   // 1 arrival: tcgen05.commit of the MMAs that read the stage
    uint64_t acc_full[2];
    uint64_t acc_empty[2];         // 4 arrivals: each epilogue warp has read the accumulator out
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(FwdControl) <= 256, "control block");

struct FwdParams {
    const float* bias;             // nullable
    __nv_bfloat16* Y;
    int64_t M;
    int C_in, C_out;
    const uint4* X4;               // X as 16-byte vectors, for the cache
    uint4* Xk4;                    // nullptr: no cache requested
    const int32_t* keep_rows;
    const int32_t* M_keep_dev;
    int64_t M_keep_cap;
    int w_out_in;                  // W is [C_out, C_in]: the B tile is K-major and arrives as one TMA box
    int32_t* status_word;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <int BN>
__global__ void __launch_bounds__(kFwdThreads, 1)
tc_forward_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                  const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t ring = (raw_addr + 1023u) & ~1023u;
    FwdControl* ctl = reinterpret_cast<FwdControl*>(smem_raw + (ring - raw_addr) + kStages * kStageBytes);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_bar[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_bar[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[a]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[a]), 4);
        }
        ctl->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
    }
    if (warp == 5) ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_slot), 2 * kAccCols);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctl->tmem_slot);
    volatile int* abort_flag = &ctl->abort_flag;
    int32_t* status_word = p.status_word;

    pdl_wait();
    const bool skip_all = status_word != nullptr && *reinterpret_cast<volatile int32_t*>(status_word) != 0;
    const int C_in = p.C_in, C_out = p.C_out;
    const uint32_t ncol = (uint32_t)((C_out + BN - 1) / BN);
    const uint32_t total = (uint32_t)((p.M + kBM - 1) / kBM) * ncol;
    const uint32_t num_kb = (uint32_t)((C_in + kBK - 1) / kBK);

    if (skip_all) {
        // an earlier check failed: leave every output untouched
    } else if (warp == 4) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t q = blockIdx.x; q < total && ok; q += gridDim.x) {
                const int row0 = (int)((q / ncol) * kBM), n0 = (int)((q % ncol) * BN);
                for (uint32_t k = 0; k < num_kb; ++k, ++it) {
                    const int s = it % kStages;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / kStages) & 1u) ^ 1u, abort_flag, status_word);
                    if (!ok) break;
                    const uint32_t full = ptx::smem_addr(&ctl->full_bar[s]);
                    const uint32_t a_dst = ring + s * kStageBytes;
                    ptx::mbar_arrive_expect_tx(full, kABytes + BN * kRowBytes);
                    ptx::tma_load_2d(a_dst, &map_x, (int)(k * kBK), row0, full);                 // 128 rows x 64 columns of X
                    if (p.w_out_in) {                                                           // BN rows (j) x 64 columns (i) of W
                        ptx::tma_load_2d(a_dst + kABytes, &map_w, (int)(k * kBK), n0, full);
                    } else {
#pragma unroll
                        for (int b = 0; b < BN / 64; ++b)                                       // 64 rows (i) x 64 columns (j) of W
                            ptx::tma_load_2d(a_dst + kABytes + b * kBlock64Bytes, &map_w, n0 + b * 64, (int)(k * kBK), full);
                    }
                }
            }
            if (!ok) {   // let the copies already issued land before shared memory goes away
                for (uint32_t j = (it > (uint32_t)kStages ? it - kStages : 0u); j < it; ++j) {
                    const uint32_t bar = ptx::smem_addr(&ctl->full_bar[j % kStages]);
                    for (int spin = 0; spin < (1 << 14); ++spin)
                        if (ptx::mbar_try_wait(bar, (j / kStages) & 1u)) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t it = 0, used = 0;
            bool ok = true;
            // A K-major; B MN-major for W [C_in, C_out], K-major for W [C_out, C_in]
            const uint32_t idesc = ptx::umma_idesc_bf16(kBM, BN, false, p.w_out_in == 0);
            const uint32_t b_step = p.w_out_in ? kUmmaK * 2 : kUmmaK * kRowBytes, b_lbo = p.w_out_in ? 16u : kBlock64Bytes;
            for (uint32_t q = blockIdx.x; q < total && ok; q += gridDim.x, ++used) {
                const uint32_t acc = used & 1u;
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_empty[acc]), ((used >> 1) & 1u) ^ 1u, abort_flag, status_word);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                for (uint32_t k = 0; k < num_kb; ++k, ++it) {
                    const int s = it % kStages;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full_bar[s]), (it / kStages) & 1u, abort_flag, status_word);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = ring + s * kStageBytes, b_addr = a_addr + kABytes;
#pragma unroll
                    for (uint32_t u = 0; u < kBK / kUmmaK; ++u) {
                        // A: a 16-deep slice is 32 bytes along the swizzled row; B: 16 rows, 64-wide blocks 8 KB apart
                        const uint64_t da = ptx::umma_desc_sw128(a_addr + u * kUmmaK * 2, 16, kAtomBytes);
                        const uint64_t db = ptx::umma_desc_sw128(b_addr + u * b_step, b_lbo, kAtomBytes);
                        ptx::umma_bf16(d_tmem, da, db, idesc, (k | u) != 0u);
                    }
                    ptx::umma_commit(ptx::smem_addr(&ctl->empty_bar[s]));
                }
                if (ok) ptx::umma_commit(ptx::smem_addr(&ctl->acc_full[acc]));
            }
        }
        __syncwarp();
    } else if (warp >= kFwdSideWarp0) {
        // ---------------- side warps: the forward cache, X_keep[m, :] = X[keep_rows[m], :] ----------------
        if (p.Xk4 != nullptr) {
            const int64_t M_keep = load_m_keep(p.M_keep_dev, p.M_keep_cap);
            const int64_t vpr = C_in / 8;                                  // 16-byte vectors per row
            const int64_t all = p.M_keep_cap * vpr, valid = M_keep * vpr;
            const int64_t stride = (int64_t)gridDim.x * kFwdSideThreads;
            constexpr int kU = 16;                                        // 16-byte loads in flight per thread
            for (int64_t base = (int64_t)blockIdx.x * kFwdSideThreads + (threadIdx.x - kFwdSideWarp0 * 32); base < all;
                 base += stride * kU) {
                int64_t src[kU];
                uint4 v[kU];
#pragma unroll
                for (int u = 0; u < kU; ++u) {
                    const int64_t i = base + u * stride;
                    src[u] = -1;
                    if (i < valid) {
                        const int64_t m = i / vpr;
                        src[u] = (int64_t)__ldg(p.keep_rows + m) * vpr + (i - m * vpr);
                    }
                }
#pragma unroll
                for (int u = 0; u < kU; ++u) v[u] = (src[u] >= 0) ? __ldg(p.X4 + src[u]) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int u = 0; u < kU; ++u) {
                    const int64_t i = base + u * stride;
                    if (i < all) p.Xk4[i] = v[u];                         // rows past M_keep are cleared
                }
            }
        }
    } else {
        // ---------------- epilogue warps ----------------
        uint32_t used = 0;
        bool ok = true;
        uint8_t* wbuf = smem_raw + (ring - raw_addr) + kStages * kStageBytes + 256 + warp * 4096;
        const int sub = lane >> 3, ch = lane & 7;
        int staged_n0[2] = {-1, -1};
        for (uint32_t q = blockIdx.x; q < total; q += gridDim.x, ++used) {
            const uint32_t acc = used & 1u;
            const uint32_t taddr = tmem_base + acc * kAccCols + ((uint32_t)(warp * 32) << 16);
            const int64_t m0 = (int64_t)(q / ncol) * kBM + warp * 32;
            const int n0 = (int)((q % ncol) * BN);
            const int strip_cols = (C_out - n0 < BN) ? C_out - n0 : BN;     // multiple of 8
            // The tile's strip of the bias goes to shared memory first (two buffers, by tile parity): read from
            // global memory inside the loop below, its 64 dependent loads per tile doubled the kernel's time.
            float* bias_s = reinterpret_cast<float*>(smem_raw + (ring - raw_addr) + kStages * kStageBytes + 256 + 4 * 4096) +
                            (used & 1u) * 256;
            if (p.bias != nullptr && staged_n0[used & 1u] != n0) {        // with one or two column tiles the strip never changes
                for (int c = threadIdx.x; c < BN; c += 128) bias_s[c] = (n0 + c < C_out) ? __ldg(p.bias + n0 + c) : 0.f;
                staged_n0[used & 1u] = n0;
            }
            if (lane == 0) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[acc]), (used >> 1) & 1u, abort_flag, status_word);
            ok = !ptx::bar_or<kEpiBarrier, 128>(!ok);                      // the four warps go on, or give up, together
            if (!ok) break;
            ptx::tc_fence_after_sync();
            // a lane holds one row of the accumulator; 64 columns at a time go through the warp's swizzled
            // 4 KB buffer so that every store instruction writes four rows x 128 contiguous bytes
            float va[32], vb[32];
            ptx::tmem_ld_32x32(taddr, va);
            ptx::tmem_ld_32x32(taddr + 32u, vb);
#pragma unroll 1
            for (int c0 = 0; c0 < strip_cols; c0 += 64) {
                ptx::tmem_ld_wait();
#pragma unroll
                for (int qd = 0; qd < 8; ++qd) {
                    float* f = (qd < 4) ? &va[qd * 8] : &vb[(qd - 4) * 8];
                    if (p.bias != nullptr) {
                        const float4 b0 = *reinterpret_cast<const float4*>(bias_s + c0 + qd * 8);
                        const float4 b1 = *reinterpret_cast<const float4*>(bias_s + c0 + qd * 8 + 4);
                        f[0] += b0.x; f[1] += b0.y; f[2] += b0.z; f[3] += b0.w;
                        f[4] += b1.x; f[5] += b1.y; f[6] += b1.z; f[7] += b1.w;
                    }
                    *reinterpret_cast<uint4*>(wbuf + lane * 128 + ((qd ^ (lane & 7)) << 4)) =
                        make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
                }
                __syncwarp();
                if (c0 + 64 < strip_cols) {
                    ptx::tmem_ld_32x32(taddr + (uint32_t)(c0 + 64), va);
                    ptx::tmem_ld_32x32(taddr + (uint32_t)(c0 + 96), vb);
                }
                const bool col_ok = c0 + ch * 8 < strip_cols;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = i * 4 + sub;
                    const uint4 pk = *reinterpret_cast<const uint4*>(wbuf + r * 128 + ((ch ^ (r & 7)) << 4));
                    if (m0 + r < p.M && col_ok)
                        ptx::st_global_v4(p.Y + (m0 + r) * C_out + n0 + c0 + ch * 8, pk.x, pk.y, pk.z, pk.w);
                }
                __syncwarp();
            }
            ptx::tc_fence_before_sync();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->acc_empty[acc]));
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 2 * kAccCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 row-major [rows, cols] matrix, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
cudaError_t launch_forward(dim3 grid, cudaStream_t stream, const CUtensorMap& map_x, const CUtensorMap& map_w,
                           const FwdParams& prm) {
    const cudaError_t opt = opt_in_dynamic_smem<tc_forward_kernel<BN>>((int)kSmemBytes);
    if (opt != cudaSuccess) return opt;
    return launch_pdl(tc_forward_kernel<BN>, grid, dim3(kFwdThreads), kSmemBytes, stream, map_x, map_w, prm);
}

}  // namespace

bool tc_forward_supported(int64_t M, int64_t C_in, int64_t C_out) {
    // every TMA box (64 columns x 64 or 128 rows) must fit inside its matrix
    return M >= kBM && M < (1ll << 31) && C_in >= 128 && C_out >= 128 && C_in % 8 == 0 && C_out % 8 == 0;
}

sbp_status launch_tc_forward(const void* X, const void* W, bool w_out_in, const float* bias, int64_t M, int64_t C_in, int64_t C_out,
                             void* Y, const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap,
                             void* X_keep, int32_t* status_word, cudaStream_t stream) {
    CUtensorMap map_x, map_w;
    const int bn = C_out >= 256 ? 256 : 128;
    if (!make_map(&map_x, X, M, C_in, (uint32_t)kBM)) return SBP_ERR_CUDA;
    if (w_out_in ? !make_map(&map_w, W, C_out, C_in, (uint32_t)bn) : !make_map(&map_w, W, C_in, C_out, 64u)) return SBP_ERR_CUDA;
    FwdParams prm;
    prm.w_out_in = w_out_in ? 1 : 0;
    prm.bias = bias;
    prm.Y = static_cast<__nv_bfloat16*>(Y);
    prm.M = M;
    prm.C_in = (int)C_in;
    prm.C_out = (int)C_out;
    prm.X4 = static_cast<const uint4*>(X);
    prm.Xk4 = static_cast<uint4*>(X_keep);
    prm.keep_rows = keep_rows;
    prm.M_keep_dev = M_keep_dev;
    prm.M_keep_cap = M_keep_cap;
    prm.status_word = status_word;
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((C_out + bn - 1) / bn);
    const dim3 grid((unsigned)(tiles < kNumSMs ? tiles : kNumSMs));
    const cudaError_t e = bn == 256 ? launch_forward<256>(grid, stream, map_x, map_w, prm)
                                    : launch_forward<128>(grid, stream, map_x, map_w, prm);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

}  // namespace sbp
