// bf16 tensor-core (tcgen05 / TMEM) kernels for the two products of the SBP linear backward (Eq. 5).
//
//   dX kernel:  D[m, i] = sum_j dY[keep_rows[m], j] * W[i, j]            (both operands K-major)
//               A = kept rows of dY, gathered straight from the full dY; B = W tile (TMA);
//               the epilogue rounds to bf16, scatters each row to dX[keep_rows[m], :] and
//               zero-fills the dropped rows between kept rows while the MMAs run.
//   dW kernel:  D[i, j] = sum_m X_keep[m, i] * dY[keep_rows[m], j]       (both operands MN-major)
//               A = X_keep tile (TMA), B = gathered dY rows; the reduction over kept rows is
//               split across blockIdx.z, partials reduced in a fixed order.
//
// One CTA computes a 128 x BN fp32 accumulator tile held in tensor memory.  Warp roles:
// warps 0-3 epilogue (TMEM lane quadrant = warp id), warp 4 TMA producer of the dense operand,
// warp 5 MMA issuer and TMEM owner, warps 6-9 gather producers: they copy the indexed rows of dY
// with coalesced 16-byte cp.async into the 128-byte-swizzled layout the MMA reads; each thread's
// copies signal the stage's barrier when they land (cp.async.mbarrier.arrive), so the producers run
// a full ring ahead of the consumer without ever waiting on their own copies.  (TMA tile::gather4
// was measured at ~45 ns of issue time per instruction per SM whatever it fetches, far too slow
// to feed a tile.)  Operand stages are 64 elements deep
// in the reduction dimension and cycle through a full/empty mbarrier ring.  Every wait is bounded.
#include "tc_ptx.cuh"

namespace sbp {
namespace {

constexpr int kTcThreads = 320;
constexpr int kGatherWarp0 = 6;          // first of the four gather warps
constexpr int kGatherThreads = 128;
constexpr int kBM = 128;                 // accumulator rows per CTA (= TMEM lanes)
constexpr int kBK = 64;                  // reduction depth per stage: 64 bf16 = one 128-byte swizzle row
constexpr uint32_t kUmmaK = 16;          // reduction depth of one tcgen05.mma for 16-bit operands
constexpr uint32_t kRowBytes = 128;      // bytes per swizzled smem row
constexpr uint32_t kAtomBytes = 1024;    // 8 rows x 128 B: one swizzle atom
constexpr uint32_t kBlock64Bytes = 64 * kRowBytes;   // a 64-row slab (MN-major operands: one 64-wide block)

template <int BN>
struct TcCfg {
    static constexpr uint32_t kABytes = kBM * kRowBytes;          // 16 KB
    static constexpr uint32_t kBBytes = BN * kRowBytes;           // 16 / 32 KB
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = (BN == 256) ? 4 : 6;
    static constexpr uint32_t kCtlBytes = 256;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + kCtlBytes + 1024;   // + alignment slack
};

struct TcControl {
    uint64_t full_bar[8];      // 1 arrival with the TMA byte count + one arrival per gather thread
    uint64_t empty_bar[8];     // 1 arrival: tcgen05.commit of the MMAs that read the stage
    uint64_t accum_bar;        // 1 arrival: all MMAs of the tile have finished
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(TcControl) <= 256, "control block");

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// position of 16-byte chunk `chunk` of row `row` inside a 128-byte-swizzled slab
__device__ __forceinline__ uint32_t swizzled(uint32_t row, uint32_t chunk) {
    return row * kRowBytes + ((chunk ^ (row & 7u)) << 4);
}

template <int BN>
__device__ __forceinline__ void init_pipeline(TcControl* ctl) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < TcCfg<BN>::kStages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_bar[s]), 1 + kGatherThreads);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_bar[s]), 1);
        }
        ptx::mbar_init(ptx::smem_addr(&ctl->accum_bar), 1);
        ctl->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if ((threadIdx.x >> 5) == 5) ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_slot), BN);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
}

// TMA thread after a failed wait: let the copies it already issued land before shared memory goes away
template <int STAGES>
__device__ __forceinline__ void drain_tma(TcControl* ctl, uint32_t issued) {
    for (uint32_t it = (issued > (uint32_t)STAGES ? issued - STAGES : 0u); it < issued; ++it) {
        const uint32_t bar = ptx::smem_addr(&ctl->full_bar[it % STAGES]);
        for (int spin = 0; spin < (1 << 14); ++spin)
            if (ptx::mbar_try_wait(bar, (it / STAGES) & 1u)) break;
    }
}

// The MMA issuer's loop is the same for both kernels up to the operand descriptors.
template <int BN, bool MN_MAJOR>
__device__ __forceinline__ void mma_loop(TcControl* ctl, uint32_t tiles, uint32_t tmem_base, uint32_t num_kb,
                                         volatile int* abort_flag, int32_t* status_word) {
    using Cfg = TcCfg<BN>;
    constexpr uint32_t idesc = ptx::umma_idesc_bf16(kBM, BN, MN_MAJOR, MN_MAJOR);
    // K-major: a 16-deep slice is 32 bytes along the swizzled row; 8-row groups sit 1024 B apart.
    // MN-major: a 16-deep slice is 16 rows (two atoms); 64-wide blocks of the MN extent sit 8 KB apart.
    constexpr uint32_t k_step = MN_MAJOR ? kUmmaK * kRowBytes : kUmmaK * 2;
    constexpr uint32_t lbo = MN_MAJOR ? kBlock64Bytes : 16;
    bool ok = true;
    for (uint32_t it = 0; it < num_kb; ++it) {
        const int s = it % Cfg::kStages;
        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full_bar[s]), (it / Cfg::kStages) & 1u, abort_flag, status_word);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        ptx::fence_async_proxy();        // the gathered operand was written by cp.async (generic proxy)
        const uint32_t a_addr = tiles + s * Cfg::kStageBytes, b_addr = a_addr + Cfg::kABytes;
#pragma unroll
        for (uint32_t k = 0; k < kBK / kUmmaK; ++k) {
            const uint64_t da = ptx::umma_desc_sw128(a_addr + k * k_step, lbo, kAtomBytes);
            const uint64_t db = ptx::umma_desc_sw128(b_addr + k * k_step, lbo, kAtomBytes);
            ptx::umma_bf16(tmem_base, da, db, idesc, (it | k) != 0u);
        }
        ptx::umma_commit(ptx::smem_addr(&ctl->empty_bar[s]));     // stage reusable once these MMAs retire
    }
    if (ok) ptx::umma_commit(ptx::smem_addr(&ctl->accum_bar));
}

// --------------------------------------------------------------------------------------------
// dX = scatter(dY_keep * W^T) with zero fill
// --------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_dx_kernel(const __grid_constant__ CUtensorMap map_w, const __nv_bfloat16* __restrict__ dY,
             const int32_t* __restrict__ keep_rows, const int32_t* __restrict__ M_keep_dev,
             int64_t M, int64_t M_keep_cap, int C_in, int C_out,
             __nv_bfloat16* __restrict__ dX, int32_t* status_word) {
    using Cfg = TcCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *reinterpret_cast<volatile int32_t*>(status_word) != 0) return;
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t m0 = (int64_t)blockIdx.x * kBM;
    const int n0 = blockIdx.y * BN;
    const int strip_cols = (C_in - n0 < BN) ? C_in - n0 : BN;       // multiple of 8
    const int strip_vecs = strip_cols >> 3;                          // 16-byte vectors per row of the strip

    if (M_keep == 0) {                   // nothing kept: the first row tile clears its column strip
        if (blockIdx.x == 0)
            for (int64_t t = threadIdx.x; t < M * strip_vecs; t += kTcThreads)
                ptx::st_global_v4(dX + (t / strip_vecs) * C_in + n0 + (t % strip_vecs) * 8, 0u, 0u, 0u, 0u);
        return;
    }
    if (m0 >= M_keep) return;

    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t tiles = (raw_addr + 1023u) & ~1023u;             // swizzle atoms need 1024-byte alignment
    TcControl* ctl = reinterpret_cast<TcControl*>(smem_raw + (tiles - raw_addr) + Cfg::kStages * Cfg::kStageBytes);
    const uint32_t num_kb = (uint32_t)((C_out + kBK - 1) / kBK);
    init_pipeline<BN>(ctl);
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctl->tmem_slot);
    volatile int* abort_flag = &ctl->abort_flag;

    if (warp == 4) {
        // ---------------- TMA producer: the W tile of every stage ----------------
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_w);
            uint32_t it = 0;
            for (; it < num_kb; ++it) {
                const int s = it % Cfg::kStages;
                if (!ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / Cfg::kStages) & 1u) ^ 1u, abort_flag, status_word))
                    break;
                const uint32_t full = ptx::smem_addr(&ctl->full_bar[s]);
                ptx::mbar_arrive_expect_tx(full, Cfg::kBBytes);
                ptx::tma_load_2d(tiles + s * Cfg::kStageBytes + Cfg::kABytes, &map_w, (int)(it * kBK), n0, full);
            }
            if (it < num_kb) drain_tma<Cfg::kStages>(ctl, it);
        }
        __syncwarp();
    } else if (warp == 5) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) mma_loop<BN, false>(ctl, tiles, tmem_base, num_kb, abort_flag, status_word);
        __syncwarp();
    } else if (warp >= kGatherWarp0) {
        // ---------------- gather producers: 128 kept rows x 128 bytes of dY per stage ----------------
        // one instruction of a warp moves 4 rows x 128 B; a warp owns 32 rows of the tile
        const int gw = warp - kGatherWarp0;
        const uint32_t chunk = lane & 7;
        const __nv_bfloat16* src[8];
        uint32_t dst[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t row = gw * 32 + i * 4 + (lane >> 3);
            int64_t m = m0 + row;
            if (m >= M_keep) m = M_keep - 1;                          // padding rows of the last tile: never stored
            src[i] = dY + (int64_t)__ldg(keep_rows + m) * C_out + chunk * 8;
            dst[i] = swizzled(row, chunk);
        }
        for (uint32_t it = 0; it < num_kb; ++it) {
            const int s = it % Cfg::kStages;
            if (!ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / Cfg::kStages) & 1u) ^ 1u, abort_flag, status_word))
                break;
            const uint32_t a_dst = tiles + s * Cfg::kStageBytes;
            const int col = (int)(it * kBK + chunk * 8);
            const uint32_t bytes = (col < C_out) ? 16u : 0u;      // columns past C_out read as zero
            const int off = (col < C_out) ? (int)(it * kBK) : 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) ptx::cp_async_16(a_dst + dst[i], src[i] + off, bytes);
            // the stage's barrier gets this thread's arrival when the copies above have landed
            ptx::cp_async_arrive_noinc(ptx::smem_addr(&ctl->full_bar[s]));
        }
        ptx::cp_async_wait_all();
    } else {
        // ---------------- epilogue warps: zero fill first, then scatter the accumulator rows ----------------
        const int64_t m = m0 + warp * 32 + lane;
        const bool valid = m < M_keep;
        const int64_t cur = valid ? (int64_t)__ldg(keep_rows + m) : -1;
        const int64_t prev = (valid && m > 0) ? (int64_t)__ldg(keep_rows + m - 1) : -1;
        for (int t = 0; t < 32; ++t) {
            if (!__shfl_sync(0xffffffffu, valid ? 1 : 0, t)) break;
            const int64_t c = __shfl_sync(0xffffffffu, cur, t);
            int64_t g = __shfl_sync(0xffffffffu, prev, t) + 1;
            for (; g < c; ++g)
                for (int v = lane; v < strip_vecs; v += 32)
                    ptx::st_global_v4(dX + g * C_in + n0 + v * 8, 0u, 0u, 0u, 0u);
            if (m0 + warp * 32 + t == M_keep - 1)                   // after the very last kept row
                for (g = c + 1; g < M; ++g)
                    for (int v = lane; v < strip_vecs; v += 32)
                        ptx::st_global_v4(dX + g * C_in + n0 + v * 8, 0u, 0u, 0u, 0u);
        }
        bool ok = true;
        if (lane == 0) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->accum_bar), 0u, abort_flag, status_word);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (ok) {
            ptx::tc_fence_after_sync();
            __nv_bfloat16* out_row = dX + (valid ? cur : 0) * C_in + n0;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                float v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (valid) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (c0 + q * 8 < strip_cols)
                            ptx::st_global_v4(out_row + c0 + q * 8,
                                              pack_bf16(v[q * 8 + 0], v[q * 8 + 1]), pack_bf16(v[q * 8 + 2], v[q * 8 + 3]),
                                              pack_bf16(v[q * 8 + 4], v[q * 8 + 5]), pack_bf16(v[q * 8 + 6], v[q * 8 + 7]));
                    }
                }
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, BN);
    }
}

// --------------------------------------------------------------------------------------------
// dW = X_keep^T * dY_keep, split over the kept rows
// --------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_dw_kernel(const __grid_constant__ CUtensorMap map_x, const __nv_bfloat16* __restrict__ dY,
             const int32_t* __restrict__ keep_rows, const int32_t* __restrict__ M_keep_dev,
             int64_t M_keep_cap, int C_in, int C_out, float* __restrict__ out, int64_t split_stride,
             int accumulate, int32_t* status_word) {
    using Cfg = TcCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    pdl_launch_dependents();
    pdl_wait();
    if (status_word != nullptr && *reinterpret_cast<volatile int32_t*>(status_word) != 0) return;
    const int64_t M_keep = load_m_keep(M_keep_dev, M_keep_cap);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j0 = blockIdx.x * BN, i0 = blockIdx.y * kBM;
    const uint32_t total_kb = (uint32_t)((M_keep + kBK - 1) / kBK);
    const uint32_t kb_per = (total_kb + gridDim.z - 1) / gridDim.z;
    const uint32_t kb_begin = kb_per * blockIdx.z;
    const uint32_t kb_end = (kb_begin + kb_per < total_kb) ? kb_begin + kb_per : total_kb;
    const uint32_t num_kb = (kb_end > kb_begin) ? kb_end - kb_begin : 0u;
    float* dst_base = out + (int64_t)blockIdx.z * split_stride;

    if (num_kb == 0) {                   // this split has no kept rows: its partial is zero
        if (!accumulate)
            for (int t = threadIdx.x; t < kBM * (BN / 4); t += kTcThreads) {
                const int i = i0 + t / (BN / 4), j = j0 + (t % (BN / 4)) * 4;
                if (i < C_in && j < C_out) ptx::st_global_v4(dst_base + (int64_t)i * C_out + j, 0u, 0u, 0u, 0u);
            }
        return;
    }

    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t tiles = (raw_addr + 1023u) & ~1023u;
    TcControl* ctl = reinterpret_cast<TcControl*>(smem_raw + (tiles - raw_addr) + Cfg::kStages * Cfg::kStageBytes);
    init_pipeline<BN>(ctl);
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctl->tmem_slot);
    volatile int* abort_flag = &ctl->abort_flag;

    if (warp == 4) {
        // ---------------- TMA producer: the X_keep tile (two 64-wide blocks) of every stage ----------------
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_x);
            uint32_t it = 0;
            for (; it < num_kb; ++it) {
                const int s = it % Cfg::kStages;
                if (!ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / Cfg::kStages) & 1u) ^ 1u, abort_flag, status_word))
                    break;
                const uint32_t full = ptx::smem_addr(&ctl->full_bar[s]);
                const uint32_t a_dst = tiles + s * Cfg::kStageBytes;
                const int row0 = (int)((kb_begin + it) * kBK);
                ptx::mbar_arrive_expect_tx(full, Cfg::kABytes);
                ptx::tma_load_2d(a_dst, &map_x, i0, row0, full);
                ptx::tma_load_2d(a_dst + kBlock64Bytes, &map_x, i0 + 64, row0, full);
            }
            if (it < num_kb) drain_tma<Cfg::kStages>(ctl, it);
        }
        __syncwarp();
    } else if (warp == 5) {
        // ---------------- MMA issuer: both operands MN-major ----------------
        if (lane == 0) mma_loop<BN, true>(ctl, tiles, tmem_base, num_kb, abort_flag, status_word);
        __syncwarp();
    } else if (warp >= kGatherWarp0) {
        // ---------------- gather producers: 64 kept rows x BN columns of dY per stage ----------------
        // a warp owns 16 rows of each stage; one instruction moves 512 contiguous bytes
        constexpr int kChunksPerRow = BN / 8;                   // 16-byte chunks of one row of the tile
        constexpr int kRowsPerInstr = 32 / kChunksPerRow;       // 1 (BN = 256) or 2 (BN = 128)
        constexpr int kInstr = 16 / kRowsPerInstr;
        const int gw = warp - kGatherWarp0;
        const uint32_t c = lane % kChunksPerRow;                // chunk within the row
        const uint32_t sub = lane / kChunksPerRow;              // which of the rows of this instruction
        const int col = j0 + (int)c * 8;
        const bool col_ok = col < C_out;                        // columns past C_out read as zero
        const __nv_bfloat16* col_ptr = dY + (col_ok ? col : 0);
        for (uint32_t it = 0; it < num_kb; ++it) {
            const int s = it % Cfg::kStages;
            // row ids of this warp's 16 rows: lanes 0..15 fetch one each
            const int64_t mrow = (int64_t)(kb_begin + it) * kBK + gw * 16 + (lane & 15);
            const int my_row = (mrow < M_keep) ? __ldg(keep_rows + mrow) : -1;
            bool ok = ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / Cfg::kStages) & 1u) ^ 1u, abort_flag, status_word);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t b_dst = tiles + s * Cfg::kStageBytes + Cfg::kABytes;
#pragma unroll
            for (int i = 0; i < kInstr; ++i) {
                const uint32_t r = gw * 16 + i * kRowsPerInstr + sub;             // row within the 64-row stage
                const int g = __shfl_sync(0xffffffffu, my_row, i * kRowsPerInstr + (int)sub);
                const bool live = g >= 0 && col_ok;                               // rows past M_keep read as zero
                ptx::cp_async_16(b_dst + (c >> 3) * kBlock64Bytes + swizzled(r, c & 7u),
                                 col_ptr + (live ? (int64_t)g * C_out : 0), live ? 16u : 0u);
            }
            ptx::cp_async_arrive_noinc(ptx::smem_addr(&ctl->full_bar[s]));
        }
        ptx::cp_async_wait_all();
    } else {
        // ---------------- epilogue: fp32 accumulator rows to dW (or to this split's partial) ----------------
        bool ok = true;
        if (lane == 0) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->accum_bar), 0u, abort_flag, status_word);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (ok) {
            ptx::tc_fence_after_sync();
            const int i = i0 + warp * 32 + lane;
            float* out_row = dst_base + (int64_t)i * C_out + j0;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                float v[32];
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                ptx::tmem_ld_wait();
                if (i < C_in) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (j0 + c0 + q * 4 < C_out) {
                            float4 w = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
                            float4* p = reinterpret_cast<float4*>(out_row + c0 + q * 4);
                            if (accumulate) { const float4 o = *p; w.x += o.x; w.y += o.y; w.z += o.z; w.w += o.w; }
                            *p = w;
                        }
                    }
                }
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, BN);
    }
}

// --------------------------------------------------------------------------------------------
// host side: tensor maps and launches
// --------------------------------------------------------------------------------------------
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

template <typename K>
cudaError_t allow_smem(K kernel, uint32_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

struct DwPlan { int bn; int splits; };

DwPlan plan_dw(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    DwPlan p;
    p.bn = (C_out >= 256) ? 256 : 128;
    const int64_t tiles = ((C_in + kBM - 1) / kBM) * ((C_out + p.bn - 1) / p.bn);
    const int64_t kb = (M_keep_cap + kBK - 1) / kBK;
    // fill the 148 SMs once: as many splits as fit in one wave, each at least 4 stages deep
    int64_t s = kNumSMs / tiles;
    if (s > kb / 4) s = kb / 4;
    if (s > 32) s = 32;
    if (s < 1) s = 1;
    p.splits = (int)s;
    return p;
}

}  // namespace

bool tc_shapes_supported(int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    // every TMA box (64 columns x up to 128/256 rows) must fit inside its matrix
    return M_keep_cap >= 64 && M < (1ll << 31) && C_in >= 128 && C_out >= 128 && C_in % 8 == 0 && C_out % 8 == 0;
}

size_t tc_dw_workspace_bytes(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    const DwPlan p = plan_dw(M_keep_cap, C_in, C_out);
    return p.splits > 1 ? (size_t)p.splits * (size_t)C_in * (size_t)C_out * sizeof(float) : 0;
}

int tc_dw_kernel_count(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    return plan_dw(M_keep_cap, C_in, C_out).splits > 1 ? 2 : 1;
}

sbp_status launch_tc_dx(const void* dY, const void* W, const int32_t* keep_rows, const int32_t* M_keep_dev,
                        int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out, void* dX,
                        int32_t* status_word, cudaStream_t stream) {
    const int bn = (C_in >= 256) ? 256 : 128;
    CUtensorMap map_w;
    if (!make_map(&map_w, W, C_in, C_out, (uint32_t)bn)) return SBP_ERR_CUDA;
    const dim3 grid((unsigned)((M_keep_cap + kBM - 1) / kBM), (unsigned)((C_in + bn - 1) / bn));
    cudaError_t launch_err;
    if (bn == 256) {
        static cudaError_t once = allow_smem(tc_dx_kernel<256>, TcCfg<256>::kSmemBytes);
        if (once != cudaSuccess) return SBP_ERR_CUDA;
        launch_err = launch_pdl(tc_dx_kernel<256>, grid, dim3(kTcThreads), TcCfg<256>::kSmemBytes, stream,
            map_w, (const __nv_bfloat16*)dY, keep_rows, M_keep_dev, M, M_keep_cap, (int)C_in, (int)C_out,
            (__nv_bfloat16*)dX, status_word);
    } else {
        static cudaError_t once = allow_smem(tc_dx_kernel<128>, TcCfg<128>::kSmemBytes);
        if (once != cudaSuccess) return SBP_ERR_CUDA;
        launch_err = launch_pdl(tc_dx_kernel<128>, grid, dim3(kTcThreads), TcCfg<128>::kSmemBytes, stream,
            map_w, (const __nv_bfloat16*)dY, keep_rows, M_keep_dev, M, M_keep_cap, (int)C_in, (int)C_out,
            (__nv_bfloat16*)dX, status_word);
    }
    return launch_err == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

sbp_status launch_tc_dw(const void* X_keep, const void* dY, const int32_t* keep_rows, const int32_t* M_keep_dev,
                        int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out, float* dW, bool accumulate,
                        float* workspace, int32_t* status_word, cudaStream_t stream) {
    (void)M;
    const DwPlan p = plan_dw(M_keep_cap, C_in, C_out);
    CUtensorMap map_x;
    if (!make_map(&map_x, X_keep, M_keep_cap, C_in, 64)) return SBP_ERR_CUDA;
    const dim3 grid((unsigned)((C_out + p.bn - 1) / p.bn), (unsigned)((C_in + kBM - 1) / kBM), (unsigned)p.splits);
    float* out = p.splits > 1 ? workspace : dW;
    const int acc_in_kernel = (p.splits == 1 && accumulate) ? 1 : 0;
    const int64_t split_stride = C_in * C_out;
    cudaError_t launch_err;
    if (p.bn == 256) {
        static cudaError_t once = allow_smem(tc_dw_kernel<256>, TcCfg<256>::kSmemBytes);
        if (once != cudaSuccess) return SBP_ERR_CUDA;
        launch_err = launch_pdl(tc_dw_kernel<256>, grid, dim3(kTcThreads), TcCfg<256>::kSmemBytes, stream,
            map_x, (const __nv_bfloat16*)dY, keep_rows, M_keep_dev, M_keep_cap, (int)C_in, (int)C_out, out,
            split_stride, acc_in_kernel, status_word);
    } else {
        static cudaError_t once = allow_smem(tc_dw_kernel<128>, TcCfg<128>::kSmemBytes);
        if (once != cudaSuccess) return SBP_ERR_CUDA;
        launch_err = launch_pdl(tc_dw_kernel<128>, grid, dim3(kTcThreads), TcCfg<128>::kSmemBytes, stream,
            map_x, (const __nv_bfloat16*)dY, keep_rows, M_keep_dev, M_keep_cap, (int)C_in, (int)C_out, out,
            split_stride, acc_in_kernel, status_word);
    }
    if (launch_err != cudaSuccess) return SBP_ERR_CUDA;
    if (p.splits > 1 &&
        launch_reduce_partials(workspace, p.splits, C_in * C_out, dW, accumulate, status_word, stream) != cudaSuccess)
        return SBP_ERR_CUDA;
    return SBP_OK;
}

}  // namespace sbp
