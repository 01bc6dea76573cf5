// Diagnostic probes (no counterpart in the paper): two micro-measurements of the machinery the tensor-core kernels are
// built from, kept in the library so that the figures the design quotes can be re-taken with one command
// (`python bench.py --probe`).
//   gather ring: rows picked by an index list are copied with 16-byte cp.async into a ring of 16 KB shared-memory
//                stages (128 rows x 128 bytes, 128-byte swizzle) behind full / empty mbarriers, exactly as the backward
//                kernel gathers the kept rows of dY; a consumer thread frees each stage as soon as it has landed.
//                Nothing is computed: the time is what the gather path alone can sustain.
//   operand feed: the gather ring together with a TMA producer that streams 16 KB boxes of a dense matrix into the same
//                stages: what shared memory can be fed with per SM when both producers of the backward kernel run.
//   mma rate:    one thread per block issues a stream of tcgen05.mma (M = 128, K = 16, bf16) of a given width on
//                constant operands and reports the clocks from the first issue to the completion of the last; the pair
//                variant issues the two-SM form (cta_group::2) from a cluster of two blocks.
#include "tc_ptx.cuh"

namespace sbp {
namespace {

struct ProbeShared {
    uint64_t full[12], empty[12], done;
    uint32_t tmem_slot;
    int abort_flag;
};

template <int THREADS>
__global__ void __launch_bounds__(THREADS + 32, 1)
probe_gather_kernel(const uint8_t* __restrict__ src, const int32_t* __restrict__ rows, int n_rows, int row_bytes, int stages,
                    int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ ProbeShared sh;
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    constexpr uint32_t kStage = 128 * 128;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&sh.full[s]), THREADS);
            ptx::mbar_init(ptx::smem_addr(&sh.empty[s]), 1);
        }
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    volatile int* abort_flag = &sh.abort_flag;
    const int ntiles = (n_rows + 127) / 128;
    const int kb_per_tile = row_bytes / 128;
    if (threadIdx.x >= THREADS) {                           // consumer warp: one lane frees the stages as they fill
        if (threadIdx.x == THREADS) {
            uint32_t it = 0;
            for (int t = blockIdx.x; t < ntiles; t += gridDim.x)
                for (int k = 0; k < kb_per_tile; ++k, ++it) {
                    const int s = it % stages;
                    if (!ptx::mbar_wait(ptx::smem_addr(&sh.full[s]), (it / stages) & 1u, abort_flag, status_word)) return;
                    ptx::mbar_arrive(ptx::smem_addr(&sh.empty[s]));
                }
        }
        return;
    }
    constexpr int RPI = THREADS / 8;                        // rows one wave of all copying threads covers
    constexpr int NI = 128 / RPI;
    const uint32_t chunk = threadIdx.x & 7u, sub = threadIdx.x >> 3;
    uint32_t it = 0;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const uint8_t* p[NI];
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            int m = t * 128 + i * RPI + (int)sub;
            if (m >= n_rows) m = n_rows - 1;
            p[i] = src + (size_t)__ldg(rows + m) * row_bytes + chunk * 16;
        }
        for (int k = 0; k < kb_per_tile; ++k, ++it) {
            const int s = it % stages;
            bool ok = ptx::mbar_wait(ptx::smem_addr(&sh.empty[s]), ((it / stages) & 1u) ^ 1u, abort_flag, status_word);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { ptx::cp_async_wait_all(); return; }
            const uint32_t dst = ring + s * kStage;
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const uint32_t r = i * RPI + sub;
                ptx::cp_async_16(dst + r * 128 + ((chunk ^ (r & 7u)) << 4), p[i] + k * 128, 16u);
            }
            ptx::cp_async_arrive_noinc(ptx::smem_addr(&sh.full[s]));
        }
    }
    ptx::cp_async_wait_all();
}

__global__ void __launch_bounds__(128, 1)
probe_mma_kernel(int N, int mn_major, int accumulators, int iters, long long* cycles_out, int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ ProbeShared sh;
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    // operands: A = 128 x 64 (16 KB) at base, B = up to 256 x 64 (32 KB) behind it; all ones (bf16 1.0)
    for (uint32_t i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3F803F80u;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&sh.done), 1);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    ptx::fence_async_proxy();
    if (threadIdx.x < 32) ptx::tmem_alloc(ptx::smem_addr(&sh.tmem_slot), 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_slot);
    if (threadIdx.x == 0) {
        const uint32_t a_addr = base, b_addr = base + 16 * 1024;
        const uint32_t idesc = ptx::umma_idesc_bf16(128, N, mn_major != 0, mn_major != 0);
        const uint32_t k_step = mn_major ? 16u * 128u : 32u;          // as in the backward kernel's two operand layouts
        const uint32_t lbo = mn_major ? 64u * 128u : 16u;
        const long long c0 = clock64();
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (uint32_t u = 0; u < 4; ++u) {
                const uint64_t da = ptx::umma_desc_sw128(a_addr + u * k_step, lbo, 1024);
                const uint64_t db = ptx::umma_desc_sw128(b_addr + u * k_step, lbo, 1024);
                ptx::umma_bf16(tmem, da, db, idesc, (it | (int)u) != 0);
                if (accumulators == 2) ptx::umma_bf16(tmem + 256u, da, db, idesc, (it | (int)u) != 0);
            }
        }
        ptx::umma_commit(ptx::smem_addr(&sh.done));
        const bool ok = ptx::mbar_wait(ptx::smem_addr(&sh.done), 0, &sh.abort_flag, status_word);
        const long long c1 = clock64();
        if (blockIdx.x == 0) cycles_out[0] = ok ? c1 - c0 : -1;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512);
    }
}

// Operand feed: what the backward kernel's two producers deliver together.  Per stage, 64 threads gather `gather_rows`
// (0, 64 or 128) rows x 128 bytes with 16-byte cp.async, as above, and one thread issues `tma_boxes` (0..3) TMA loads of
// 128 rows x 128 bytes (16 KB, 128-byte swizzle) at scattered places of a dense bf16 matrix; a consumer thread frees the
// stage as soon as everything has landed.  Nothing is computed and nothing is written to global memory.
__global__ void __launch_bounds__(128, 1)
probe_feed_kernel(const __grid_constant__ CUtensorMap map, const uint8_t* __restrict__ src, const int32_t* __restrict__ rows, int n_rows,
                  int row_bytes, int gather_rows, int dense_row_boxes, int dense_col_boxes, int tma_boxes, int stages, int steps,
                  int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ ProbeShared sh;
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    const uint32_t stage_bytes = (uint32_t)gather_rows * 128u + (uint32_t)tma_boxes * 16384u;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&sh.full[s]), 1 + (gather_rows > 0 ? 64 : 0));
            ptx::mbar_init(ptx::smem_addr(&sh.empty[s]), 1);
        }
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map);
    }
    __syncthreads();
    volatile int* abort_flag = &sh.abort_flag;
    if (warp == 3) {                                        // consumer
        if (threadIdx.x == 96)
            for (int it = 0; it < steps; ++it) {
                const int s = it % stages;
                if (!ptx::mbar_wait(ptx::smem_addr(&sh.full[s]), (it / stages) & 1u, abort_flag, status_word)) break;
                ptx::mbar_arrive(ptx::smem_addr(&sh.empty[s]));
            }
    } else if (warp == 2) {                                 // TMA producer
        if (threadIdx.x == 64) {
            int it = 0;
            bool ok = true;
            for (; it < steps; ++it) {
                const int s = it % stages;
                ok = ptx::mbar_wait(ptx::smem_addr(&sh.empty[s]), ((it / stages) & 1u) ^ 1u, abort_flag, status_word);
                if (!ok) break;
                const uint32_t full = ptx::smem_addr(&sh.full[s]);
                ptx::mbar_arrive_expect_tx(full, (uint32_t)tma_boxes * 16384u);
                const uint32_t dst = ring + s * stage_bytes + (uint32_t)gather_rows * 128u;
                for (int b = 0; b < tma_boxes; ++b) {
                    const int x = ((it * 7 + (int)blockIdx.x) % dense_col_boxes) * 64;
                    const int y = ((it * 13 + (int)blockIdx.x * 31 + b * 5) % dense_row_boxes) * 128;
                    ptx::tma_load_2d(dst + b * 16384u, &map, x, y, full);
                }
            }
            if (!ok)                                        // let the loads already issued land before shared memory goes away
                for (int j = (it > stages ? it - stages : 0); j < it; ++j)
                    for (int spin = 0; spin < (1 << 14); ++spin)
                        if (ptx::mbar_try_wait(ptx::smem_addr(&sh.full[j % stages]), (j / stages) & 1u)) break;
        }
    } else if (gather_rows > 0) {                           // gather producers: 8 rows x 128 bytes per pass of the 64 threads
        // as in the backward kernel a tile's row pointers are fetched once and serve all its 128-byte pieces
        const uint32_t chunk = threadIdx.x & 7u, sub = threadIdx.x >> 3;
        const int pieces = row_bytes / 128;
        int it = 0;
        bool ok = true;
        const int tiles = n_rows / gather_rows;             // the list is walked again from its start when it runs out
        for (int tile = (int)blockIdx.x % tiles; ok && it < steps; tile = (tile + (int)gridDim.x) % tiles) {
            const uint8_t* p[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int m = tile * gather_rows + (i * 8 + (int)sub) % gather_rows;
                p[i] = src + (size_t)__ldg(rows + m) * row_bytes + chunk * 16;
            }
            for (int piece = 0; piece < pieces && it < steps; ++piece, ++it) {
                const int s = it % stages;
                ok = ptx::mbar_wait(ptx::smem_addr(&sh.empty[s]), ((it / stages) & 1u) ^ 1u, abort_flag, status_word);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t dst = ring + s * stage_bytes;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const uint32_t r = i * 8 + sub;
                    if ((int)r < gather_rows) ptx::cp_async_16(dst + r * 128 + ((chunk ^ (r & 7u)) << 4), p[i] + piece * 128, 16u);
                }
                ptx::cp_async_arrive_noinc(ptx::smem_addr(&sh.full[s]));
            }
        }
        ptx::cp_async_wait_all();
    }
}

// The same stream issued for a pair of SMs: a cluster of two blocks, tensor memory allocated for the pair, and block 0's
// thread 0 issuing tcgen05.mma.cta_group::2 (M = 256 over the pair: 128 accumulator rows in each SM; each SM supplies
// its 128 rows of A and N / 2 rows of B from its own shared memory).  Block 1 only provides its operands and stays until
// block 0 has seen the last product finish (cluster barrier, reached on every path).
__global__ void __launch_bounds__(128, 1)
probe_mma_pair_kernel(int N, int mn_major, int iters, long long* cycles_out, int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ ProbeShared sh;
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    for (uint32_t i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3F803F80u;
    uint32_t cta_rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(cta_rank));
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&sh.done), 1);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    ptx::fence_async_proxy();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_addr(&sh.tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    ptx::tc_fence_before_sync();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_slot);
    if (cta_rank == 0 && threadIdx.x == 0) {
        const uint32_t a_addr = base, b_addr = base + 16 * 1024;
        const uint32_t idesc = ptx::umma_idesc_bf16(256, N, mn_major != 0, mn_major != 0);
        const uint32_t k_step = mn_major ? 16u * 128u : 32u;
        const uint32_t lbo = mn_major ? 64u * 128u : 16u;
        const long long c0 = clock64();
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (uint32_t u = 0; u < 4; ++u) {
                const uint64_t da = ptx::umma_desc_sw128(a_addr + u * k_step, lbo, 1024);
                const uint64_t db = ptx::umma_desc_sw128(b_addr + u * k_step, lbo, 1024);
                const uint32_t acc = (it | (int)u) != 0;
                asm volatile(
                    "{\n\t.reg .pred p;\n\t"
                    "setp.ne.b32 p, %4, 0;\n\t"
                    "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                    ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
            }
        }
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(ptx::smem_addr(&sh.done)) : "memory");
        const bool ok = ptx::mbar_wait(ptx::smem_addr(&sh.done), 0, &sh.abort_flag, status_word);
        const long long c1 = clock64();
        if (blockIdx.x == 0) cycles_out[0] = ok ? c1 - c0 : -1;
    }
    ptx::tc_fence_before_sync();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (threadIdx.x < 32) {
        ptx::tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

}  // namespace
}  // namespace sbp

extern "C" {

sbp_status sbp_probe_gather_ring(const void* src, int64_t row_bytes, const int32_t* rows, int64_t n_rows, int threads, int stages,
                                 int blocks, int32_t* status_word, void* stream) {
    using namespace sbp;
    if (src == nullptr || rows == nullptr || (reinterpret_cast<uintptr_t>(src) & 15u) || (reinterpret_cast<uintptr_t>(rows) & 3u))
        return SBP_ERR_INVALID_ARG;
    if (row_bytes < 128 || row_bytes % 128 != 0 || row_bytes > (1 << 20) || n_rows <= 0 || n_rows >= (1ll << 31)) return SBP_ERR_INVALID_ARG;
    if (stages < 2 || stages > 12 || blocks < 1 || blocks > 4 * kNumSMs) return SBP_ERR_INVALID_ARG;
    const size_t smem = (size_t)stages * 16384 + 1024;
    cudaError_t e;
    cudaStream_t st = (cudaStream_t)stream;
    if (threads == 64) {
        e = opt_in_dynamic_smem<probe_gather_kernel<64>>(197 * 1024);
        if (e == cudaSuccess) probe_gather_kernel<64><<<blocks, 96, smem, st>>>((const uint8_t*)src, rows, (int)n_rows, (int)row_bytes, stages, status_word);
    } else if (threads == 128) {
        e = opt_in_dynamic_smem<probe_gather_kernel<128>>(197 * 1024);
        if (e == cudaSuccess) probe_gather_kernel<128><<<blocks, 160, smem, st>>>((const uint8_t*)src, rows, (int)n_rows, (int)row_bytes, stages, status_word);
    } else if (threads == 256) {
        e = opt_in_dynamic_smem<probe_gather_kernel<256>>(197 * 1024);
        if (e == cudaSuccess) probe_gather_kernel<256><<<blocks, 288, smem, st>>>((const uint8_t*)src, rows, (int)n_rows, (int)row_bytes, stages, status_word);
    } else {
        return SBP_ERR_INVALID_ARG;
    }
    if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return SBP_ERR_CUDA;
    return SBP_OK;
}

sbp_status sbp_probe_operand_feed(const void* src, int64_t row_bytes, const int32_t* rows, int64_t n_rows, int gather_rows,
                                  const void* dense, int64_t dense_rows, int64_t dense_cols, int tma_boxes, int stages, int steps,
                                  int blocks, int32_t* status_word, void* stream) {
    using namespace sbp;
    if (src == nullptr || rows == nullptr || dense == nullptr || (reinterpret_cast<uintptr_t>(src) & 15u) ||
        (reinterpret_cast<uintptr_t>(dense) & 15u) || (reinterpret_cast<uintptr_t>(rows) & 3u))
        return SBP_ERR_INVALID_ARG;
    if (row_bytes < 128 || row_bytes % 128 != 0 || row_bytes > (1 << 20) || n_rows < 128 || n_rows >= (1ll << 31)) return SBP_ERR_INVALID_ARG;
    if ((gather_rows != 0 && gather_rows != 64 && gather_rows != 128) || tma_boxes < 0 || tma_boxes > 3 || (gather_rows == 0 && tma_boxes == 0))
        return SBP_ERR_INVALID_ARG;
    if (dense_rows < 128 || dense_rows % 128 != 0 || dense_cols < 64 || dense_cols % 64 != 0 || dense_rows >= (1ll << 31) || dense_cols >= (1ll << 31))
        return SBP_ERR_INVALID_ARG;
    const size_t stage_bytes = (size_t)gather_rows * 128 + (size_t)tma_boxes * 16384;
    if (stages < 2 || stages > 12 || (size_t)stages * stage_bytes > 192 * 1024 || steps < 1 || steps > (1 << 20) || blocks < 1 || blocks > kNumSMs)
        return SBP_ERR_INVALID_ARG;
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                 const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || fn == nullptr)
        return SBP_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)dense_cols, (cuuint64_t)dense_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)dense_cols * 2};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t elem_strides[2] = {1, 1};
    if (reinterpret_cast<EncodeFn>(fn)(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(dense), dims, strides, box, elem_strides,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SBP_ERR_CUDA;
    const cudaError_t e = opt_in_dynamic_smem<probe_feed_kernel>(197 * 1024);
    if (e != cudaSuccess) return SBP_ERR_CUDA;
    probe_feed_kernel<<<blocks, 128, (size_t)stages * stage_bytes + 1024, (cudaStream_t)stream>>>(
        map, (const uint8_t*)src, rows, (int)n_rows, (int)row_bytes, gather_rows, (int)(dense_rows / 128), (int)(dense_cols / 64), tma_boxes, stages,
        steps, status_word);
    return cudaGetLastError() == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

sbp_status sbp_probe_mma_rate(int N, int mn_major, int accumulators, int iters, int blocks, int64_t* cycles_out, int32_t* status_word,
                              void* stream) {
    using namespace sbp;
    if (cycles_out == nullptr || (reinterpret_cast<uintptr_t>(cycles_out) & 7u)) return SBP_ERR_INVALID_ARG;
    if (N < 16 || N > 256 || N % 16 != 0 || (accumulators != 1 && accumulators != 2) || iters < 1 || iters > 100000 || blocks < 1 ||
        blocks > kNumSMs)
        return SBP_ERR_INVALID_ARG;
    const cudaError_t e = opt_in_dynamic_smem<probe_mma_kernel>(50 * 1024);
    if (e != cudaSuccess) return SBP_ERR_CUDA;
    probe_mma_kernel<<<blocks, 128, 50 * 1024, (cudaStream_t)stream>>>(N, mn_major, accumulators, iters, reinterpret_cast<long long*>(cycles_out),
                                                                       status_word);
    return cudaGetLastError() == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

sbp_status sbp_probe_mma_pair_rate(int N, int mn_major, int iters, int pairs, int64_t* cycles_out, int32_t* status_word, void* stream) {
    using namespace sbp;
    if (cycles_out == nullptr || (reinterpret_cast<uintptr_t>(cycles_out) & 7u)) return SBP_ERR_INVALID_ARG;
    if (N < 32 || N > 256 || N % 32 != 0 || iters < 1 || iters > 100000 || pairs < 1 || pairs > kNumSMs / 2) return SBP_ERR_INVALID_ARG;
    const cudaError_t e = opt_in_dynamic_smem<probe_mma_pair_kernel>(50 * 1024);
    if (e != cudaSuccess) return SBP_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = 50 * 1024;
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t l = cudaLaunchKernelEx(&cfg, probe_mma_pair_kernel, N, mn_major, iters, reinterpret_cast<long long*>(cycles_out), status_word);
    return (l == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SBP_OK : SBP_ERR_CUDA;
}

}  // extern "C"
