// SBP backward of scaled dot-product attention on token subsets (Sec. 4, "How to apply SBP on MHSA?"; supplementary,
// "Gradient Calculation of Attention Layers"), bf16 on the tensor cores (tcgen05 / TMEM), head dimension 64.
//
// One (sample, head) problem at a time per block (persistent blocks, one per SM).  With Zq the kept query tokens and Zk
// the kept key / value tokens of the sample (at most 256 each):
//     S  = softmax_j(q_i . k_j / sqrt(d))  over j in Zk          (recomputed here: no n x n map is cached at all)
//     dS = dA V^T,   dM = S * (dS - rowsum(S * dS)) / sqrt(d)
//     dV = S^T dA,   dK = dM^T Q,   dQ = dM K
// All five products run as tcgen05.mma on operands staged once in shared memory (128-byte swizzle): a row-major
// [tokens x 64] tile serves as the K-major operand of Q K^T / dA V^T and, unchanged, as the MN-major operand of the
// three gradient products.  A first pass over the query tiles finds each row's softmax statistics (maximum, sum,
// rowsum(S * dS)) from S and dS in tensor memory; the second pass recomputes 128 x 128 blocks of S and dS, turns them
// into bf16 blocks of S and dM in shared memory, and accumulates dV, dK (per key tile) and dQ (per query tile) in
// tensor memory: 128 + 128 + 64 + 64 + 2 * 64 = 512 columns.  Rows of the outputs outside the token sets are zeroed
// by a small kernel of their own.  Every wait is bounded and reports through the status word.
#include "tc_ptx.cuh"

namespace sbp {
namespace {

constexpr int kAttnThreads = 256;
constexpr int kD = 64;                          // head dimension (one 128-byte swizzle row of bf16)
constexpr int kMaxTok = 256;                    // most kept tokens of a sample on either side
constexpr uint32_t kRowB = 128;
constexpr uint32_t kTokBytes = kMaxTok * kRowB;             // 32 KB: one [256 x 64] operand
constexpr uint32_t kBlkBytes = 128 * kRowB;                 // 16 KB: [128 rows x 64 columns]
constexpr uint32_t kAttnSmem = 4 * kTokBytes + 2 * 2 * kBlkBytes + 1024;   // Q, K, V, dA + S block + dM block (+ alignment slack)
static_assert(kAttnSmem <= 227 * 1024, "shared memory per block");

// tensor-memory columns
constexpr uint32_t kColS = 0, kColDS = 128, kColDV = 256, kColDK = 320, kColDQ = 384;   // second pass
constexpr uint32_t kColS1 = 0, kColDS1 = 256;                                            // first pass: up to 256 keys each

struct AttnParams {
    const __nv_bfloat16 *Q, *K, *V, *dA;
    int64_t ld_qkv, ld_da, ld_out;
    const int32_t *q_rows, *q_offs, *k_rows, *k_offs;     // null rows = every token of the sample
    int B, N, heads;
    __nv_bfloat16 *dQ, *dK, *dV;
    float scale;
    int zero_fill;                // 1: the rows of a sample that its list leaves out are written as zeros
    int32_t* status_word;
};

struct AttnShared {
    uint64_t bar_s, bar_o;
    uint32_t tmem_slot;
    int abort_flag;
    float part[2][128][3];        // per column half: running maximum, sum, sum of e^(s-m) * dS
    float stat[kMaxTok][3];       // per query row: -maximum (base 2, scaled), 1 / sum, -rowsum(S * dS) / sqrt(d)
    int32_t q_glob[kMaxTok], k_glob[kMaxTok];   // global row of every query / key of the problem (-1: none)
};

__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t chunk) { return row * kRowB + ((chunk ^ (row & 7u)) << 4); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Zeros for one head's 64 columns in the rows of sample b that an ascending token list leaves out.  `glob` holds the
// global row of every listed token of the sample (shared memory, filled by the block before the barrier in front of
// this call).  Eight threads share a row (one 128-byte line, 16 bytes each, so that a warp's store covers four whole
// lines); such a group takes the runs of rows in front of listed token g, g + groups, ..., the run behind the last
// token counting as one more.  Rows are clamped to the sample, so that a list that breaks the ascending order cannot
// send a store anywhere else.  The stores are fire and forget: issued while the first products run.
__device__ __forceinline__ void zero_gap_rows(__nv_bfloat16* out0, __nv_bfloat16* out1, int64_t ld, int col0, const int32_t* glob,
                                              int count, int base_row, int N, int t, int threads) {
    const int end = base_row + N;
    const int chunk = (t & 7) * 8;
    for (int g = t >> 3; g <= count; g += threads >> 3) {
        int lo = g > 0 ? glob[g - 1] + 1 : base_row;
        int hi = g < count ? glob[g] : end;
        lo = lo < base_row ? base_row : lo;
        hi = hi > end ? end : hi;
        for (int r = lo; r < hi; ++r) {
            ptx::st_global_v4(out0 + (int64_t)r * ld + col0 + chunk, 0u, 0u, 0u, 0u);
            if (out1 != nullptr) ptx::st_global_v4(out1 + (int64_t)r * ld + col0 + chunk, 0u, 0u, 0u, 0u);
        }
    }
}
__device__ __forceinline__ void zero_unlisted_rows(const AttnParams& p, int prob, int nq, int nk, const int32_t* q_glob,
                                                   const int32_t* k_glob, int t, int threads) {
    if (!p.zero_fill) return;
    const int b = prob / p.heads, col0 = (prob % p.heads) * kD;
    if (p.q_rows != nullptr) zero_gap_rows(p.dQ, nullptr, p.ld_out, col0, q_glob, nq, b * p.N, p.N, t, threads);
    if (p.k_rows != nullptr) zero_gap_rows(p.dK, p.dV, p.ld_out, col0, k_glob, nk, b * p.N, p.N, t, threads);
}

// What a thread needs to know about a problem before it can start its copies: the token counts, the global rows
// (t / 8 + 32 i) whose 16-byte chunk t % 8 it copies on the query and on the key side, and the global rows of query
// and key number t (for the read-out).  Fetched one problem ahead, so that these dependent index loads never sit in
// front of the copies.
struct BigMeta {
    int nq, nk;
    int32_t qid[8], kid[8];       // -1: no such token (the row is zero-filled)
    int32_t q_glob, k_glob;
};
__device__ __forceinline__ BigMeta fetch_big_meta(const AttnParams& p, int prob) {
    BigMeta mt;
    mt.nq = mt.nk = 0;
    if (prob >= p.B * p.heads) return mt;
    const int b = prob / p.heads;
    const int base_row = b * p.N;
    const int q0 = p.q_rows ? __ldg(p.q_offs + b) : 0, k0 = p.k_rows ? __ldg(p.k_offs + b) : 0;
    mt.nq = p.q_rows ? __ldg(p.q_offs + b + 1) - q0 : p.N;
    mt.nk = p.k_rows ? __ldg(p.k_offs + b + 1) - k0 : p.N;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (threadIdx.x >> 3) + 32 * i;
        mt.qid[i] = r < mt.nq ? (p.q_rows ? __ldg(p.q_rows + q0 + r) : base_row + r) : -1;
        mt.kid[i] = r < mt.nk ? (p.k_rows ? __ldg(p.k_rows + k0 + r) : base_row + r) : -1;
    }
    const int r = threadIdx.x;
    mt.q_glob = r < mt.nq ? (p.q_rows ? __ldg(p.q_rows + q0 + r) : base_row + r) : -1;
    mt.k_glob = r < mt.nk ? (p.k_rows ? __ldg(p.k_rows + k0 + r) : base_row + r) : -1;
    return mt;
}
// rows past `count` (up to the next multiple of 16, which is as far as the products step) become zeros
__device__ __forceinline__ void load_rows_big(uint32_t dst, const __nv_bfloat16* src, int64_t ld, const int32_t (&id)[8], int count, int col0) {
    const uint32_t chunk = threadIdx.x & 7u;
    const int padded = (count + 15) & ~15;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (threadIdx.x >> 3) + 32 * i;
        if (r < padded)
            ptx::cp_async_16(dst + swz((uint32_t)r, chunk), src + (id[i] >= 0 ? (int64_t)id[i] * ld + col0 + chunk * 8 : 0), id[i] >= 0 ? 16u : 0u);
    }
}

__global__ void __launch_bounds__(kAttnThreads, 1) attention_bwd_kernel(const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ AttnShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - raw);                 // generic pointer to the same place
    const uint32_t sQ = base, sK = base + kTokBytes, sV = base + 2 * kTokBytes, sDA = base + 3 * kTokBytes;
    const uint32_t sP = base + 4 * kTokBytes, sDM = sP + 2 * kBlkBytes;     // [2 blocks of 64 keys][128 query rows][128 B]
    uint8_t* gP = gen + 4 * kTokBytes;
    uint8_t* gDM = gP + 2 * kBlkBytes;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&sh.bar_s), 1);
        ptx::mbar_init(ptx::smem_addr(&sh.bar_o), 1);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0) ptx::tmem_alloc(ptx::smem_addr(&sh.tmem_slot), 512);
    // operand rows a problem does not fill are still read by the products (they only reach accumulator rows nobody
    // stores), so they must hold finite numbers: clear everything once
    for (uint32_t w = threadIdx.x; w < (4 * kTokBytes + 4 * kBlkBytes) / 16; w += kAttnThreads) reinterpret_cast<uint4*>(gen)[w] = make_uint4(0u, 0u, 0u, 0u);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_slot);
    volatile int* abort_flag = &sh.abort_flag;
    pdl_wait();
    const bool skip_all = p.status_word != nullptr && *reinterpret_cast<volatile int32_t*>(p.status_word) != 0;

    const int q4 = warp & 3, half = warp >> 2;              // TMEM lane quadrant of this warp; which half of the columns it takes
    const int row = q4 * 32 + lane;                         // accumulator row (query row, or key row in the dV / dK read-out)
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const float sl2 = p.scale * 1.4426950408889634f;        // scores are kept in base 2: e^(x) = 2^(x log2 e)
    uint32_t n_s = 0, n_o = 0;                              // completed uses of the two barriers
    bool ok = !skip_all;
    BigMeta cur = fetch_big_meta(p, ok ? (int)blockIdx.x : p.B * p.heads);

    for (int prob = blockIdx.x; ok && prob < p.B * p.heads; prob += gridDim.x) {
        const int nq = cur.nq, nk = cur.nk;
        const int col0 = (prob % p.heads) * kD;
        if (nq > 0 && nk > 0) {
            load_rows_big(sQ, p.Q, p.ld_qkv, cur.qid, nq, col0);
            load_rows_big(sK, p.K, p.ld_qkv, cur.kid, nk, col0);
            load_rows_big(sDA, p.dA, p.ld_da, cur.qid, nq, col0);
            load_rows_big(sV, p.V, p.ld_qkv, cur.kid, nk, col0);
        }
        sh.q_glob[threadIdx.x] = cur.q_glob;
        sh.k_glob[threadIdx.x] = cur.k_glob;
        cur = fetch_big_meta(p, prob + (int)gridDim.x);      // the next problem's indices travel while this one computes
        if (nq <= 0 || nk <= 0) {                            // nothing to compute: only the zeros of the unlisted rows
            __syncthreads();
            zero_unlisted_rows(p, prob, nq, nk, sh.q_glob, sh.k_glob, (int)threadIdx.x, kAttnThreads);
            __syncthreads();
            continue;
        }
        const int QT = (nq + 127) >> 7, KT = (nk + 127) >> 7;
        const int keys_pad = (nk + 15) & ~15;               // accumulator columns of the first pass (a multiple of 16)
        ptx::cp_async_wait_all();
        ptx::fence_async_proxy();
        __syncthreads();

        // ---- first pass: softmax statistics of every query row (S and dS over all keys: up to 256 columns each) ----
        for (int qt = 0; qt < QT && ok; ++qt) {
            if (threadIdx.x == 0) {
                ptx::tc_fence_after_sync();
                const uint32_t idesc = ptx::umma_idesc_bf16(128, keys_pad, false, false);
#pragma unroll
                for (uint32_t u = 0; u < 4; ++u) {          // the two products alternate: they fill different accumulators
                    ptx::umma_bf16(tmem + kColS1, ptx::umma_desc_sw128(sQ + qt * kBlkBytes + u * 32, 16, 1024),
                                   ptx::umma_desc_sw128(sK + u * 32, 16, 1024), idesc, u != 0);
                    ptx::umma_bf16(tmem + kColDS1, ptx::umma_desc_sw128(sDA + qt * kBlkBytes + u * 32, 16, 1024),
                                   ptx::umma_desc_sw128(sV + u * 32, 16, 1024), idesc, u != 0);
                }
                ptx::umma_commit(ptx::smem_addr(&sh.bar_s));
            }
            if (qt == 0) zero_unlisted_rows(p, prob, nq, nk, sh.q_glob, sh.k_glob, (int)threadIdx.x, kAttnThreads);
            ok = ptx::mbar_wait(ptx::smem_addr(&sh.bar_s), n_s & 1u, abort_flag, p.status_word);
            ++n_s;
            ok = !__syncthreads_or(!ok);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            // this thread: row `row`, columns [128 half, 128 half + 128) below keys_pad; two sweeps (maximum; sums)
            const int cbeg = half * 128, cend = keys_pad < cbeg + 128 ? keys_pad : cbeg + 128;
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four interleaved chains, not one long one
            for (int c = cbeg; c < cend; c += 32) {
                float s[32];
                ptx::tmem_ld_32x32(tmem + kColS1 + (uint32_t)c + lane_off, s);
                ptx::tmem_ld_wait();
                if (c + 32 <= nk) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], s[j]);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], (c + j < nk) ? s[j] : -INFINITY);
                }
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            float l4[4] = {0.f, 0.f, 0.f, 0.f}, u4[4] = {0.f, 0.f, 0.f, 0.f};
            if (mx > -INFINITY) {
                const float nm = -mx * sl2;
                for (int c = cbeg; c < cend; c += 32) {
                    float s[32], ds[32];
                    ptx::tmem_ld_32x32(tmem + kColS1 + (uint32_t)c + lane_off, s);
                    ptx::tmem_ld_32x32(tmem + kColDS1 + (uint32_t)c + lane_off, ds);
                    ptx::tmem_ld_wait();
                    const bool whole = c + 32 <= nk;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float e = ex2(fmaf(s[j], sl2, nm)), g = ds[j];
                        if (!whole) {                        // a stale column may hold anything, NaN included
                            e = (c + j < nk) ? e : 0.f;
                            g = (c + j < nk) ? g : 0.f;
                        }
                        l4[j & 3] += e;
                        u4[j & 3] = fmaf(e, g, u4[j & 3]);
                    }
                }
            }
            const float l = (l4[0] + l4[1]) + (l4[2] + l4[3]), u_acc = (u4[0] + u4[1]) + (u4[2] + u4[3]);
            sh.part[half][row][0] = mx; sh.part[half][row][1] = l; sh.part[half][row][2] = u_acc;
            ptx::tc_fence_before_sync();
            __syncthreads();
            if (half == 0) {                                 // the two halves of a row, rescaled to their common maximum
                const float m0 = sh.part[0][row][0], m1 = sh.part[1][row][0];
                const float mm = fmaxf(m0, m1);
                const float f0 = (m0 > -INFINITY) ? ex2((m0 - mm) * sl2) : 0.f, f1 = (m1 > -INFINITY) ? ex2((m1 - mm) * sl2) : 0.f;
                const float ll = sh.part[0][row][1] * f0 + sh.part[1][row][1] * f1;
                const float uu = sh.part[0][row][2] * f0 + sh.part[1][row][2] * f1;
                const float inv_l = 1.f / ll;
                sh.stat[qt * 128 + row][0] = -mm * sl2;
                sh.stat[qt * 128 + row][1] = inv_l;
                sh.stat[qt * 128 + row][2] = -uu * inv_l * p.scale;      // -rowsum(S dS) / sqrt(d)
            }
            __syncthreads();
        }
        if (!ok) break;

        // ---- second pass: 128 x 128 blocks of S and dM, and the three gradient products ----
        for (int kt = 0; kt < KT && ok; ++kt) {
            const int kb = keys_pad - kt * 128 < 128 ? keys_pad - kt * 128 : 128;      // key columns of this tile (a multiple of 16)
            const uint32_t k_steps = (uint32_t)kb >> 4;
            for (int qt = 0; qt < QT && ok; ++qt) {
                const int q_rows_here = nq - qt * 128 < 128 ? nq - qt * 128 : 128;
                const uint32_t q_steps = (uint32_t)(q_rows_here + 15) >> 4;
                if (threadIdx.x == 0) {
                    ptx::tc_fence_after_sync();
                    const uint32_t idesc = ptx::umma_idesc_bf16(128, kb, false, false);
#pragma unroll
                    for (uint32_t u = 0; u < 4; ++u) {
                        ptx::umma_bf16(tmem + kColS, ptx::umma_desc_sw128(sQ + qt * kBlkBytes + u * 32, 16, 1024),
                                       ptx::umma_desc_sw128(sK + kt * kBlkBytes + u * 32, 16, 1024), idesc, u != 0);
                        ptx::umma_bf16(tmem + kColDS, ptx::umma_desc_sw128(sDA + qt * kBlkBytes + u * 32, 16, 1024),
                                       ptx::umma_desc_sw128(sV + kt * kBlkBytes + u * 32, 16, 1024), idesc, u != 0);
                    }
                    ptx::umma_commit(ptx::smem_addr(&sh.bar_s));
                }
                ok = ptx::mbar_wait(ptx::smem_addr(&sh.bar_s), n_s & 1u, abort_flag, p.status_word);
                ++n_s;
                ok = !__syncthreads_or(!ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const float nm = sh.stat[qt * 128 + row][0], inv_l = sh.stat[qt * 128 + row][1], nds = sh.stat[qt * 128 + row][2];
#pragma unroll
                for (int c = 0; c < 64; c += 32) {
                    const int cc = half * 64 + c;           // column within the tile
                    if (cc < kb) {
                        float s[32], ds[32];
                        ptx::tmem_ld_32x32(tmem + kColS + (uint32_t)cc + lane_off, s);
                        ptx::tmem_ld_32x32(tmem + kColDS + (uint32_t)cc + lane_off, ds);
                        ptx::tmem_ld_wait();
                        const bool whole = kt * 128 + cc + 32 <= nk;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            float e = ex2(fmaf(s[j], sl2, nm)), g = ds[j];
                            if (!whole) {
                                e = (kt * 128 + cc + j < nk) ? e : 0.f;
                                g = (kt * 128 + cc + j < nk) ? g : 0.f;
                            }
                            const float pj = e * inv_l;
                            s[j] = pj;
                            ds[j] = pj * fmaf(g, p.scale, nds);      // dM / sqrt(d)
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t off = (uint32_t)half * kBlkBytes + swz((uint32_t)row, (uint32_t)(c / 8 + q));
                            *reinterpret_cast<uint4*>(gP + off) =
                                make_uint4(pack2(s[q * 8], s[q * 8 + 1]), pack2(s[q * 8 + 2], s[q * 8 + 3]), pack2(s[q * 8 + 4], s[q * 8 + 5]), pack2(s[q * 8 + 6], s[q * 8 + 7]));
                            *reinterpret_cast<uint4*>(gDM + off) =
                                make_uint4(pack2(ds[q * 8], ds[q * 8 + 1]), pack2(ds[q * 8 + 2], ds[q * 8 + 3]), pack2(ds[q * 8 + 4], ds[q * 8 + 5]), pack2(ds[q * 8 + 6], ds[q * 8 + 7]));
                        }
                    }
                }
                ptx::fence_async_proxy();                    // the blocks are read by the tensor core
                ptx::tc_fence_before_sync();
                __syncthreads();
                if (threadIdx.x == 0) {
                    ptx::tc_fence_after_sync();
                    const uint32_t id_t = ptx::umma_idesc_bf16(128, 64, true, true);     // dV, dK: both operands MN-major
                    const uint32_t id_q = ptx::umma_idesc_bf16(128, 64, false, true);    // dQ: dM K-major, K MN-major
                    const uint32_t steps = q_steps > k_steps ? q_steps : k_steps;
                    for (uint32_t u = 0; u < steps; ++u) {   // three accumulators take turns; only the 16-row steps that hold tokens run
                        if (u < q_steps) {                   // reductions over the query rows of the tile
                            ptx::umma_bf16(tmem + kColDV, ptx::umma_desc_sw128(sP + u * 2048, kBlkBytes, 1024),
                                           ptx::umma_desc_sw128(sDA + qt * kBlkBytes + u * 2048, kBlkBytes, 1024), id_t, (qt | (int)u) != 0);
                            ptx::umma_bf16(tmem + kColDK, ptx::umma_desc_sw128(sDM + u * 2048, kBlkBytes, 1024),
                                           ptx::umma_desc_sw128(sQ + qt * kBlkBytes + u * 2048, kBlkBytes, 1024), id_t, (qt | (int)u) != 0);
                        }
                        if (u < k_steps)                     // reduction over the keys of the tile: two 64-key blocks x four steps
                            ptx::umma_bf16(tmem + kColDQ + (uint32_t)qt * 64u, ptx::umma_desc_sw128(sDM + (u >> 2) * kBlkBytes + (u & 3u) * 32, 16, 1024),
                                           ptx::umma_desc_sw128(sK + kt * kBlkBytes + u * 2048, kBlkBytes, 1024), id_q, (kt | (int)u) != 0);
                    }
                    ptx::umma_commit(ptx::smem_addr(&sh.bar_o));
                }
                ok = ptx::mbar_wait(ptx::smem_addr(&sh.bar_o), n_o & 1u, abort_flag, p.status_word);
                ++n_o;
                ok = !__syncthreads_or(!ok);
            }
            if (!ok) break;
            // ---- dV and dK of this key tile: accumulator row = key; through shared memory (the S and dM blocks are free)
            //      so that every store instruction writes whole 128-byte rows ----
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                float v[32];
                ptx::tmem_ld_32x32(tmem + (which ? kColDK : kColDV) + (uint32_t)(half * 32) + lane_off, v);
                ptx::tmem_ld_wait();
                uint8_t* stage = which ? gDM : gP;
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4*>(stage + swz((uint32_t)row, (uint32_t)(half * 4 + q))) =
                        make_uint4(pack2(v[q * 8], v[q * 8 + 1]), pack2(v[q * 8 + 2], v[q * 8 + 3]), pack2(v[q * 8 + 4], v[q * 8 + 5]), pack2(v[q * 8 + 6], v[q * 8 + 7]));
            }
            ptx::tc_fence_before_sync();
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int idx = threadIdx.x + kAttnThreads * i;          // 2 outputs x 128 rows x 8 chunks
                const int which = idx >> 10, r = (idx >> 3) & 127, ch = idx & 7;
                const int32_t g = sh.k_glob[kt * 128 + r];
                if (kt * 128 + r < nk && g >= 0) {
                    const uint4 pk = *reinterpret_cast<const uint4*>((which ? gDM : gP) + swz((uint32_t)r, (uint32_t)ch));
                    ptx::st_global_v4((which ? p.dK : p.dV) + (int64_t)g * p.ld_out + col0 + ch * 8, pk.x, pk.y, pk.z, pk.w);
                }
            }
            __syncthreads();                                 // the stages become S / dM blocks again
        }
        if (!ok) break;
        // ---- dQ of every query tile ----
        ptx::tc_fence_after_sync();
        for (int qt = 0; qt < QT; ++qt) {
            float v[32];
            ptx::tmem_ld_32x32(tmem + kColDQ + (uint32_t)(qt * 64 + half * 32) + lane_off, v);
            ptx::tmem_ld_wait();
            uint8_t* stage = qt ? gDM : gP;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4*>(stage + swz((uint32_t)row, (uint32_t)(half * 4 + q))) =
                    make_uint4(pack2(v[q * 8], v[q * 8 + 1]), pack2(v[q * 8 + 2], v[q * 8 + 3]), pack2(v[q * 8 + 4], v[q * 8 + 5]), pack2(v[q * 8 + 6], v[q * 8 + 7]));
        }
        ptx::tc_fence_before_sync();
        __syncthreads();
        for (int i = 0; i < 4 * QT; ++i) {
            const int idx = threadIdx.x + kAttnThreads * i;              // QT tiles x 128 rows x 8 chunks
            const int qt = idx >> 10, r = (idx >> 3) & 127, ch = idx & 7;
            const int32_t g = sh.q_glob[qt * 128 + r];
            if (qt * 128 + r < nq && g >= 0) {
                const uint4 pk = *reinterpret_cast<const uint4*>((qt ? gDM : gP) + swz((uint32_t)r, (uint32_t)ch));
                ptx::st_global_v4(p.dQ + (int64_t)g * p.ld_out + col0 + ch * 8, pk.x, pk.y, pk.z, pk.w);
            }
        }
        ptx::tc_fence_before_sync();
        __syncthreads();                                     // operands, stages and accumulators are free for the next problem
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512);
    }
}

// ---------------------------------------------------------------------------------------------
// At most 128 kept tokens on both sides (keep ratios up to 0.5 on 14 x 14 maps, the paper's setting): one 128 x 128
// tile per problem, so S and dS are computed once, the statistics and the blocks come from the same accumulators, and
// the block is small enough for two per SM (96 KB of operands, 256 tensor-memory columns, 128 threads): while one block
// waits for its loads or its products, the other computes.  Each thread owns one query row: it keeps the row's dM as
// packed bf16 in registers while the S block feeds dV, then writes dM over the S block for dK and dQ.
// ---------------------------------------------------------------------------------------------
constexpr int kSmallThreads = 128;
constexpr uint32_t kSmallSmem = 4 * kBlkBytes + 2 * kBlkBytes + 1024;      // Q, K, V, dA + one S / dM block (+ alignment slack)

struct SmallShared {
    uint64_t bar_s, bar_o;
    uint32_t tmem_slot;
    int abort_flag;
    int32_t q_glob[kSmallThreads], k_glob[kSmallThreads];   // global row of every query / key of the problem (-1: none)
};

// What a thread needs to know about a problem before it can start its copies: the token counts, the global rows
// (t / 8 + 16 i) whose 16-byte chunk t % 8 it copies on the query and on the key side, and the rows whose results it
// stores.  Fetched one problem ahead, so that these dependent index loads never sit in front of the copies.
struct SmallMeta {
    int nq, nk;
    int32_t qid[8], kid[8];       // -1: no such token (the row is zero-filled)
    int32_t q_out, k_out;         // global row of query / key number threadIdx.x, -1 if there is none
};
__device__ __forceinline__ SmallMeta fetch_meta(const AttnParams& p, int prob) {
    SmallMeta mt;
    mt.nq = mt.nk = 0;
    if (prob >= p.B * p.heads) return mt;
    const int b = prob / p.heads;
    const int base_row = b * p.N;
    const int q0 = p.q_rows ? __ldg(p.q_offs + b) : 0, k0 = p.k_rows ? __ldg(p.k_offs + b) : 0;
    mt.nq = p.q_rows ? __ldg(p.q_offs + b + 1) - q0 : p.N;
    mt.nk = p.k_rows ? __ldg(p.k_offs + b + 1) - k0 : p.N;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (threadIdx.x >> 3) + 16 * i;
        mt.qid[i] = r < mt.nq ? (p.q_rows ? __ldg(p.q_rows + q0 + r) : base_row + r) : -1;
        mt.kid[i] = r < mt.nk ? (p.k_rows ? __ldg(p.k_rows + k0 + r) : base_row + r) : -1;
    }
    const int r = threadIdx.x;
    mt.q_out = r < mt.nq ? (p.q_rows ? __ldg(p.q_rows + q0 + r) : base_row + r) : -1;
    mt.k_out = r < mt.nk ? (p.k_rows ? __ldg(p.k_rows + k0 + r) : base_row + r) : -1;
    return mt;
}
// rows past `count` (up to the next multiple of 16, which is as far as the products step) become zeros
__device__ __forceinline__ void load_rows_small(uint32_t dst, const __nv_bfloat16* src, int64_t ld, const int32_t (&id)[8], int count, int col0) {
    const uint32_t chunk = threadIdx.x & 7u;
    const int padded = (count + 15) & ~15;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (threadIdx.x >> 3) + 16 * i;
        if (r < padded)
            ptx::cp_async_16(dst + swz((uint32_t)r, chunk), src + (id[i] >= 0 ? (int64_t)id[i] * ld + col0 + chunk * 8 : 0), id[i] >= 0 ? 16u : 0u);
    }
}
__global__ void __launch_bounds__(kSmallThreads, 2) attention_bwd_small_kernel(const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ SmallShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - raw);
    const uint32_t sQ = base, sK = base + kBlkBytes, sV = base + 2 * kBlkBytes, sDA = base + 3 * kBlkBytes;
    const uint32_t sP = base + 4 * kBlkBytes;              // [2 blocks of 64 keys][128 query rows][128 B]: S, later dM
    uint8_t* gP = gen + 4 * kBlkBytes;
    uint8_t* gV = gen + 2 * kBlkBytes;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&sh.bar_s), 1);
        ptx::mbar_init(ptx::smem_addr(&sh.bar_o), 1);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0) ptx::tmem_alloc(ptx::smem_addr(&sh.tmem_slot), 256);
    // operand rows that a problem does not fill are still read by the products (they only reach accumulator rows nobody
    // stores), so they must hold finite numbers: clear everything once
    for (uint32_t w = threadIdx.x; w < 6 * kBlkBytes / 16; w += kSmallThreads) reinterpret_cast<uint4*>(gen)[w] = make_uint4(0u, 0u, 0u, 0u);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_slot);
    volatile int* abort_flag = &sh.abort_flag;
    pdl_wait();
    const bool skip_all = p.status_word != nullptr && *reinterpret_cast<volatile int32_t*>(p.status_word) != 0;

    const int row = threadIdx.x;                            // accumulator row of this thread: a query, or a key in the dV / dK read-out
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const float sl2 = p.scale * 1.4426950408889634f;        // scores in base 2: e^x = 2^(x log2 e)
    uint32_t n_s = 0, n_o = 0;
    bool ok = !skip_all;
    SmallMeta cur = fetch_meta(p, ok ? (int)blockIdx.x : p.B * p.heads);

    for (int prob = blockIdx.x; ok && prob < p.B * p.heads; prob += gridDim.x) {
        const int nq = cur.nq, nk = cur.nk;
        const int col0 = (prob % p.heads) * kD;
        const int32_t q_out = cur.q_out, k_out = cur.k_out;
        if (nq > 0 && nk > 0) {
            load_rows_small(sQ, p.Q, p.ld_qkv, cur.qid, nq, col0);
            load_rows_small(sK, p.K, p.ld_qkv, cur.kid, nk, col0);
            load_rows_small(sDA, p.dA, p.ld_da, cur.qid, nq, col0);
            load_rows_small(sV, p.V, p.ld_qkv, cur.kid, nk, col0);
        }
        if (p.zero_fill) {
            sh.q_glob[threadIdx.x] = q_out;
            sh.k_glob[threadIdx.x] = k_out;
        }
        cur = fetch_meta(p, prob + (int)gridDim.x);          // the next problem's indices travel while this one computes
        if (nq <= 0 || nk <= 0) {                            // nothing to compute: only the zeros of the unlisted rows
            __syncthreads();
            zero_unlisted_rows(p, prob, nq, nk, sh.q_glob, sh.k_glob, (int)threadIdx.x, kSmallThreads);
            __syncthreads();
            continue;
        }
        const uint32_t q_steps = (uint32_t)(nq + 15) >> 4, k_steps = (uint32_t)(nk + 15) >> 4;   // 16-row steps that hold tokens
        const uint32_t n_keys = k_steps * 16u;              // accumulator columns computed (a multiple of 16)
        ptx::cp_async_wait_all();
        ptx::fence_async_proxy();
        __syncthreads();
        if (threadIdx.x == 0) {
            ptx::tc_fence_after_sync();
            const uint32_t idesc = ptx::umma_idesc_bf16(128, (int)n_keys, false, false);
#pragma unroll
            for (uint32_t u = 0; u < 4; ++u) {              // the two products alternate: they fill different accumulators
                ptx::umma_bf16(tmem, ptx::umma_desc_sw128(sQ + u * 32, 16, 1024), ptx::umma_desc_sw128(sK + u * 32, 16, 1024), idesc, u != 0);
                ptx::umma_bf16(tmem + 128u, ptx::umma_desc_sw128(sDA + u * 32, 16, 1024), ptx::umma_desc_sw128(sV + u * 32, 16, 1024), idesc, u != 0);
            }
            ptx::umma_commit(ptx::smem_addr(&sh.bar_s));
        }
        zero_unlisted_rows(p, prob, nq, nk, sh.q_glob, sh.k_glob, (int)threadIdx.x, kSmallThreads);
        ok = ptx::mbar_wait(ptx::smem_addr(&sh.bar_s), n_s & 1u, abort_flag, p.status_word);
        ++n_s;
        ok = !__syncthreads_or(!ok);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        // ---- this thread's row of S and dS, three sweeps over the accumulators: the maximum; the sum and
        //      rowsum(e^(s - m) dS); then the S block to shared memory with dM kept in registers.  Columns from nk on
        //      (padding keys, stale columns past n_keys) are masked; only the chunk holding column nk pays for it. ----
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four interleaved chains, not one of n_keys links
        for (uint32_t c = 0; c < n_keys; c += 32) {
            float s[32];
            ptx::tmem_ld_32x32(tmem + c + lane_off, s);
            ptx::tmem_ld_wait();
            if ((int)c + 32 <= nk) {
#pragma unroll
                for (int j = 0; j < 32; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], s[j]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], ((int)c + j < nk) ? s[j] : -INFINITY);
            }
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const float nm = -mx * sl2;
        float l4[4] = {0.f, 0.f, 0.f, 0.f}, u4[4] = {0.f, 0.f, 0.f, 0.f};
        for (uint32_t c = 0; c < n_keys; c += 32) {
            float s[32], ds[32];
            ptx::tmem_ld_32x32(tmem + c + lane_off, s);
            ptx::tmem_ld_32x32(tmem + 128u + c + lane_off, ds);
            ptx::tmem_ld_wait();
            const bool whole = (int)c + 32 <= nk;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                float e = ex2(fmaf(s[j], sl2, nm)), g = ds[j];
                if (!whole) {                                // a stale column may hold anything, NaN included
                    e = ((int)c + j < nk) ? e : 0.f;
                    g = ((int)c + j < nk) ? g : 0.f;
                }
                l4[j & 3] += e;
                u4[j & 3] = fmaf(e, g, u4[j & 3]);
            }
        }
        const float l = (l4[0] + l4[1]) + (l4[2] + l4[3]), u_acc = (u4[0] + u4[1]) + (u4[2] + u4[3]);
        const float inv_l = 1.f / l;
        const float nds = -u_acc * inv_l * p.scale;         // -rowsum(S dS) / sqrt(d)
        uint32_t dm[64];
#pragma unroll
        for (uint32_t c = 0; c < 128; c += 32) {
            if (c < n_keys) {
                float s[32], ds[32];
                ptx::tmem_ld_32x32(tmem + c + lane_off, s);
                ptx::tmem_ld_32x32(tmem + 128u + c + lane_off, ds);
                ptx::tmem_ld_wait();
                const bool whole = (int)c + 32 <= nk;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float e = ex2(fmaf(s[j], sl2, nm)), g = ds[j];
                    if (!whole) {
                        e = ((int)c + j < nk) ? e : 0.f;
                        g = ((int)c + j < nk) ? g : 0.f;
                    }
                    const float pj = e * inv_l;
                    s[j] = pj;
                    ds[j] = pj * fmaf(g, p.scale, nds);      // dM / sqrt(d)
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    *reinterpret_cast<uint4*>(gP + (c >> 6) * kBlkBytes + swz((uint32_t)row, ((c & 63u) >> 3) + q)) =
                        make_uint4(pack2(s[q * 8], s[q * 8 + 1]), pack2(s[q * 8 + 2], s[q * 8 + 3]), pack2(s[q * 8 + 4], s[q * 8 + 5]), pack2(s[q * 8 + 6], s[q * 8 + 7]));
#pragma unroll
                    for (int e = 0; e < 4; ++e) dm[(c >> 1) + q * 4 + e] = pack2(ds[q * 8 + 2 * e], ds[q * 8 + 2 * e + 1]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) dm[(c >> 1) + e] = 0u;
            }
        }
        ptx::fence_async_proxy();
        ptx::tc_fence_before_sync();
        __syncthreads();                                     // S and dS in tensor memory are dead from here on
        if (threadIdx.x == 0) {
            ptx::tc_fence_after_sync();
            const uint32_t id_t = ptx::umma_idesc_bf16(128, 64, true, true);
            for (uint32_t u = 0; u < q_steps; ++u)           // dV = S^T dA over the query rows
                ptx::umma_bf16(tmem, ptx::umma_desc_sw128(sP + u * 2048, kBlkBytes, 1024), ptx::umma_desc_sw128(sDA + u * 2048, kBlkBytes, 1024), id_t, u != 0);
            ptx::umma_commit(ptx::smem_addr(&sh.bar_o));
        }
        ok = ptx::mbar_wait(ptx::smem_addr(&sh.bar_o), n_o & 1u, abort_flag, p.status_word);
        ++n_o;
        ok = !__syncthreads_or(!ok);
        if (!ok) break;
        // ---- dM over the S block ----
#pragma unroll
        for (uint32_t c = 0; c < 128; c += 8)
            if (c < n_keys)
                *reinterpret_cast<uint4*>(gP + (c >> 6) * kBlkBytes + swz((uint32_t)row, (c & 63u) >> 3)) =
                    make_uint4(dm[c >> 1], dm[(c >> 1) + 1], dm[(c >> 1) + 2], dm[(c >> 1) + 3]);
        ptx::fence_async_proxy();
        ptx::tc_fence_before_sync();
        __syncthreads();
        if (threadIdx.x == 0) {
            ptx::tc_fence_after_sync();
            const uint32_t id_t = ptx::umma_idesc_bf16(128, 64, true, true), id_q = ptx::umma_idesc_bf16(128, 64, false, true);
            const uint32_t steps = q_steps > k_steps ? q_steps : k_steps;
            for (uint32_t u = 0; u < steps; ++u) {           // dK = dM^T Q over the query rows, dQ = dM K over the keys, alternating
                if (u < q_steps)
                    ptx::umma_bf16(tmem + 64u, ptx::umma_desc_sw128(sP + u * 2048, kBlkBytes, 1024), ptx::umma_desc_sw128(sQ + u * 2048, kBlkBytes, 1024), id_t, u != 0);
                if (u < k_steps)
                    ptx::umma_bf16(tmem + 128u, ptx::umma_desc_sw128(sP + (u >> 2) * kBlkBytes + (u & 3u) * 32, 16, 1024),
                                   ptx::umma_desc_sw128(sK + u * 2048, kBlkBytes, 1024), id_q, u != 0);
            }
            ptx::umma_commit(ptx::smem_addr(&sh.bar_o));
        }
        ok = ptx::mbar_wait(ptx::smem_addr(&sh.bar_o), n_o & 1u, abort_flag, p.status_word);
        ++n_o;
        ok = !__syncthreads_or(!ok);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        // ---- read-out.  A thread holds one accumulator row (a key for dV and dK, a query for dQ), but a store that
        //      touches 32 rows costs 32 transactions: each warp passes its 32 rows through shared memory (the S block's
        //      two halves and the V operand are free by now) and writes four whole 128-byte rows per instruction. ----
#pragma unroll
        for (int which = 0; which < 3; ++which) {
            uint8_t* stage = which == 0 ? gP : which == 1 ? gP + kBlkBytes : gV;
#pragma unroll
            for (int c = 0; c < 64; c += 32) {
                float v[32];
                ptx::tmem_ld_32x32(tmem + (uint32_t)(which * 64 + c) + lane_off, v);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4*>(stage + swz((uint32_t)row, (uint32_t)(c / 8 + q))) =
                        make_uint4(pack2(v[q * 8], v[q * 8 + 1]), pack2(v[q * 8 + 2], v[q * 8 + 3]), pack2(v[q * 8 + 4], v[q * 8 + 5]), pack2(v[q * 8 + 6], v[q * 8 + 7]));
            }
        }
        __syncwarp();
#pragma unroll
        for (int which = 0; which < 3; ++which) {
            const uint8_t* stage = which == 0 ? gP : which == 1 ? gP + kBlkBytes : gV;
            __nv_bfloat16* out = (which == 0 ? p.dV : which == 1 ? p.dK : p.dQ) + col0 + (lane & 7) * 8;
            const int32_t mine = which == 2 ? q_out : k_out;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = i * 4 + (lane >> 3);                                   // row within this warp's 32
                const int32_t g = __shfl_sync(0xffffffffu, mine, r);
                const uint4 pk = *reinterpret_cast<const uint4*>(stage + swz((uint32_t)(warp * 32 + r), (uint32_t)(lane & 7)));
                if (g >= 0) ptx::st_global_v4(out + (int64_t)g * p.ld_out, pk.x, pk.y, pk.z, pk.w);
            }
        }
        ptx::tc_fence_before_sync();
        __syncthreads();                                     // operands, stages and accumulators are free for the next problem
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 256);
    }
}

// rows of an output [M, ld] (columns [0, cols)) that are not in its ascending list rows[0 .. *total) become +0.0:
// entry m of the list owns the gap in front of it, one extra worker the tail; blockIdx.y picks the output
}  // namespace

bool attention_supported(sbp_dtype dt, int64_t head_dim) { return dt == SBP_BF16 && head_dim == kD; }
int64_t attention_max_tokens() { return kMaxTok; }

cudaError_t launch_attention_backward(const void* Q, const void* K, const void* V, int64_t ld_qkv, const void* dA, int64_t ld_da,
                                      const int32_t* q_rows, const int32_t* q_offs, const int32_t* k_rows, const int32_t* k_offs,
                                      int64_t B, int64_t N, int64_t heads, int64_t most_tokens, void* dQ, void* dK, void* dV,
                                      int64_t ld_out, bool zero_other_rows, int32_t* status_word, cudaStream_t stream) {
    AttnParams prm;
    prm.Q = static_cast<const __nv_bfloat16*>(Q); prm.K = static_cast<const __nv_bfloat16*>(K);
    prm.V = static_cast<const __nv_bfloat16*>(V); prm.dA = static_cast<const __nv_bfloat16*>(dA);
    prm.ld_qkv = ld_qkv; prm.ld_da = ld_da; prm.ld_out = ld_out;
    prm.q_rows = q_rows; prm.q_offs = q_offs; prm.k_rows = k_rows; prm.k_offs = k_offs;
    prm.B = (int)B; prm.N = (int)N; prm.heads = (int)heads;
    prm.dQ = static_cast<__nv_bfloat16*>(dQ); prm.dK = static_cast<__nv_bfloat16*>(dK); prm.dV = static_cast<__nv_bfloat16*>(dV);
    prm.scale = 1.0f / sqrtf((float)kD);
    prm.status_word = status_word;
    const int64_t problems = B * heads;
    // the zeros for the rows outside the lists are written by the same kernel, between a problem's copies and its products
    prm.zero_fill = (zero_other_rows && (q_rows != nullptr || k_rows != nullptr)) ? 1 : 0;
    if (most_tokens <= 128) {
        const cudaError_t opt = opt_in_dynamic_smem<attention_bwd_small_kernel>((int)kSmallSmem);
        if (opt != cudaSuccess) return opt;
        const dim3 grid((unsigned)(problems < 2 * kNumSMs ? problems : 2 * kNumSMs));
        return launch_pdl(attention_bwd_small_kernel, grid, dim3(kSmallThreads), kSmallSmem, stream, prm);
    }
    const cudaError_t opt = opt_in_dynamic_smem<attention_bwd_kernel>((int)kAttnSmem);
    if (opt != cudaSuccess) return opt;
    const dim3 grid((unsigned)(problems < kNumSMs ? problems : kNumSMs));
    return launch_pdl(attention_bwd_kernel, grid, dim3(kAttnThreads), kAttnSmem, stream, prm);
}

}  // namespace sbp
