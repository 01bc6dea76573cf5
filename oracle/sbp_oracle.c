/*
 * CPU oracle for the Stochastic Backpropagation (SBP) linear-layer hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is checked against; it shares no code with the CUDA path and is
 * never on the product path.  Floating point is fp64 throughout; the index
 * work is exact integer arithmetic.
 *
 * What each function follows (paper: "An In-depth Study of Stochastic
 * Backpropagation", arXiv 2210.00129):
 *   - keep / drop index sets and the keep ratio r:      Sec. 3.2.1 (text after Eq. 3)
 *   - random and grid-wise mask sampling:               Sec. 4 ("How to sample the
 *                                                       gradient keep mask?"), Supp. A.4
 *   - forward cache of the kept rows:                   Algorithm 1, Sec. 3.1
 *   - dW, dX of a linear / point-wise layer under SBP:  Eq. 5 and the text after it
 *   - full backward for the invariants:                 Eq. 3
 *   - no gradient rescaling:                            Eq. 1
 *   - attention with the gradient kept on token subsets: Sec. 4 ("How to apply SBP on MHSA?"), Supp.
 *                                                       "Gradient Calculation of Attention Layers"
 * The paper names no random generator; the sampler uses Philox4x32-10
 * (Salmon, Moraes, Dror, Shaw: "Parallel Random Numbers: As Easy as 1, 2, 3",
 * SC'11), written here from that paper's definition of the round function.
 *
 * Parity pins: every function here is pinned by tests that do not call it to
 * check itself (published Philox known answers, brute-force selection, hand
 * computed integer cases, reduction to library matrix products, enumeration
 * of all masks; for the attention functions: central differences of the forward,
 * the full backward written as matrix products, the paper's exact-on-kept-rows
 * statement and its printed memory ratios).  Nothing in this file is "parity unpinned".
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_MASK_RANDOM 0
#define ORACLE_MASK_GRID   1
#define ORACLE_MASK_TEMPORAL 2   /* whole frames of a video: H = frames, W = positions per frame */
#define ORACLE_MASK_TEMPORAL_GRID 3   /* frames on a lattice in time (the "even index on T" example) */
#define ORACLE_FLAG_SHARE_MASK 1u

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (SC'11, Sec. 3.3 and Table 2 of that paper)            */
/* ------------------------------------------------------------------ */

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t MUL_A = 0xD2511F53u;   /* multiplier applied to word 0 */
    const uint64_t MUL_B = 0xCD9E8D57u;   /* multiplier applied to word 2 */
    const uint32_t WEYL_0 = 0x9E3779B9u;  /* key schedule increments */
    const uint32_t WEYL_1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += WEYL_0; k1 += WEYL_1; }
        uint64_t pa = MUL_A * (uint64_t)c0;
        uint64_t pb = MUL_B * (uint64_t)c2;
        uint32_t hi_a = (uint32_t)(pa >> 32), lo_a = (uint32_t)pa;
        uint32_t hi_b = (uint32_t)(pb >> 32), lo_b = (uint32_t)pb;
        uint32_t n0 = hi_b ^ c1 ^ k0;
        uint32_t n1 = lo_b;
        uint32_t n2 = hi_a ^ c3 ^ k1;
        uint32_t n3 = lo_a;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit random word attached to position n of global sample gid.
 * Counter layout: word0 = n / 4, word1 = global sample id, word2 = step,
 * word3 = stream tag (0 = random-mask keys, 1 = grid phase); key = seed.
 * Position n takes output word n mod 4. */
static uint32_t position_word(uint64_t seed, uint32_t step, uint32_t gid, uint32_t n)
{
    uint32_t ctr[4] = { n >> 2, gid, step, 0u };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return out[n & 3u];
}

static uint32_t grid_phase_word(uint64_t seed, uint32_t step, uint32_t gid)
{
    uint32_t ctr[4] = { 0u, gid, step, 1u };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return out[0];
}

/* ------------------------------------------------------------------ */
/* keep ratio -> number of kept positions (Sec. 3.2.1: r = #kept / #all) */
/* ------------------------------------------------------------------ */

/* which member of the 2x2 grid family a ratio selects; 0 when none */
static int grid_family(double r)
{
    if (r == 0.25) return 1;
    if (r == 0.5)  return 2;
    if (r == 0.75) return 3;
    if (r == 1.0)  return 4;
    return 0;
}

/* is (h, w) kept by grid family member fam at phase p ? */
static int grid_keeps(int fam, uint32_t p, int64_t h, int64_t w)
{
    switch (fam) {
    case 1: return ((h & 1) == (int64_t)(p >> 1)) && ((w & 1) == (int64_t)(p & 1));
    case 2: return (((h + w) & 1) == (int64_t)p);
    case 3: return !(((h & 1) == (int64_t)(p >> 1)) && ((w & 1) == (int64_t)(p & 1)));
    case 4: return 1;
    }
    return 0;
}

/* is frame f kept by the lattice in time of family fam at phase p ?
 * r = 0.25: every fourth frame; r = 0.5: every second frame (phase 0 is the paper's
 * "even index on T", Sec. 3.2.1); r = 0.75: all but every fourth; r = 1: all. */
static int frame_keeps(int fam, uint32_t p, int64_t f)
{
    switch (fam) {
    case 1: return (f & 3) == (int64_t)p;
    case 2: return (f & 1) == (int64_t)p;
    case 3: return (f & 3) != (int64_t)p;
    case 4: return 1;
    }
    return 0;
}

/* Random mode: the exact per-sample count K = clamp(floor(r*N + 1/2), 1, N).
 * Grid mode: the largest count any phase can give (capacity per sample).
 * Returns -1 for arguments outside the method's domain. */
int64_t oracle_keep_count(int mode, int64_t H, int64_t W, double r)
{
    if (H <= 0 || W <= 0 || !(r > 0.0) || !(r <= 1.0)) return -1;
    int64_t N = H * W;
    if (mode == ORACLE_MASK_RANDOM) {
        int64_t K = (int64_t)floor(r * (double)N + 0.5);
        if (K < 1) K = 1;
        if (K > N) K = N;
        return K;
    }
    if (mode == ORACLE_MASK_TEMPORAL) {      /* K_T frames of H, each with all its W positions */
        int64_t KT = (int64_t)floor(r * (double)H + 0.5);
        if (KT < 1) KT = 1;
        if (KT > H) KT = H;
        return KT * W;
    }
    if (mode == ORACLE_MASK_TEMPORAL_GRID) {  /* capacity: the phase that keeps the most frames, times W */
        int fam = grid_family(r);
        if (!fam) return -1;
        int phases = (fam == 2) ? 2 : (fam == 4 ? 1 : 4);
        int64_t best = 0;
        for (int p = 0; p < phases; ++p) {
            int64_t cnt = 0;
            for (int64_t f = 0; f < H; ++f) cnt += frame_keeps(fam, (uint32_t)p, f);
            if (cnt > best) best = cnt;
        }
        return best * W;
    }
    if (mode == ORACLE_MASK_GRID) {
        int fam = grid_family(r);
        if (!fam) return -1;
        int phases = (fam == 2) ? 2 : (fam == 4 ? 1 : 4);
        int64_t best = 0;
        for (int p = 0; p < phases; ++p) {
            int64_t cnt = 0;
            for (int64_t h = 0; h < H; ++h)
                for (int64_t w = 0; w < W; ++w)
                    cnt += grid_keeps(fam, (uint32_t)p, h, w);
            if (cnt > best) best = cnt;
        }
        return best;
    }
    return -1;
}

/* ------------------------------------------------------------------ */
/* keep-index sampling (Sec. 4; Supp. A.4: one fresh mask per step)     */
/* ------------------------------------------------------------------ */

static int cmp_u64(const void* a, const void* b)
{
    uint64_t x = *(const uint64_t*)a, y = *(const uint64_t*)b;
    return (x > y) - (x < y);
}

/* Writes the global row ids b*N + n of the kept positions, ascending, and the
 * per-sample prefix keep_offsets[0..B].  Returns M_keep, or -1 on bad input.
 * Random mode: every position gets the 64-bit score (word << 32) | n; the K
 * positions with the smallest scores are kept (all K-subsets equally likely).
 * Grid mode: a periodic 2x2 lattice whose phase is drawn per sample.
 * Temporal mode (Sec. 3.1 and 3.2.1: a subset of video frames): H frames of W
 * positions; frame f gets the score (word << 32) | f from the same word stream as
 * position f of a random-mode map, the K_T frames with the smallest scores are
 * kept, each with all of its positions.
 * Temporal grid mode: frames on a lattice in time (every second or fourth frame, or
 * the complement), the phase drawn per sample like the spatial grid phase. */
int64_t oracle_sample_keep(int mode, int64_t B, int64_t H, int64_t W, double r,
                           uint64_t seed, uint64_t step, int64_t sample_offset,
                           uint32_t flags, int32_t* keep_rows, int32_t* keep_offsets)
{
    if (B <= 0 || H <= 0 || W <= 0) return -1;
    int64_t N = H * W;
    if (oracle_keep_count(mode, H, W, r) < 0) return -1;
    if (step >> 32) return -1;
    if (sample_offset < 0 || ((uint64_t)(sample_offset + B - 1) >> 32)) return -1;
    if (B * N >= ((int64_t)1 << 31)) return -1;

    int64_t out = 0;
    keep_offsets[0] = 0;
    if (mode == ORACLE_MASK_RANDOM) {
        int64_t K = oracle_keep_count(mode, H, W, r);
        uint64_t* score = (uint64_t*)malloc((size_t)N * sizeof(uint64_t));
        unsigned char* kept = (unsigned char*)malloc((size_t)N);
        for (int64_t b = 0; b < B; ++b) {
            uint32_t gid = (flags & ORACLE_FLAG_SHARE_MASK) ? 0u : (uint32_t)(sample_offset + b);
            for (int64_t n = 0; n < N; ++n) {
                uint64_t u = position_word(seed, (uint32_t)step, gid, (uint32_t)n);
                score[n] = (u << 32) | (uint64_t)n;
            }
            qsort(score, (size_t)N, sizeof(uint64_t), cmp_u64);
            memset(kept, 0, (size_t)N);
            for (int64_t k = 0; k < K; ++k) kept[score[k] & 0xffffffffu] = 1;
            for (int64_t n = 0; n < N; ++n)
                if (kept[n]) keep_rows[out++] = (int32_t)(b * N + n);
            keep_offsets[b + 1] = (int32_t)out;
        }
        free(score); free(kept);
    } else if (mode == ORACLE_MASK_TEMPORAL) {
        int64_t KT = oracle_keep_count(mode, H, W, r) / W;
        uint64_t* score = (uint64_t*)malloc((size_t)H * sizeof(uint64_t));
        unsigned char* kept = (unsigned char*)malloc((size_t)H);
        for (int64_t b = 0; b < B; ++b) {
            uint32_t gid = (flags & ORACLE_FLAG_SHARE_MASK) ? 0u : (uint32_t)(sample_offset + b);
            for (int64_t f = 0; f < H; ++f) {
                uint64_t u = position_word(seed, (uint32_t)step, gid, (uint32_t)f);
                score[f] = (u << 32) | (uint64_t)f;
            }
            qsort(score, (size_t)H, sizeof(uint64_t), cmp_u64);
            memset(kept, 0, (size_t)H);
            for (int64_t k = 0; k < KT; ++k) kept[score[k] & 0xffffffffu] = 1;
            for (int64_t f = 0; f < H; ++f)
                if (kept[f])
                    for (int64_t q = 0; q < W; ++q) keep_rows[out++] = (int32_t)(b * N + f * W + q);
            keep_offsets[b + 1] = (int32_t)out;
        }
        free(score); free(kept);
    } else if (mode == ORACLE_MASK_TEMPORAL_GRID) {
        /* frames on a lattice in time, the phase drawn per sample from the same word as the spatial grid phase */
        int fam = grid_family(r);
        uint32_t phases = (fam == 2) ? 2u : (fam == 4 ? 1u : 4u);
        for (int64_t b = 0; b < B; ++b) {
            uint32_t gid = (flags & ORACLE_FLAG_SHARE_MASK) ? 0u : (uint32_t)(sample_offset + b);
            uint32_t p = grid_phase_word(seed, (uint32_t)step, gid) % phases;
            for (int64_t f = 0; f < H; ++f)
                if (frame_keeps(fam, p, f))
                    for (int64_t q = 0; q < W; ++q) keep_rows[out++] = (int32_t)(b * N + f * W + q);
            keep_offsets[b + 1] = (int32_t)out;
        }
    } else {
        int fam = grid_family(r);
        uint32_t phases = (fam == 2) ? 2u : (fam == 4 ? 1u : 4u);
        for (int64_t b = 0; b < B; ++b) {
            uint32_t gid = (flags & ORACLE_FLAG_SHARE_MASK) ? 0u : (uint32_t)(sample_offset + b);
            uint32_t p = grid_phase_word(seed, (uint32_t)step, gid) % phases;
            for (int64_t h = 0; h < H; ++h)
                for (int64_t w = 0; w < W; ++w)
                    if (grid_keeps(fam, p, h, w)) keep_rows[out++] = (int32_t)(b * N + h * W + w);
            keep_offsets[b + 1] = (int32_t)out;
        }
    }
    return out;
}

/* ------------------------------------------------------------------ */
/* forward cache (Algorithm 1: only inputs[keep] is retained)           */
/* ------------------------------------------------------------------ */

/* Byte-exact row gather: X_keep[m, :] = X[keep_rows[m], :], rows of row_bytes. */
void oracle_forward_cache(const void* X, int64_t row_bytes, const int32_t* keep_rows,
                          int64_t M_keep, void* X_keep)
{
    for (int64_t m = 0; m < M_keep; ++m)
        memcpy((char*)X_keep + m * row_bytes,
               (const char*)X + (int64_t)keep_rows[m] * row_bytes, (size_t)row_bytes);
}

/* ------------------------------------------------------------------ */
/* forward of the layer (Eq. 2; with SBP every row is still computed,   */
/* Eq. 4 and Algorithm 1: only what is cached differs)                  */
/* ------------------------------------------------------------------ */

/* Y[m, j] = sum_i X[m, i] * W[i, j] (+ bias[j] when bias is not NULL), the sum over i
 * in ascending order.  X [M, C_in], W [C_in, C_out] row-major, Y [M, C_out]. */
void oracle_linear_forward(const double* X, const double* W, const double* bias,
                           int64_t M, int64_t C_in, int64_t C_out, double* Y)
{
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        double* y = Y + m * C_out;
        for (int64_t j = 0; j < C_out; ++j) y[j] = 0.0;
        for (int64_t i = 0; i < C_in; ++i) {
            double x = X[m * C_in + i];
            const double* w = W + i * C_out;
            for (int64_t j = 0; j < C_out; ++j) y[j] += x * w[j];
        }
        if (bias)
            for (int64_t j = 0; j < C_out; ++j) y[j] += bias[j];
    }
}

/* ------------------------------------------------------------------ */
/* SBP backward of a linear layer (Eq. 5; bias gradient by the same     */
/* masking of dY; nothing is rescaled, Eq. 1)                           */
/* ------------------------------------------------------------------ */

/* X_keep [M_keep, C_in], dY [M, C_out] (full; only kept rows are read),
 * W [C_in, C_out] row-major (Y = X W), keep_rows ascending global row ids.
 *   dW[i, j] = sum_m X_keep[m, i] * dY[keep_rows[m], j]
 *   db[j]    = sum_m dY[keep_rows[m], j]
 *   dX[keep_rows[m], i] = sum_j dY[keep_rows[m], j] * W[i, j];  other rows +0.0
 * Any of dW, db, dX may be NULL.  Sums run over m (resp. j) in ascending order. */
void oracle_linear_backward(const double* X_keep, const double* dY, const double* W,
                            const int32_t* keep_rows, int64_t M_keep, int64_t M,
                            int64_t C_in, int64_t C_out,
                            double* dW, double* db, double* dX)
{
    if (dW) {
        #pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < C_in; ++i) {
            double* dWi = dW + i * C_out;
            for (int64_t j = 0; j < C_out; ++j) dWi[j] = 0.0;
            for (int64_t m = 0; m < M_keep; ++m) {
                double x = X_keep[m * C_in + i];
                const double* g = dY + (int64_t)keep_rows[m] * C_out;
                for (int64_t j = 0; j < C_out; ++j) dWi[j] += x * g[j];
            }
        }
    }
    if (db) {
        for (int64_t j = 0; j < C_out; ++j) db[j] = 0.0;
        for (int64_t m = 0; m < M_keep; ++m) {
            const double* g = dY + (int64_t)keep_rows[m] * C_out;
            for (int64_t j = 0; j < C_out; ++j) db[j] += g[j];
        }
    }
    if (dX) {
        #pragma omp parallel for schedule(static)
        for (int64_t t = 0; t < M * C_in; ++t) dX[t] = 0.0;
        #pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M_keep; ++m) {
            const double* g = dY + (int64_t)keep_rows[m] * C_out;
            double* o = dX + (int64_t)keep_rows[m] * C_in;
            for (int64_t i = 0; i < C_in; ++i) {
                const double* w = W + i * C_out;
                double acc = 0.0;
                for (int64_t j = 0; j < C_out; ++j) acc += g[j] * w[j];
                o[i] = acc;
            }
        }
    }
}

/* Full backward of the same layer (Eq. 3): dW = X^T dY, db = column sums of
 * dY, dX = dY W^T, over all M rows. */
void oracle_full_backward(const double* X, const double* dY, const double* W,
                          int64_t M, int64_t C_in, int64_t C_out,
                          double* dW, double* db, double* dX)
{
    if (dW) {
        #pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < C_in; ++i) {
            double* dWi = dW + i * C_out;
            for (int64_t j = 0; j < C_out; ++j) dWi[j] = 0.0;
            for (int64_t m = 0; m < M; ++m) {
                double x = X[m * C_in + i];
                const double* g = dY + m * C_out;
                for (int64_t j = 0; j < C_out; ++j) dWi[j] += x * g[j];
            }
        }
    }
    if (db) {
        for (int64_t j = 0; j < C_out; ++j) db[j] = 0.0;
        for (int64_t m = 0; m < M; ++m)
            for (int64_t j = 0; j < C_out; ++j) db[j] += dY[m * C_out + j];
    }
    if (dX) {
        #pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m) {
            const double* g = dY + m * C_out;
            for (int64_t i = 0; i < C_in; ++i) {
                const double* w = W + i * C_out;
                double acc = 0.0;
                for (int64_t j = 0; j < C_out; ++j) acc += g[j] * w[j];
                dX[m * C_in + i] = acc;
            }
        }
    }
}

/* sets the number of threads the row loops use (for the single-thread baseline timing) */
void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* threads the row loops above will use */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* SBP on multi-head self-attention (Sec. 4, "How to apply SBP on MHSA?";   */
/* Supp. "Gradient Calculation of Attention Layers")                   */
/* ------------------------------------------------------------------ */
/*
 * One head of one sample, with the gradient path restricted to a set Zq of query tokens and a set Zk
 * of key / value tokens (both given as per-sample lists of global row ids, as the sampler writes them):
 *
 *   forward (the supplementary's attention equation on the chosen tokens):
 *     M_ij = q_i . k_j / sqrt(d)      i in Zq, j in Zk
 *     S_i: = softmax_j(M_i:)          over j in Zk
 *     A_i  = sum_j S_ij v_j
 *   backward (the supplementary's gradients of query, key and value, dQ = dM K / sqrt(d),
 *   dK = Q^T dM / sqrt(d), dV = S^T dA, with the derivative of the row softmax between dS and dM):
 *     dS_ij = dA_i . v_j
 *     dM_ij = S_ij (dS_ij - sum_l S_il dS_il)
 *     dQ_i  = sum_j dM_ij k_j / sqrt(d);  dK_j = sum_i dM_ij q_i / sqrt(d);  dV_j = sum_i S_ij dA_i
 *   rows outside Zq (dQ) or Zk (dK, dV) receive +0.0: their gradient is dropped.
 *
 * Zq = kept tokens, Zk = all tokens is the paper's "Drop Query only" (its worked derivation: dM of the
 * dropped queries is zero, dQ is exact on the kept rows, dK = Q_keep^T dM_keep / sqrt(d)); Zq = Zk = kept
 * tokens is "Drop QKV", read as attention among the kept tokens (the reading of Algorithm 1 applied to the
 * attention operation, whose cached maps are the r^2 n^2 ones of the paper's memory formula); Zq = Zk = all
 * tokens is ordinary attention.  Matrices are [M, heads * d] row-major, head hh in columns [hh*d, (hh+1)*d).
 */
void oracle_attention_forward(const double* Q, const double* K, const double* V,
                              const int32_t* q_rows, const int32_t* q_offs,
                              const int32_t* k_rows, const int32_t* k_offs,
                              int64_t B, int64_t M, int64_t heads, int64_t d, double* A)
{
    const int64_t C = heads * d;
    const double scale = 1.0 / sqrt((double)d);
    for (int64_t e = 0; e < M * C; ++e) A[e] = 0.0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t hh = 0; hh < heads; ++hh) {
            const int64_t nk = k_offs[b + 1] - k_offs[b];
            double* s = (double*)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
            for (int64_t a = q_offs[b]; a < q_offs[b + 1]; ++a) {
                const double* q = Q + (int64_t)q_rows[a] * C + hh * d;
                double mx = -INFINITY;
                for (int64_t j = 0; j < nk; ++j) {
                    const double* k = K + (int64_t)k_rows[k_offs[b] + j] * C + hh * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += q[c] * k[c];
                    s[j] = acc * scale;
                    if (s[j] > mx) mx = s[j];
                }
                double sum = 0.0;
                for (int64_t j = 0; j < nk; ++j) { s[j] = exp(s[j] - mx); sum += s[j]; }
                double* out = A + (int64_t)q_rows[a] * C + hh * d;
                for (int64_t j = 0; j < nk; ++j) {
                    const double* v = V + (int64_t)k_rows[k_offs[b] + j] * C + hh * d;
                    const double p = s[j] / sum;
                    for (int64_t c = 0; c < d; ++c) out[c] += p * v[c];
                }
            }
            free(s);
        }
}

void oracle_attention_backward(const double* Q, const double* K, const double* V, const double* dA,
                               const int32_t* q_rows, const int32_t* q_offs,
                               const int32_t* k_rows, const int32_t* k_offs,
                               int64_t B, int64_t M, int64_t heads, int64_t d,
                               double* dQ, double* dK, double* dV)
{
    const int64_t C = heads * d;
    const double scale = 1.0 / sqrt((double)d);
    for (int64_t e = 0; e < M * C; ++e) { dQ[e] = 0.0; dK[e] = 0.0; dV[e] = 0.0; }
    /* one (sample, head) pair touches only its own rows and columns: the pairs are independent */
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t hh = 0; hh < heads; ++hh) {
            const int64_t nk = k_offs[b + 1] - k_offs[b];
            double* p = (double*)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
            double* ds = (double*)malloc(sizeof(double) * (size_t)(nk > 0 ? nk : 1));
            for (int64_t a = q_offs[b]; a < q_offs[b + 1]; ++a) {
                const int64_t qi = (int64_t)q_rows[a] * C + hh * d;
                double mx = -INFINITY;
                for (int64_t j = 0; j < nk; ++j) {
                    const double* k = K + (int64_t)k_rows[k_offs[b] + j] * C + hh * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += Q[qi + c] * k[c];
                    p[j] = acc * scale;
                    if (p[j] > mx) mx = p[j];
                }
                double sum = 0.0;
                for (int64_t j = 0; j < nk; ++j) { p[j] = exp(p[j] - mx); sum += p[j]; }
                double delta = 0.0;
                for (int64_t j = 0; j < nk; ++j) {
                    const double* v = V + (int64_t)k_rows[k_offs[b] + j] * C + hh * d;
                    p[j] /= sum;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += dA[qi + c] * v[c];
                    ds[j] = acc;
                    delta += p[j] * acc;
                }
                for (int64_t j = 0; j < nk; ++j) {
                    const int64_t kj = (int64_t)k_rows[k_offs[b] + j] * C + hh * d;
                    const double dm = p[j] * (ds[j] - delta);
                    for (int64_t c = 0; c < d; ++c) {
                        dQ[qi + c] += dm * K[kj + c] * scale;
                        dK[kj + c] += dm * Q[qi + c] * scale;
                        dV[kj + c] += p[j] * dA[qi + c];
                    }
                }
            }
            free(p);
            free(ds);
        }
}

/*
 * Cached activations of an attention layer under SBP relative to full backpropagation, counted term by term as
 * the paper lists them (Sec. 4): QKV vectors h d n each, attention maps before and after the softmax h n n each.
 *   mode 0, Drop Query only: K and V whole, Q and both maps at keep ratio r:  (2 + r) h d n + 2 r h n n
 *   mode 1, Drop QKV:        Q, K, V at r, both maps at r^2:                   3 r h d n + 2 r^2 h n n
 * over 3 h d n + 2 h n n.
 */
double oracle_attention_memory_ratio(int mode, double d, double n, double r)
{
    const double full = 3.0 * d * n + 2.0 * n * n;
    if (mode == 0) return ((2.0 + r) * d * n + 2.0 * r * n * n) / full;
    return (3.0 * r * d * n + 2.0 * r * r * n * n) / full;
}

/* ------------------------------------------------------------------ */
/* Convolution with stride >= kernel size under SBP (Sec. 3.2.2, the   */
/* text after Eq. 6: with s >= k the neighbour effect disappears and   */
/* the layer behaves like a point-wise one; ConvNeXt's 2 x 2 / stride 2 */
/* down-sampling layers, Sec. 5)                                        */
/* ------------------------------------------------------------------ */
/*
 * Channels-last tensors: X [B, H, W, C], weights Wt [k, k, C, Co], Y and dY [B, Ho, Wo, Co] with
 * Ho = (H - k) / s + 1, Wo = (W - k) / s + 1 (no padding), s >= k:
 *   Y[b, ho, wo, j] = sum_{dh, dw, c} X[b, s ho + dh, s wo + dw, c] Wt[dh, dw, c, j] (+ bias[j])
 * Every output position reads its own k x k patch; patches of different output positions do not overlap.
 * Backward (Eq. 6 written out for this case) with dY dropped outside the kept output positions
 * (keep_rows: ascending global ids (b Ho + ho) Wo + wo):
 *   dW[dh, dw, c, j] = sum_{kept m} X[patch of m at (dh, dw), c] dY[m, j]
 *   db[j]            = sum_{kept m} dY[m, j]
 *   dX[patch of m at (dh, dw), c] = sum_j dY[m, j] Wt[dh, dw, c, j]   for kept m; every other input position +0.0
 */
void oracle_patch_conv_forward(const double* X, const double* Wt, const double* bias, int64_t B, int64_t H,
                               int64_t W, int64_t C, int64_t Co, int64_t k, int64_t s, double* Y)
{
    const int64_t Ho = (H - k) / s + 1, Wo = (W - k) / s + 1;
#pragma omp parallel for collapse(2)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t ho = 0; ho < Ho; ++ho)
            for (int64_t wo = 0; wo < Wo; ++wo) {
                double* y = Y + ((b * Ho + ho) * Wo + wo) * Co;
                for (int64_t j = 0; j < Co; ++j) y[j] = bias ? bias[j] : 0.0;
                for (int64_t dh = 0; dh < k; ++dh)
                    for (int64_t dw = 0; dw < k; ++dw) {
                        const double* x = X + ((b * H + s * ho + dh) * W + s * wo + dw) * C;
                        const double* w = Wt + (dh * k + dw) * C * Co;
                        for (int64_t c = 0; c < C; ++c)
                            for (int64_t j = 0; j < Co; ++j) y[j] += x[c] * w[c * Co + j];
                    }
            }
}

void oracle_patch_conv_backward(const double* X, const double* dY, const double* Wt, const int32_t* keep_rows,
                                int64_t M_keep, int64_t B, int64_t H, int64_t W, int64_t C, int64_t Co,
                                int64_t k, int64_t s, double* dW, double* db, double* dX)
{
    const int64_t Ho = (H - k) / s + 1, Wo = (W - k) / s + 1;
    if (dW) for (int64_t e = 0; e < k * k * C * Co; ++e) dW[e] = 0.0;
    if (db) for (int64_t j = 0; j < Co; ++j) db[j] = 0.0;
    if (dX) for (int64_t e = 0; e < B * H * W * C; ++e) dX[e] = 0.0;
    for (int64_t m = 0; m < M_keep; ++m) {
        const int64_t g = keep_rows[m];
        const int64_t b = g / (Ho * Wo), ho = (g / Wo) % Ho, wo = g % Wo;
        const double* dy = dY + g * Co;
        if (db) for (int64_t j = 0; j < Co; ++j) db[j] += dy[j];
        for (int64_t dh = 0; dh < k; ++dh)
            for (int64_t dw = 0; dw < k; ++dw) {
                const int64_t pix = (b * H + s * ho + dh) * W + s * wo + dw;
                const double* w = Wt + (dh * k + dw) * C * Co;
                for (int64_t c = 0; c < C; ++c) {
                    if (dW) for (int64_t j = 0; j < Co; ++j) dW[((dh * k + dw) * C + c) * Co + j] += X[pix * C + c] * dy[j];
                    if (dX) {
                        double acc = 0.0;
                        for (int64_t j = 0; j < Co; ++j) acc += dy[j] * w[c * Co + j];
                        dX[pix * C + c] = acc;
                    }
                }
            }
    }
}

/* ------------------------------------------------------------------ */
/* Position-wise activation between two SBP layers of a block (Sec. 3.3.1; */
/* the supplementary's chain rule for transformer blocks): element-wise,   */
/* so it acts on the kept rows alone.  GELU in its exact form,             */
/* gelu(z) = z Phi(z),  gelu'(z) = Phi(z) + z phi(z).                      */
/* ------------------------------------------------------------------ */
void oracle_gelu(const double* z, int64_t n, double* out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = 0.5 * z[i] * (1.0 + erf(z[i] / sqrt(2.0)));
}

void oracle_act_backward_gelu(const double* z, const double* dh, int64_t n, double* dz)
{
    const double inv_sqrt_2pi = 1.0 / sqrt(2.0 * acos(-1.0));
    for (int64_t i = 0; i < n; ++i) {
        const double Phi = 0.5 * (1.0 + erf(z[i] / sqrt(2.0)));
        const double phi = inv_sqrt_2pi * exp(-0.5 * z[i] * z[i]);
        dz[i] = dh[i] * (Phi + z[i] * phi);
    }
}
