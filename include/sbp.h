/*
 * sbp.h - C ABI of the B200 (sm_100a) Stochastic Backpropagation linear-layer library.
 *
 * Stochastic Backpropagation (SBP; "An In-depth Study of Stochastic
 * Backpropagation", arXiv 2210.00129) runs the forward pass of a linear /
 * point-wise layer on every spatial position but caches, and back-propagates
 * through, only a randomly kept subset of positions.  This library is the hot
 * path of that method for one layer Y = X W:
 *
 *   sbp_sample_keep      draw the kept positions of every sample      (Sec. 3.2.1, Sec. 4)
 *   sbp_forward_cache    X_keep = X[keep_rows, :]                     (Algorithm 1)
 *   sbp_linear_forward   Y = X W + b, with that cache written by the same launch (Eq. 2)
 *   sbp_linear_backward  dW = X_keep^T dY_keep, db = sum dY_keep,
 *                        dX = scatter(dY_keep W^T), zeros elsewhere   (Eq. 5)
 *   sbp_attention_backward  dQ, dK, dV of attention on the kept tokens (Sec. 4, Drop QKV / Drop Query only)
 *   sbp_act_backward     dZ = dH * gelu'(Z_keep) on packed rows between two layers of a block (Sec. 3.3.1)
 *   sbp_patch_cache / sbp_patch_scatter  stride >= kernel convolutions as linear layers on patch rows (Sec. 3.2.2)
 *
 * Nothing is rescaled by 1/r: Eq. 1 keeps the plain 1/B factor.
 *
 * Conventions
 *   - M = B*N rows, N = H*W positions per sample, row id = b*N + h*W + w.
 *   - All matrices are row-major, dense (no padding), inner stride 1.
 *     W is [C_in, C_out] (the paper's orientation, Y = X W) unless SBP_FLAG_W_OUT_IN says otherwise.
 *   - "dev" pointers are CUDA device pointers owned by the caller; the library
 *     allocates and frees nothing and keeps no pointer after a call returns.
 *     Device buffers must be 16-byte aligned.
 *   - Calls enqueue work on the caller's stream (a cudaStream_t passed as
 *     void*, NULL = default stream) and return without synchronising.
 *   - Errors detectable on the host are returned before anything is launched.
 *     Conditions only the device can see (bad indices under SBP_FLAG_VALIDATE,
 *     a bounded wait that ran out) are written to the optional status word.
 *   - No call throws; every call returns an sbp_status.
 */
#ifndef SBP_H_
#define SBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SBP_OK = 0,
    SBP_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, size or ratio out of range */
    SBP_ERR_UNSUPPORTED = 2,   /* valid request this build has no kernel for */
    SBP_ERR_WORKSPACE = 3,     /* workspace missing or too small */
    SBP_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed */
    SBP_ERR_TIMEOUT = 5,       /* device status word: a bounded wait inside a kernel expired */
    SBP_ERR_BAD_INDICES = 6    /* device status word: keep_rows not ascending / out of range */
} sbp_status;

typedef enum { SBP_F32 = 0, SBP_BF16 = 1 } sbp_dtype;

/* position-wise activations sbp_act_backward knows */
typedef enum { SBP_ACT_GELU = 0 /* exact form: z Phi(z) */ } sbp_activation;

/* Sec. 4, "How to sample the gradient keep mask?": uniformly random positions,
 * or a structured periodic ("grid-wise") mask. */
typedef enum { SBP_MASK_RANDOM = 0, SBP_MASK_GRID = 1, SBP_MASK_TEMPORAL = 2, SBP_MASK_TEMPORAL_GRID = 3 } sbp_mask_mode;

enum {
    SBP_FLAG_SHARE_MASK = 1,  /* every sample of the call uses sample 0's mask (one mask per iteration, Supp. A.4) */
    SBP_FLAG_ACCUMULATE = 2,  /* dW += and db += instead of overwrite (gradient accumulation) */
    SBP_FLAG_VALIDATE = 4,    /* check keep_rows on the device before use; result in the status word */
    SBP_FLAG_PLAIN_FMA = 8,   /* bf16 only: use the CUDA-core FMA kernels instead of the tensor-core ones */
    SBP_FLAG_DY_COMPACT = 16, /* dY holds only the kept rows, packed: [M_keep_cap, C_out] (chained layers, Sec. 3.3.1) */
    SBP_FLAG_DX_COMPACT = 32, /* dX receives only the kept rows, packed: [M_keep_cap, C_in]; no zero rows are written */
    SBP_FLAG_W_OUT_IN = 64,   /* W, and dW, are stored [C_out, C_in] (the usual layout of framework linear layers) */
    SBP_FLAG_ATTN_ALL_KEYS = 128, /* sbp_attention_backward: keys and values are all tokens, only queries are dropped */
    SBP_FLAG_ATTN_KEPT_ROWS_ONLY = 256 /* sbp_attention_backward: write only the rows in the token lists, leave every other row alone */
};

const char* sbp_status_string(sbp_status s);

/*
 * Kept positions per sample for keep ratio r = #kept / #all (Sec. 3.2.1).
 * Pure host function.
 *   SBP_MASK_RANDOM: the exact count K = clamp(floor(r*H*W + 1/2), 1, H*W).
 *   SBP_MASK_GRID:   the largest count any phase of the mask gives (buffer capacity
 *                    per sample); r must be one of 0.25, 0.5, 0.75, 1.0.
 *   SBP_MASK_TEMPORAL: H is the number of frames, W the positions per frame;
 *                    clamp(floor(r*H + 1/2), 1, H) whole frames, times W.
 *   SBP_MASK_TEMPORAL_GRID: as SBP_MASK_GRID in time: the largest frame count any phase
 *                    gives, times W; r must be one of 0.25, 0.5, 0.75, 1.0.
 * Returns -1 when H, W <= 0, r outside (0, 1], or the ratio has no grid mask.
 */
int64_t sbp_keep_count(sbp_mask_mode mode, int64_t H, int64_t W, double keep_ratio);

/*
 * Draw the keep set of each of B samples (Sec. 3.2.1 index sets; Sec. 4 masks;
 * Supp. A.4: a fresh mask every training step).
 *
 * SBP_MASK_RANDOM: position n of global sample g = sample_offset + b gets the
 *   32-bit word u = Philox4x32-10(counter = {n/4, g, step, 0}, key = seed)[n mod 4];
 *   the K positions with the smallest 64-bit scores (u << 32 | n) are kept, so
 *   every K-subset is equally likely.  Pass H = N, W = 1 for unstructured rows.
 * SBP_MASK_GRID: a 2x2-periodic lattice with a random phase p per sample,
 *   p = Philox4x32-10({0, g, step, 1}, seed)[0] mod (#phases):
 *     r = 0.25  keep (h mod 2, w mod 2) == (p / 2, p mod 2)      (4 phases)
 *     r = 0.5   keep (h + w) mod 2 == p                           (2 phases)
 *     r = 0.75  complement of the r = 0.25 mask                   (4 phases)
 *     r = 1.0   keep everything
 * SBP_MASK_TEMPORAL (video: the kept subset is a subset of frames, Sec. 3.1 and the
 *   frame example of Sec. 3.2.1): a sample is H frames of W positions; frame f gets
 *   the word of position f above, the K_T frames with the smallest scores are kept,
 *   each with all W positions (rows (b*H + f)*W + q).  At most 2048 frames
 *   (SBP_ERR_UNSUPPORTED beyond).
 * SBP_MASK_TEMPORAL_GRID (the "even index on T" example of Sec. 3.2.1): frames on a
 *   lattice in time with a random phase p per sample, p drawn as for SBP_MASK_GRID:
 *     r = 0.25  keep f mod 4 == p;  r = 0.5  keep f mod 2 == p (p = 0: the even frames);
 *     r = 0.75  keep f mod 4 != p;  r = 1.0  keep every frame.
 *   Counts depend on the phase when H is not a multiple of the period: read M_keep from
 *   keep_offsets[B].
 * The mask depends only on (seed, step, g, n): it does not change with how a
 * batch is split over calls or devices.
 *
 * Outputs (dev): keep_rows, capacity B * sbp_keep_count(...), receives the global
 * row ids b*N + n of kept positions in ascending order (entries past the total
 * are left untouched); keep_offsets[B + 1] receives the per-sample prefix,
 * keep_offsets[B] = M_keep.
 *
 * Errors: SBP_ERR_INVALID_ARG for null/misaligned outputs, B, H, W <= 0,
 * B*H*W >= 2^31, r outside (0, 1], step >= 2^32, sample ids >= 2^32 or < 0;
 * SBP_ERR_UNSUPPORTED for a grid ratio outside the four above;
 * SBP_ERR_CUDA if the launch fails.
 */
sbp_status sbp_sample_keep(sbp_mask_mode mode, int64_t B, int64_t H, int64_t W,
                           double keep_ratio, uint64_t seed, uint64_t step,
                           int64_t sample_offset, uint32_t flags,
                           int32_t* keep_rows /* dev */, int32_t* keep_offsets /* dev */,
                           void* stream);

/*
 * Forward cache (Algorithm 1: only inputs[keep] is retained for backward):
 *   X_keep[m, :] = X[keep_rows[m], :]   for m < M_keep, a bit-exact copy.
 * X is [M, C]; X_keep is [M_keep_cap, C]; rows M_keep <= m < M_keep_cap are set
 * to zero (sbp_linear_backward relies on those padding rows being finite).
 * M_keep is *M_keep_dev when that device pointer is non-NULL (e.g. &keep_offsets[B]),
 * else M_keep_cap.  Dropped rows of X are never read.
 * Requires C * sizeof(element) to be a multiple of 16 (else SBP_ERR_UNSUPPORTED).
 * keep_rows entries must lie in [0, M); they are not checked here.
 */
sbp_status sbp_forward_cache(sbp_dtype dt, const void* X /* dev */, int64_t M, int64_t C,
                             const int32_t* keep_rows /* dev */,
                             const int32_t* M_keep_dev /* dev, nullable */,
                             int64_t M_keep_cap, void* X_keep /* dev */, void* stream);

/*
 * Forward of the layer with the SBP cache fused in (Eq. 2: Y = X W; with SBP every
 * row is still computed, Eq. 4, and only the kept rows of the input are retained for
 * the backward pass, Algorithm 1):
 *   Y[m, j]      = sum_i X[m, i] * W[i, j] + bias[j]            dt [M, C_out]
 *   X_keep[m, :] = X[keep_rows[m], :] for m < M_keep, zero rows up to M_keep_cap
 * X [M, C_in], W [C_in, C_out], bias fp32 [C_out] or NULL.  X_keep may be NULL (no
 * cache: keep_rows and M_keep_dev are then ignored); otherwise it is what
 * sbp_forward_cache would produce, written by the same launch so that X is read
 * from memory once.  SBP_BF16: bf16 inputs and output, fp32 accumulation on the
 * tensor cores, one rounding of (sum + bias) to bf16.  SBP_F32: fp32 FMA arithmetic.
 * C_in and C_out must be multiples of 8 (bf16) / 4 (fp32), else SBP_ERR_UNSUPPORTED.
 * flags: SBP_FLAG_PLAIN_FMA, SBP_FLAG_W_OUT_IN (W is [C_out, C_in]; read in place, no
 * copy) or 0.  status_word as for sbp_linear_backward.
 * SBP_ERR_INVALID_ARG for null or misaligned (16 bytes) pointers and bad sizes.
 */
sbp_status sbp_linear_forward(sbp_dtype dt, const void* X /* dev */, const void* W /* dev */,
                              const float* bias /* dev, nullable */, int64_t M, int64_t C_in, int64_t C_out,
                              void* Y /* dev */, const int32_t* keep_rows /* dev, nullable with X_keep */,
                              const int32_t* M_keep_dev /* dev, nullable */, int64_t M_keep_cap,
                              void* X_keep /* dev, nullable */, uint32_t flags,
                              int32_t* status_word /* dev, nullable */, void* stream);

/* Scratch bytes sbp_linear_backward needs for these sizes, whatever flags the call uses (never 0):
 * partial sums of split reductions, and room for one copy of W and of dW for SBP_FLAG_W_OUT_IN. */
size_t sbp_linear_backward_workspace_bytes(sbp_dtype dt, int64_t M, int64_t M_keep_cap,
                                           int64_t C_in, int64_t C_out);

/*
 * SBP backward of one linear layer (Eq. 5 and the text after it; bias gradient
 * by the same masking of dY; no rescaling, Eq. 1):
 *   dW[i, j]            = sum_{m < M_keep} X_keep[m, i] * dY[keep_rows[m], j]     fp32 [C_in, C_out]
 *   db[j]               = sum_{m < M_keep} dY[keep_rows[m], j]                    fp32 [C_out]
 *   dX[keep_rows[m], :] = dY[keep_rows[m], :] * W^T                                dt   [M, C_in]
 *   every other row of dX = +0.0
 * Inputs: X_keep [M_keep_cap, C_in] (from sbp_forward_cache; rows past M_keep must
 * be finite), dY [M, C_out] (the full upstream gradient; only kept rows are read),
 * W [C_in, C_out], keep_rows strictly ascending ids in [0, M).  M_keep is
 * *M_keep_dev if non-NULL, else M_keep_cap.  Any of dW, db, dX may be NULL to skip
 * that product.
 *
 * Chained layers (Sec. 3.3.1, Eq. 9: with the same keep set on consecutive point-wise
 * layers the kept and dropped sets pass through unchanged, so the gradient between
 * them is non-zero only in the kept rows).  Such a block can keep that gradient
 * packed: SBP_FLAG_DX_COMPACT makes this call write dX[m, :] = dY_row(m) * W^T into a
 * [M_keep_cap, C_in] tensor (rows in [M_keep, M_keep_cap) are zeroed, no other zeros
 * are written), and SBP_FLAG_DY_COMPACT makes it read row m of a [M_keep_cap, C_out]
 * dY instead of row keep_rows[m] of the full one.  The layer at the block's boundary
 * uses neither flag on its side facing the rest of the network.  With both flags
 * keep_rows is not used and may be NULL.
 *
 * Weight layout.  The paper writes Y = X W with W [C_in, C_out] (Sec. 3.2.1), and that
 * is the native layout here.  With SBP_FLAG_W_OUT_IN both W and dW are [C_out, C_in]
 * (dW[j, i] as above with the indices swapped): W is transposed into the workspace
 * before the products and dW is transposed out of it after them (two small extra
 * launches); the results are the same numbers.
 *
 * SBP_BF16: inputs bf16, products accumulated in fp32 on the tensor cores, dX
 * rounded to bf16 (nearest even).  SBP_F32: plain fp32 FMA arithmetic.
 * C_in and C_out must be multiples of 8 (bf16) / 4 (fp32), else SBP_ERR_UNSUPPORTED.
 *
 * flags: SBP_FLAG_ACCUMULATE adds into dW and db; SBP_FLAG_VALIDATE first checks
 * keep_rows on the device and, on failure, writes SBP_ERR_BAD_INDICES to
 * *status_word and makes the compute kernels return without touching outputs
 * (needs a status word); SBP_FLAG_PLAIN_FMA forces the CUDA-core kernels.
 * workspace: at least sbp_linear_backward_workspace_bytes(...) bytes, 256-byte
 * aligned, used only during the call's kernels (SBP_ERR_WORKSPACE if short).
 * status_word (dev, nullable): must be zero before the call; receives the first
 * device-side error (SBP_ERR_TIMEOUT, SBP_ERR_BAD_INDICES), else stays zero.
 * Results are deterministic: no floating-point atomics are used.
 */
sbp_status sbp_linear_backward(sbp_dtype dt,
                               const void* X_keep /* dev */, const void* dY /* dev */,
                               const void* W /* dev */,
                               const int32_t* keep_rows /* dev */,
                               const int32_t* M_keep_dev /* dev, nullable */,
                               int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out,
                               float* dW /* dev, nullable */, float* db /* dev, nullable */,
                               void* dX /* dev, nullable */,
                               uint32_t flags, void* workspace /* dev */, size_t workspace_bytes,
                               int32_t* status_word /* dev, nullable */, void* stream);

/*
 * Number of kernels one sbp_linear_backward call with these arguments enqueues (diagnostic,
 * pure host function; the paper has no counterpart).  want_* select the outputs requested.
 */
int sbp_linear_backward_kernel_count(sbp_dtype dt, int64_t M, int64_t M_keep_cap, int64_t C_in,
                                     int64_t C_out, int want_dW, int want_db, int want_dX,
                                     uint32_t flags);

/*
 * Backward of a position-wise activation between two SBP layers that share a keep set (Sec. 3.3.1 and the
 * supplementary's chain rule for transformer blocks: kept positions stay kept and dropped ones stay dropped through
 * position-wise operations, so inside an MLP block - linear, GELU, linear - the gradient can stay packed):
 *   dZ[m, c] = dH[m, c] * act'(Z_keep[m, c])   for m < M_keep;  rows [M_keep, M_keep_cap) of dZ = 0
 * Z_keep [M_keep_cap, C]: the cached pre-activation rows of the kept positions (what sbp_forward_cache or
 * sbp_linear_forward's cache holds for the layer behind the activation); dH [M_keep_cap, C]: the packed gradient of
 * the activation's output (the SBP_FLAG_DX_COMPACT output of the layer above); dZ [M_keep_cap, C]: the packed gradient
 * of its input (the SBP_FLAG_DY_COMPACT input of the layer below); dZ may alias dH.  SBP_ACT_GELU:
 * gelu'(z) = (1 + erf(z / sqrt 2)) / 2 + z exp(-z^2 / 2) / sqrt(2 pi).  Arithmetic in fp32, one rounding to dt.
 * C * sizeof(element) must be a multiple of 16 (else SBP_ERR_UNSUPPORTED); other activations SBP_ERR_UNSUPPORTED.
 */
sbp_status sbp_act_backward(sbp_dtype dt, sbp_activation act, const void* Z_keep /* dev */, const void* dH /* dev */,
                            const int32_t* M_keep_dev /* dev, nullable */, int64_t M_keep_cap, int64_t C,
                            void* dZ /* dev */, int32_t* status_word /* dev, nullable */, void* stream);

/*
 * Convolutions with stride >= kernel size as SBP layers (Sec. 3.2.2, the text after Eq. 6: with s >= k the
 * neighbour effect disappears and the layer behaves like a point-wise one; ConvNeXt's 2 x 2 / stride 2
 * down-sampling layers, Sec. 5).  Channels-last X [B, H, W, C], weights [k, k, C, C_out] = a [k*k*C, C_out]
 * matrix, output grid Ho = (H - k) / stride + 1, Wo = (W - k) / stride + 1 (no padding); keep_rows are kept
 * OUTPUT positions (b*Ho + ho)*Wo + wo, as sbp_sample_keep draws them on an Ho x Wo map.  Each output position
 * reads its own k x k patch, so the layer is a linear layer on patch rows of k*k*C values (ordered dh, dw, c):
 *
 *   sbp_patch_cache     X_keep[m, (dh, dw, c)] = X[b, stride*ho + dh, stride*wo + dw, c]  for kept m = (b, ho, wo);
 *                       [M_keep_cap, k*k*C], rows past M_keep zeroed: the forward cache (Algorithm 1)
 *   sbp_linear_backward with C_in = k*k*C on X_keep, dY [B*Ho*Wo, C_out] and SBP_FLAG_DX_COMPACT: dW, db and the
 *                       packed input gradient dX_patches [M_keep_cap, k*k*C]
 *   sbp_patch_scatter   dX[b, stride*ho + dh, stride*wo + dw, c] = dX_patches[m, (dh, dw, c)] for kept m; every
 *                       other input position (dropped patches, positions no patch covers) = +0.0.  Every element
 *                       of dX is written exactly once.  workspace: sbp_patch_scatter_workspace_bytes(...) bytes,
 *                       256-byte aligned (one int32 per output position).
 * C * sizeof(element) must be a multiple of 16 (else SBP_ERR_UNSUPPORTED); stride < k, k larger than the map and
 * other bad sizes or pointers give SBP_ERR_INVALID_ARG; a short workspace SBP_ERR_WORKSPACE.  M_keep is
 * *M_keep_dev when given, else M_keep_cap.  Bit-exact copies; deterministic.
 */
sbp_status sbp_patch_cache(sbp_dtype dt, const void* X /* dev */, int64_t B, int64_t H, int64_t W, int64_t C,
                           int64_t k, int64_t stride, const int32_t* keep_rows /* dev */,
                           const int32_t* M_keep_dev /* dev, nullable */, int64_t M_keep_cap, void* X_keep /* dev */,
                           void* stream);
size_t sbp_patch_scatter_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t k, int64_t stride);
sbp_status sbp_patch_scatter(sbp_dtype dt, const void* dX_patches /* dev */, int64_t B, int64_t H, int64_t W, int64_t C,
                             int64_t k, int64_t stride, const int32_t* keep_rows /* dev */,
                             const int32_t* M_keep_dev /* dev, nullable */, int64_t M_keep_cap, void* dX /* dev */,
                             void* workspace /* dev */, size_t workspace_bytes, int32_t* status_word /* dev, nullable */,
                             void* stream);

/*
 * SBP backward of multi-head scaled dot-product attention (Sec. 4, "How to apply SBP on MHSA?"; supplementary,
 * "Gradient Calculation of Attention Layers": A = softmax(Q K^T / sqrt(d)) V per head, dQ = dM K / sqrt(d),
 * dK = Q^T dM / sqrt(d), dV = S^T dA), with the gradient path restricted to token subsets.  Per sample b and head,
 * with Zq the query tokens of the sample listed in q_rows and Zk its key / value tokens:
 *   S_ij  = softmax over j in Zk of q_i . k_j / sqrt(d)                 i in Zq   (recomputed; no attention map is cached)
 *   dS_ij = dA_i . v_j,   dM_ij = S_ij (dS_ij - sum_l S_il dS_il)
 *   dQ_i  = sum_j dM_ij k_j / sqrt(d),  dK_j = sum_i dM_ij q_i / sqrt(d),  dV_j = sum_i S_ij dA_i
 *   rows of dQ outside Zq and rows of dK, dV outside Zk = +0.0 (their gradient is dropped); with
 *   SBP_FLAG_ATTN_KEPT_ROWS_ONLY those rows are not written at all - enough when the outputs feed an
 *   sbp_linear_backward with the same keep list, which reads the kept rows only
 * Which subsets:
 *   Drop QKV (what the paper applies to image transformers): kv_rows = NULL, flags = 0: Zk = Zq = the kept tokens;
 *     the gradient path is attention among the kept tokens (the wrapped-operation reading of Algorithm 1; its maps
 *     are the r^2 n^2 ones of the paper's memory formula).
 *   Drop Query only (the supplementary's worked derivation): SBP_FLAG_ATTN_ALL_KEYS: Zk = all N tokens; dQ is the exact
 *     gradient on the kept rows, dK = Q_keep^T dM_keep / sqrt(d), dV = S_keep^T dA_keep (dA is read on kept rows only:
 *     inside a block that drops the same tokens everywhere its other rows are zero).
 *   kv_rows / kv_offsets given: any other pair of subsets.  q_rows = NULL: every token is a query (with
 *     SBP_FLAG_ATTN_ALL_KEYS this is ordinary attention backward, keep ratio 1).
 * Layout: Q, K, V [B*N, ld_qkv] and dQ, dK, dV [B*N, ld_out] hold head hh in columns [hh*d, (hh+1)*d) from their
 * own base pointers, so the three slices of a fused [B*N, 3*heads*d] projection output can be passed with
 * ld = 3*heads*d; dA [B*N, ld_da] likewise.  q_rows / q_offsets (and kv_*) are lists as sbp_sample_keep writes them:
 * ascending global row ids b*N + n and B + 1 offsets; max_kept = the largest per-sample count any list may hold
 * (e.g. sbp_keep_count(...)), ignored when no list is given.
 * This build: SBP_BF16 with d = 64, at most 256 tokens of a sample on either side (N <= 256 where a side takes all
 * tokens), leading dimensions multiples of 8: otherwise SBP_ERR_UNSUPPORTED.  P = S and dM are rounded to bf16
 * between the products, accumulation is fp32.  SBP_ERR_INVALID_ARG for null / misaligned pointers and bad sizes.
 * status_word as for sbp_linear_backward.  Deterministic.
 */
sbp_status sbp_attention_backward(sbp_dtype dt, const void* Q /* dev */, const void* K /* dev */, const void* V /* dev */,
                                  int64_t ld_qkv, const void* dA /* dev */, int64_t ld_da,
                                  const int32_t* q_rows /* dev, nullable */, const int32_t* q_offsets /* dev, nullable */,
                                  const int32_t* kv_rows /* dev, nullable */, const int32_t* kv_offsets /* dev, nullable */,
                                  int64_t B, int64_t N, int64_t heads, int64_t head_dim, int64_t max_kept,
                                  void* dQ /* dev */, void* dK /* dev */, void* dV /* dev */, int64_t ld_out,
                                  uint32_t flags, int32_t* status_word /* dev, nullable */, void* stream);

/*
 * Diagnostic (pure host function; no counterpart in the paper): how many times this process has
 * searched for the cut of the weight-gradient reduction of a layer shape.  The answer for a shape
 * is remembered for the life of the process, so the count stops growing once every shape of a
 * model has been seen: neither sbp_linear_backward nor the workspace-size query repeats a search.
 */
int64_t sbp_plan_search_count(void);

/*
 * One whole SBP step of a layer for callers whose tensors live in HOST memory: copies X, dY, W
 * to the device, draws the keep set (Sec. 4), builds the forward cache (Algorithm 1), runs the
 * backward (Eq. 5) and copies dW, db, dX (and optionally the indices) back, all enqueued on
 * `stream`; the caller synchronises the stream before reading the host outputs.  Host buffers
 * should be page-locked so the copies run asynchronously.
 *
 * X_host [B*H*W, C_in], dY_host [B*H*W, C_out], W_host [C_in, C_out]: element type dt.
 * dW_host [C_in, C_out] fp32, db_host [C_out] fp32, dX_host [B*H*W, C_in] dt.
 * keep_rows_host (nullable, capacity B * sbp_keep_count(...); entries past keep_offsets[B] are
 * unspecified), keep_offsets_host (nullable, B + 1 entries), status_host (nullable, one int32: the device status word of the step).
 * arena (dev): caller-owned scratch of at least sbp_step_host_arena_bytes(...) bytes, 256-byte
 * aligned; holds the device copies of every tensor during the step.  Nothing is allocated.
 * flags: SBP_FLAG_SHARE_MASK, SBP_FLAG_VALIDATE, SBP_FLAG_PLAIN_FMA (accumulation is not offered).
 * Errors as for the three calls it is built from; SBP_ERR_WORKSPACE for a short arena.
 */
size_t sbp_step_host_arena_bytes(sbp_dtype dt, sbp_mask_mode mode, int64_t B, int64_t H, int64_t W,
                                 int64_t C_in, int64_t C_out, double keep_ratio);

sbp_status sbp_step_host(sbp_dtype dt, sbp_mask_mode mode, int64_t B, int64_t H, int64_t W,
                         int64_t C_in, int64_t C_out, double keep_ratio, uint64_t seed, uint64_t step,
                         int64_t sample_offset, uint32_t flags,
                         const void* X_host, const void* dY_host, const void* W_host,
                         float* dW_host, float* db_host, void* dX_host,
                         int32_t* keep_rows_host /* nullable */, int32_t* keep_offsets_host /* nullable */,
                         int32_t* status_host /* nullable */,
                         void* arena /* dev */, size_t arena_bytes, void* stream);

/*
 * Bias gradient without any workspace argument (an addition of this library; the paper has no
 * counterpart):  db[j] (+)= sum_{m < M_keep} dY[keep_rows[m], j], as sbp_linear_backward computes it.
 *
 * For callers that cannot allocate device memory and so cannot supply a workspace - operator
 * plugins that receive only their tensors, code under a memory pool owned and locked by another
 * framework, services with a fixed device-memory budget.  The split-reduction scratch lives in a
 * fixed 1 MiB device array inside the library (held by every GPU that loads the library until the
 * process exits).  The call allocates and frees nothing.
 *
 * Limits: C_out <= 4096 (SBP_ERR_WORKSPACE beyond it: the built-in scratch is too small; use
 * sbp_linear_backward with a workspace).  C_out a multiple of 8 (bf16) / 4 (fp32).
 * flags: SBP_FLAG_ACCUMULATE or 0.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  All calls on a device share the array, which
 * keeps the previous call's contents (nothing in it needs clearing: each call overwrites every
 * entry it later reads); calls whose kernels may overlap on the GPU (different streams) race on it
 * and must be ordered by the caller.
 */
sbp_status sbp_bias_grad_static(sbp_dtype dt, const void* dY /* dev */, const int32_t* keep_rows /* dev */,
                                const int32_t* M_keep_dev /* dev, nullable */, int64_t M, int64_t M_keep_cap,
                                int64_t C_out, float* db /* dev */, uint32_t flags, void* stream);

/*
 * Diagnostic (no counterpart in the paper): runs the library's bounded device-side wait
 * on a barrier that is never completed, with a limit of limit_ms (0 < limit_ms <= 2000).
 * On return of the kernel *completed (dev) is 0 and *status_word (dev, zero before the
 * call) holds SBP_ERR_TIMEOUT; the stream and the context remain usable.  This is the
 * mechanism every pipeline kernel uses instead of an unbounded spin.
 */
sbp_status sbp_selftest_bounded_wait(double limit_ms, int32_t* status_word /* dev */,
                                     int32_t* completed /* dev */, void* stream);

/*
 * Diagnostic probes (no counterpart in the paper): micro-measurements of the machinery the tensor-core kernels are
 * built from; `python bench.py --probe` prints their tables.  The caller times the calls with events.
 *
 * sbp_probe_gather_ring: copies the rows `rows[0 .. n_rows)` (each an index of a row of `row_bytes` bytes in `src`,
 *   row_bytes a multiple of 128; the indices must lie inside src) with 16-byte cp.async into a ring of `stages`
 *   (2..12) 16 KB shared-memory stages per block, `threads` (64, 128 or 256) copying threads and `blocks` blocks, the
 *   way the backward kernel gathers the kept rows of dY; a consumer frees each stage as it lands.  Nothing is written
 *   to global memory.
 * sbp_probe_operand_feed: the same ring fed by both producers of the backward kernel: per stage 64 threads gather
 *   `gather_rows` (0, 64 or 128) rows x 128 bytes as above and one thread issues `tma_boxes` (0..3) TMA loads of 128 rows
 *   x 128 bytes at scattered places of the bf16 matrix `dense` [dense_rows (multiple of 128), dense_cols (multiple of
 *   64)]; each of `blocks` blocks runs `steps` stages through a ring of `stages` stages (at most 192 KB).
 * sbp_probe_mma_rate: one thread per block issues 4 * iters tcgen05.mma (M = 128, K = 16, bf16, width N a multiple of
 *   16 up to 256, operands K-major or MN-major) into one accumulator, or alternating between two accumulators 256
 *   columns apart (accumulators = 2: 8 * iters instructions); cycles_out[0] (dev) receives the SM clocks from the
 *   first issue to the completion of the last instruction on block 0, or -1 if the bounded wait ran out.
 * sbp_probe_mma_pair_rate: the same stream in the two-SM form: `pairs` clusters of two blocks, the first block's
 *   thread issuing 4 * iters tcgen05.mma.cta_group::2 (M = 256 over the pair, N a multiple of 32 up to 256, each SM
 *   supplying its 128 rows of A and N / 2 rows of B); cycles_out[0] as above.
 * SBP_ERR_INVALID_ARG for sizes outside these ranges and null / misaligned pointers.
 */
sbp_status sbp_probe_gather_ring(const void* src /* dev */, int64_t row_bytes, const int32_t* rows /* dev */, int64_t n_rows,
                                 int threads, int stages, int blocks, int32_t* status_word /* dev, nullable */, void* stream);
sbp_status sbp_probe_operand_feed(const void* src /* dev */, int64_t row_bytes, const int32_t* rows /* dev */, int64_t n_rows,
                                  int gather_rows, const void* dense /* dev */, int64_t dense_rows, int64_t dense_cols, int tma_boxes,
                                  int stages, int steps, int blocks, int32_t* status_word /* dev, nullable */, void* stream);
sbp_status sbp_probe_mma_rate(int N, int mn_major, int accumulators, int iters, int blocks, int64_t* cycles_out /* dev */,
                              int32_t* status_word /* dev, nullable */, void* stream);
sbp_status sbp_probe_mma_pair_rate(int N, int mn_major, int iters, int pairs, int64_t* cycles_out /* dev */,
                                   int32_t* status_word /* dev, nullable */, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SBP_H_ */
