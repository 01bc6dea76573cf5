// The extern "C" boundary declared in include/sbp.h: argument checks, kernel choice, launches.
#include <math.h>

#include "sbp_common.cuh"

namespace {

using namespace sbp;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int grid_family_of(double r) {
    if (r == 0.25) return 1;
    if (r == 0.5) return 2;
    if (r == 0.75) return 3;
    if (r == 1.0) return 4;
    return 0;
}

inline bool ratio_ok(double r) { return r > 0.0 && r <= 1.0; }   // false for NaN

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// scratch for the bias sums: the stand-alone kernel's row splits, or one partial row per SM when the
// sums ride along in the tensor-core kernel
inline size_t db_scratch_bytes(sbp_dtype dt, int64_t M_keep_cap, int64_t C_out) {
    const size_t a = db_workspace_bytes(dt, M_keep_cap, C_out, kDbMaxSplits);
    const size_t b = (size_t)kNumSMs * (size_t)C_out * sizeof(float);
    return align_up(a > b ? a : b, 256);
}

inline bool use_tensor_cores(sbp_dtype dt, uint32_t flags, int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    return dt == SBP_BF16 && !(flags & SBP_FLAG_PLAIN_FMA) && tc_shapes_supported(M, M_keep_cap, C_in, C_out);
}

}  // namespace

extern "C" {

const char* sbp_status_string(sbp_status s) {
    switch (s) {
        case SBP_OK: return "ok";
        case SBP_ERR_INVALID_ARG: return "invalid argument";
        case SBP_ERR_UNSUPPORTED: return "unsupported request";
        case SBP_ERR_WORKSPACE: return "workspace missing or too small";
        case SBP_ERR_CUDA: return "CUDA call failed";
        case SBP_ERR_TIMEOUT: return "bounded device wait expired";
        case SBP_ERR_BAD_INDICES: return "keep_rows not strictly ascending or out of range";
    }
    return "unknown status";
}

int64_t sbp_keep_count(sbp_mask_mode mode, int64_t H, int64_t W, double keep_ratio) {
    if (H <= 0 || W <= 0 || !ratio_ok(keep_ratio)) return -1;
    const int64_t N = H * W;
    if (mode == SBP_MASK_RANDOM) {
        int64_t K = (int64_t)floor(keep_ratio * (double)N + 0.5);
        if (K < 1) K = 1;
        if (K > N) K = N;
        return K;
    }
    if (mode == SBP_MASK_TEMPORAL) {          // H frames of W positions each: whole frames are kept
        int64_t KT = (int64_t)floor(keep_ratio * (double)H + 0.5);
        if (KT < 1) KT = 1;
        if (KT > H) KT = H;
        return KT * W;
    }
    if (mode == SBP_MASK_TEMPORAL_GRID) {     // capacity: the phase (0) that keeps the most frames, times W
        switch (grid_family_of(keep_ratio)) {
            case 1: return ((H + 3) / 4) * W;
            case 2: return ((H + 1) / 2) * W;
            case 3: return (H - H / 4) * W;          // all but the phase-3 class, the smallest one
            case 4: return H * W;
            default: return -1;
        }
    }
    if (mode == SBP_MASK_GRID) {
        const int64_t quarter_max = ((H + 1) / 2) * ((W + 1) / 2);   // phase (0, 0) holds the most lattice points
        const int64_t quarter_min = (H / 2) * (W / 2);               // phase (1, 1) the fewest
        switch (grid_family_of(keep_ratio)) {
            case 1: return quarter_max;
            case 2: return (N + 1) / 2;
            case 3: return N - quarter_min;
            case 4: return N;
            default: return -1;
        }
    }
    return -1;
}

sbp_status sbp_sample_keep(sbp_mask_mode mode, int64_t B, int64_t H, int64_t W, double keep_ratio,
                           uint64_t seed, uint64_t step, int64_t sample_offset, uint32_t flags,
                           int32_t* keep_rows, int32_t* keep_offsets, void* stream) {
    if (mode != SBP_MASK_RANDOM && mode != SBP_MASK_GRID && mode != SBP_MASK_TEMPORAL && mode != SBP_MASK_TEMPORAL_GRID)
        return SBP_ERR_INVALID_ARG;
    if (keep_rows == nullptr || keep_offsets == nullptr) return SBP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(keep_rows) & 3u) || (reinterpret_cast<uintptr_t>(keep_offsets) & 3u))
        return SBP_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || !ratio_ok(keep_ratio)) return SBP_ERR_INVALID_ARG;
    if (H >= (1ll << 31) || W >= (1ll << 31) || H * W >= (1ll << 31) || B >= (1ll << 31) ||
        B * (H * W) >= (1ll << 31))
        return SBP_ERR_INVALID_ARG;
    if (step >> 32) return SBP_ERR_INVALID_ARG;
    if (sample_offset < 0 || ((uint64_t)(sample_offset + B - 1) >> 32)) return SBP_ERR_INVALID_ARG;
    const int family = grid_family_of(keep_ratio);
    if ((mode == SBP_MASK_GRID || mode == SBP_MASK_TEMPORAL_GRID) && family == 0) return SBP_ERR_UNSUPPORTED;
    if ((mode == SBP_MASK_TEMPORAL || mode == SBP_MASK_TEMPORAL_GRID) && H > (int64_t)sample_keep_max_frames())
        return SBP_ERR_UNSUPPORTED;
    const int64_t K = sbp_keep_count(mode, H, W, keep_ratio);
    const cudaError_t e = launch_sample_keep((int)mode, family, B, H, W, K, seed, (uint32_t)step,
                                             (uint32_t)sample_offset, (flags & SBP_FLAG_SHARE_MASK) != 0,
                                             keep_rows, keep_offsets, (cudaStream_t)stream);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

sbp_status sbp_forward_cache(sbp_dtype dt, const void* X, int64_t M, int64_t C, const int32_t* keep_rows,
                             const int32_t* M_keep_dev, int64_t M_keep_cap, void* X_keep, void* stream) {
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (X == nullptr || X_keep == nullptr || keep_rows == nullptr) return SBP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(X_keep)) return SBP_ERR_INVALID_ARG;
    if (M <= 0 || C <= 0 || M_keep_cap < 0 || M >= (1ll << 31) || M_keep_cap > M) return SBP_ERR_INVALID_ARG;
    const int64_t row_bytes = C * (dt == SBP_BF16 ? 2 : 4);
    if (row_bytes % 16 != 0) return SBP_ERR_UNSUPPORTED;
    const cudaError_t e = launch_gather_rows(X, row_bytes, keep_rows, M_keep_dev, M_keep_cap, X_keep,
                                             (cudaStream_t)stream);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

sbp_status sbp_linear_forward(sbp_dtype dt, const void* X, const void* W, const float* bias, int64_t M, int64_t C_in,
                              int64_t C_out, void* Y, const int32_t* keep_rows, const int32_t* M_keep_dev,
                              int64_t M_keep_cap, void* X_keep, uint32_t flags, int32_t* status_word, void* stream_v) {
    cudaStream_t stream = (cudaStream_t)stream_v;
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (X == nullptr || W == nullptr || Y == nullptr) return SBP_ERR_INVALID_ARG;
    if (M <= 0 || M >= (1ll << 31) || C_in <= 0 || C_out <= 0 || C_in >= (1ll << 24) || C_out >= (1ll << 24))
        return SBP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || !aligned16(bias) || !aligned16(X_keep))
        return SBP_ERR_INVALID_ARG;
    if (X_keep != nullptr) {
        if (keep_rows == nullptr || (reinterpret_cast<uintptr_t>(keep_rows) & 3u) || M_keep_cap < 0 || M_keep_cap > M)
            return SBP_ERR_INVALID_ARG;
    }
    const int64_t mult = (dt == SBP_BF16) ? 8 : 4;
    if (C_in % mult != 0 || C_out % mult != 0) return SBP_ERR_UNSUPPORTED;
    if (dt == SBP_BF16 && !(flags & SBP_FLAG_PLAIN_FMA) && tc_forward_supported(M, C_in, C_out)) {
        // The cache rides along in the product kernel (four side warps per SM, about 12 GB/s each SM) when that
        // copy takes no more than a quarter of the product's own time (a longer one slows the operand loads down more than
        // a second launch costs); otherwise the stand-alone gather kernel follows.
        bool ride = X_keep != nullptr;
        if (ride) {
            const double copy_us = (double)M_keep_cap * (double)C_in * 2.0 / (double)kNumSMs / 12e3;
            const double flop_us = 2.0 * (double)M * (double)C_in * (double)C_out / 1.0e9;            // at 1000 TFLOP/s
            const double byte_us = ((double)M * (double)(C_in + C_out) * 2.0) / 5.0e6;                 // at 5 TB/s
            ride = copy_us <= 0.25 * (flop_us > byte_us ? flop_us : byte_us);
        }
        const sbp_status s = launch_tc_forward(X, W, (flags & SBP_FLAG_W_OUT_IN) != 0, bias, M, C_in, C_out, Y, keep_rows,
                                               M_keep_dev, M_keep_cap, ride ? X_keep : nullptr, status_word, stream);
        if (s != SBP_OK) return s;
        if (X_keep != nullptr && !ride &&
            launch_gather_rows(X, C_in * 2, keep_rows, M_keep_dev, M_keep_cap, X_keep, stream) != cudaSuccess)
            return SBP_ERR_CUDA;
        return SBP_OK;
    }
    if (launch_simt_forward(dt, X, W, (flags & SBP_FLAG_W_OUT_IN) != 0, bias, M, C_in, C_out, Y, status_word, stream) !=
        cudaSuccess)
        return SBP_ERR_CUDA;
    if (X_keep != nullptr &&
        launch_gather_rows(X, C_in * (dt == SBP_BF16 ? 2 : 4), keep_rows, M_keep_dev, M_keep_cap, X_keep, stream) !=
            cudaSuccess)
        return SBP_ERR_CUDA;
    return SBP_OK;
}

namespace {
size_t base_workspace_bytes(sbp_dtype dt, int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out);
// after the kernels' own scratch: room for W and dW in the [C_in, C_out] layout, used with SBP_FLAG_W_OUT_IN
size_t w_copy_bytes(sbp_dtype dt, int64_t C_in, int64_t C_out) {
    return align_up((size_t)C_in * (size_t)C_out * (dt == SBP_BF16 ? 2 : 4), 256);
}
size_t dw_copy_bytes(int64_t C_in, int64_t C_out) { return align_up((size_t)C_in * (size_t)C_out * 4, 256); }
}  // namespace

size_t sbp_linear_backward_workspace_bytes(sbp_dtype dt, int64_t M, int64_t M_keep_cap, int64_t C_in,
                                           int64_t C_out) {
    if (M <= 0 || M_keep_cap < 0 || C_in <= 0 || C_out <= 0) return 256;
    return base_workspace_bytes(dt, M, M_keep_cap, C_in, C_out) + w_copy_bytes(dt, C_in, C_out) +
           dw_copy_bytes(C_in, C_out);
}

namespace {
size_t base_workspace_bytes(sbp_dtype dt, int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    const size_t db_part = db_scratch_bytes(dt, M_keep_cap, C_out);
    size_t dw_part = simt_dw_workspace_bytes(M_keep_cap, C_in, C_out);
    if (dt == SBP_BF16 && tc_shapes_supported(M, M_keep_cap, C_in, C_out)) {
        const size_t t = tc_dw_workspace_bytes(M_keep_cap, C_in, C_out);
        if (t > dw_part) dw_part = t;
    }
    return db_part + align_up(dw_part, 256) + 256;
}
}  // namespace

namespace {
// the backward with W and dW in the paper's [C_in, C_out] layout
sbp_status backward_in_out(sbp_dtype dt, const void* X_keep, const void* dY, const void* W,
                           const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M,
                           int64_t M_keep_cap, int64_t C_in, int64_t C_out, float* dW, float* db, void* dX,
                           uint32_t flags, void* workspace, size_t workspace_bytes, size_t workspace_required,
                           int32_t* status_word, cudaStream_t stream) {
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    const bool dy_compact = (flags & SBP_FLAG_DY_COMPACT) != 0, dx_compact = (flags & SBP_FLAG_DX_COMPACT) != 0;
    // the packed forms address rows by their position m; keep_rows is needed for whichever side is not packed
    const bool need_rows = !dy_compact || (dX != nullptr && !dx_compact) || (flags & SBP_FLAG_VALIDATE);
    if (dY == nullptr || (need_rows && keep_rows == nullptr)) return SBP_ERR_INVALID_ARG;
    if (M <= 0 || M >= (1ll << 31) || M_keep_cap < 0 || M_keep_cap > M || C_in <= 0 || C_out <= 0 ||
        C_in >= (1ll << 24) || C_out >= (1ll << 24))
        return SBP_ERR_INVALID_ARG;
    if (dW != nullptr && X_keep == nullptr) return SBP_ERR_INVALID_ARG;
    if (dX != nullptr && W == nullptr) return SBP_ERR_INVALID_ARG;
    if (!aligned16(X_keep) || !aligned16(dY) || !aligned16(W) || !aligned16(dW) || !aligned16(db) ||
        !aligned16(dX) || (reinterpret_cast<uintptr_t>(keep_rows) & 3u))
        return SBP_ERR_INVALID_ARG;
    if ((flags & SBP_FLAG_VALIDATE) && status_word == nullptr) return SBP_ERR_INVALID_ARG;
    const int64_t mult = (dt == SBP_BF16) ? 8 : 4;
    if (C_in % mult != 0 || C_out % mult != 0) return SBP_ERR_UNSUPPORTED;
    const bool need_ws = (dW != nullptr) || (db != nullptr);
    if (need_ws) {
        if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
            workspace_bytes < workspace_required)
            return SBP_ERR_WORKSPACE;
    }
    const bool accumulate = (flags & SBP_FLAG_ACCUMULATE) != 0;
    float* ws_db = static_cast<float*>(workspace);
    float* ws_dw = need_ws ? reinterpret_cast<float*>(static_cast<char*>(workspace) +
                                                      db_scratch_bytes(dt, M_keep_cap, C_out))
                           : nullptr;

    const int32_t* dy_rows = dy_compact ? nullptr : keep_rows;
    const int32_t* dx_rows = dx_compact ? nullptr : keep_rows;
    const int64_t M_dx = dx_compact ? M_keep_cap : M;            // rows of the dX tensor
    if (flags & SBP_FLAG_VALIDATE) {
        if (launch_validate_keep_rows(keep_rows, M_keep_dev, M_keep_cap, M, status_word, stream) != cudaSuccess)
            return SBP_ERR_CUDA;
    }
    const bool tc = use_tensor_cores(dt, flags, M, M_keep_cap, C_in, C_out);
    // with the tensor-core kernel running, the bias sums ride along in it; otherwise they get their own kernel
    const bool db_rides = tc && db != nullptr && (dW != nullptr || dX != nullptr);
    if (db != nullptr && !db_rides) {
        if (launch_db(dt, dY, dy_rows, M_keep_dev, M_keep_cap, C_out, db, accumulate, ws_db, kDbMaxSplits,
                      status_word, stream) != cudaSuccess)
            return SBP_ERR_CUDA;
    }
    if (tc) {
        // both products (and the bias sums) in one persistent tensor-core kernel
        const sbp_status s = launch_tc_backward(X_keep, dY, W, dy_rows, dx_rows, M_keep_dev, M_dx, M_keep_cap, C_in, C_out, dW,
                                                accumulate, dX, db_rides ? db : nullptr, ws_dw, ws_db, status_word,
                                                stream);
        if (s != SBP_OK) return s;
    } else {
        if (dW != nullptr && launch_simt_dw(dt, X_keep, dY, dy_rows, M_keep_dev, M_keep_cap, C_in, C_out, dW,
                                            accumulate, ws_dw, status_word, stream) != cudaSuccess)
            return SBP_ERR_CUDA;
        if (dX != nullptr && launch_simt_dx(dt, dY, W, dy_rows, dx_rows, M_keep_dev, M_dx, M_keep_cap, C_in, C_out, dX,
                                            status_word, stream) != cudaSuccess)
            return SBP_ERR_CUDA;
    }
    return SBP_OK;
}

}  // namespace

sbp_status sbp_linear_backward(sbp_dtype dt, const void* X_keep, const void* dY, const void* W,
                               const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M,
                               int64_t M_keep_cap, int64_t C_in, int64_t C_out, float* dW, float* db, void* dX,
                               uint32_t flags, void* workspace, size_t workspace_bytes, int32_t* status_word,
                               void* stream_v) {
    cudaStream_t stream = (cudaStream_t)stream_v;
    if (!(flags & SBP_FLAG_W_OUT_IN) || (dW == nullptr && dX == nullptr))
        return backward_in_out(dt, X_keep, dY, W, keep_rows, M_keep_dev, M, M_keep_cap, C_in, C_out, dW, db, dX, flags,
                               workspace, workspace_bytes,
                               (M > 0 && M_keep_cap >= 0 && C_in > 0 && C_out > 0)
                                   ? sbp_linear_backward_workspace_bytes(dt, M, M_keep_cap, C_in, C_out) : 0,
                               status_word, stream);
    // W and dW are [C_out, C_in]: transpose W into the workspace, run the products on the copies, transpose dW out
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (M <= 0 || M_keep_cap < 0 || C_in <= 0 || C_out <= 0 || C_in >= (1ll << 24) || C_out >= (1ll << 24))
        return SBP_ERR_INVALID_ARG;
    if ((dX != nullptr && W == nullptr) || !aligned16(W) || !aligned16(dW)) return SBP_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < sbp_linear_backward_workspace_bytes(dt, M, M_keep_cap, C_in, C_out))
        return SBP_ERR_WORKSPACE;
    const size_t base = base_workspace_bytes(dt, M, M_keep_cap, C_in, C_out);
    void* w_copy = static_cast<char*>(workspace) + base;
    float* dw_copy = reinterpret_cast<float*>(static_cast<char*>(workspace) + base + w_copy_bytes(dt, C_in, C_out));
    const uint32_t inner = flags & ~(uint32_t)SBP_FLAG_W_OUT_IN;
    if (dX != nullptr &&
        launch_transpose(dt == SBP_BF16 ? 2 : 4, W, w_copy, C_out, C_in, status_word, stream) != cudaSuccess)
        return SBP_ERR_CUDA;
    const bool accumulate = (flags & SBP_FLAG_ACCUMULATE) != 0;
    sbp_status s;
    if (accumulate && dW != nullptr) {
        // dW is produced fresh in the copy and added in by the transpose; db accumulates in place on its own
        s = backward_in_out(dt, X_keep, dY, dX != nullptr ? w_copy : nullptr, keep_rows, M_keep_dev, M, M_keep_cap, C_in,
                            C_out, dw_copy, nullptr, dX, inner & ~(uint32_t)SBP_FLAG_ACCUMULATE, workspace, base, base,
                            status_word, stream);
        if (s == SBP_OK && db != nullptr)
            s = backward_in_out(dt, nullptr, dY, nullptr, keep_rows, M_keep_dev, M, M_keep_cap, C_in, C_out, nullptr, db,
                                nullptr, inner & ~(uint32_t)SBP_FLAG_VALIDATE, workspace, base, base, status_word, stream);
    } else {
        s = backward_in_out(dt, X_keep, dY, dX != nullptr ? w_copy : nullptr, keep_rows, M_keep_dev, M, M_keep_cap, C_in,
                            C_out, dW != nullptr ? dw_copy : nullptr, db, dX, inner, workspace, base, base, status_word, stream);
    }
    if (s != SBP_OK) return s;
    if (dW != nullptr &&
        launch_transpose_add_f32(dw_copy, dW, C_in, C_out, accumulate, status_word, stream) != cudaSuccess)
        return SBP_ERR_CUDA;
    return SBP_OK;
}

int sbp_linear_backward_kernel_count(sbp_dtype dt, int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out,
                                     int want_dW, int want_db, int want_dX, uint32_t flags) {
    const bool tc = use_tensor_cores(dt, flags, M, M_keep_cap, C_in, C_out);
    int n = (flags & SBP_FLAG_VALIDATE) ? 1 : 0;
    if ((flags & SBP_FLAG_W_OUT_IN) && (want_dW || want_dX)) n += (want_dX ? 1 : 0) + (want_dW ? 1 : 0);   // transposes
    const bool db_rides = tc && want_db && (want_dW || want_dX);
    if (want_db && !db_rides) n += 2;                      // strip partials + fixed-order reduce
    if (tc) return n + tc_backward_kernel_count(M_keep_cap, C_in, C_out, want_dW != 0, want_dX != 0, db_rides,
                                                (flags & SBP_FLAG_DY_COMPACT) != 0);
    if (want_dW) n += simt_dw_kernel_count(M_keep_cap, C_in, C_out);
    if (want_dX) n += 1;
    return n;
}

int64_t sbp_plan_search_count(void) { return tc_plan_searches(); }

sbp_status sbp_act_backward(sbp_dtype dt, sbp_activation act, const void* Z_keep, const void* dH, const int32_t* M_keep_dev,
                            int64_t M_keep_cap, int64_t C, void* dZ, int32_t* status_word, void* stream) {
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (act != SBP_ACT_GELU) return SBP_ERR_UNSUPPORTED;
    if (Z_keep == nullptr || dH == nullptr || dZ == nullptr || !aligned16(Z_keep) || !aligned16(dH) || !aligned16(dZ))
        return SBP_ERR_INVALID_ARG;
    if (M_keep_cap < 0 || M_keep_cap >= (1ll << 31) || C <= 0 || C >= (1ll << 24)) return SBP_ERR_INVALID_ARG;
    const int64_t row_bytes = C * (dt == SBP_BF16 ? 2 : 4);
    if (row_bytes % 16 != 0) return SBP_ERR_UNSUPPORTED;
    const cudaError_t e = launch_act_backward(dt, Z_keep, dH, dZ, row_bytes, M_keep_dev, M_keep_cap, status_word, (cudaStream_t)stream);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

namespace {
// shared argument checks of the two patch calls; returns SBP_OK and the output grid when the geometry is usable
sbp_status patch_geometry(sbp_dtype dt, int64_t B, int64_t H, int64_t W, int64_t C, int64_t k, int64_t stride, int64_t M_keep_cap,
                          int64_t* Ho, int64_t* Wo) {
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C <= 0 || k <= 0 || stride < k || k > H || k > W) return SBP_ERR_INVALID_ARG;
    if (B * H * W >= (1ll << 31) || C >= (1ll << 24) || k > 64) return SBP_ERR_INVALID_ARG;
    *Ho = (H - k) / stride + 1;
    *Wo = (W - k) / stride + 1;
    if (M_keep_cap < 0 || M_keep_cap > B * *Ho * *Wo) return SBP_ERR_INVALID_ARG;
    if ((C * (dt == SBP_BF16 ? 2 : 4)) % 16 != 0) return SBP_ERR_UNSUPPORTED;
    return SBP_OK;
}
}  // namespace

sbp_status sbp_patch_cache(sbp_dtype dt, const void* X, int64_t B, int64_t H, int64_t W, int64_t C, int64_t k, int64_t stride,
                           const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap, void* X_keep, void* stream) {
    int64_t Ho = 0, Wo = 0;
    const sbp_status g = patch_geometry(dt, B, H, W, C, k, stride, M_keep_cap, &Ho, &Wo);
    if (g != SBP_OK) return g;
    if (X == nullptr || X_keep == nullptr || keep_rows == nullptr || !aligned16(X) || !aligned16(X_keep) ||
        (reinterpret_cast<uintptr_t>(keep_rows) & 3u))
        return SBP_ERR_INVALID_ARG;
    const cudaError_t e = launch_patch_gather(X, H, W, C * (dt == SBP_BF16 ? 2 : 4), k, stride, keep_rows, M_keep_dev, M_keep_cap,
                                              X_keep, (cudaStream_t)stream);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

size_t sbp_patch_scatter_workspace_bytes(int64_t B, int64_t H, int64_t W, int64_t k, int64_t stride) {
    if (B <= 0 || H <= 0 || W <= 0 || k <= 0 || stride < k || k > H || k > W) return 256;
    return align_up((size_t)(B * ((H - k) / stride + 1) * ((W - k) / stride + 1)) * sizeof(int32_t), 256);
}

sbp_status sbp_patch_scatter(sbp_dtype dt, const void* dX_patches, int64_t B, int64_t H, int64_t W, int64_t C, int64_t k,
                             int64_t stride, const int32_t* keep_rows, const int32_t* M_keep_dev, int64_t M_keep_cap, void* dX,
                             void* workspace, size_t workspace_bytes, int32_t* status_word, void* stream) {
    int64_t Ho = 0, Wo = 0;
    const sbp_status g = patch_geometry(dt, B, H, W, C, k, stride, M_keep_cap, &Ho, &Wo);
    if (g != SBP_OK) return g;
    if (dX_patches == nullptr || dX == nullptr || keep_rows == nullptr || !aligned16(dX_patches) || !aligned16(dX) ||
        (reinterpret_cast<uintptr_t>(keep_rows) & 3u))
        return SBP_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < sbp_patch_scatter_workspace_bytes(B, H, W, k, stride))
        return SBP_ERR_WORKSPACE;
    const cudaError_t e = launch_patch_scatter(dX_patches, B, H, W, C * (dt == SBP_BF16 ? 2 : 4), k, stride, keep_rows, M_keep_dev,
                                               M_keep_cap, dX, static_cast<int32_t*>(workspace), status_word, (cudaStream_t)stream);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

sbp_status sbp_attention_backward(sbp_dtype dt, const void* Q, const void* K, const void* V, int64_t ld_qkv, const void* dA,
                                  int64_t ld_da, const int32_t* q_rows, const int32_t* q_offsets, const int32_t* kv_rows,
                                  const int32_t* kv_offsets, int64_t B, int64_t N, int64_t heads, int64_t head_dim,
                                  int64_t max_kept, void* dQ, void* dK, void* dV, int64_t ld_out, uint32_t flags,
                                  int32_t* status_word, void* stream) {
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (Q == nullptr || K == nullptr || V == nullptr || dA == nullptr || dQ == nullptr || dK == nullptr || dV == nullptr)
        return SBP_ERR_INVALID_ARG;
    if (B <= 0 || N <= 0 || heads <= 0 || head_dim <= 0 || B * N >= (1ll << 31) || heads * head_dim >= (1ll << 24))
        return SBP_ERR_INVALID_ARG;
    if ((q_rows == nullptr) != (q_offsets == nullptr) || (kv_rows == nullptr) != (kv_offsets == nullptr))
        return SBP_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(SBP_FLAG_ATTN_ALL_KEYS | SBP_FLAG_ATTN_KEPT_ROWS_ONLY)) return SBP_ERR_INVALID_ARG;
    if ((flags & SBP_FLAG_ATTN_ALL_KEYS) && kv_rows != nullptr) return SBP_ERR_INVALID_ARG;
    const int64_t C = heads * head_dim;
    if (ld_qkv < C || ld_da < C || ld_out < C) return SBP_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dA) || !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) ||
        (reinterpret_cast<uintptr_t>(q_rows) & 3u) || (reinterpret_cast<uintptr_t>(q_offsets) & 3u) ||
        (reinterpret_cast<uintptr_t>(kv_rows) & 3u) || (reinterpret_cast<uintptr_t>(kv_offsets) & 3u))
        return SBP_ERR_INVALID_ARG;
    if (!attention_supported(dt, head_dim)) return SBP_ERR_UNSUPPORTED;
    if (ld_qkv % 8 != 0 || ld_da % 8 != 0 || ld_out % 8 != 0) return SBP_ERR_UNSUPPORTED;
    // keys and values: their own lists, else all tokens when asked for, else the query lists (Drop QKV)
    const int32_t* k_rows = kv_rows != nullptr ? kv_rows : ((flags & SBP_FLAG_ATTN_ALL_KEYS) ? nullptr : q_rows);
    const int32_t* k_offs = kv_rows != nullptr ? kv_offsets : ((flags & SBP_FLAG_ATTN_ALL_KEYS) ? nullptr : q_offsets);
    // most tokens a sample can bring to either side: N where a side takes all tokens, else the caller's bound on its lists
    const bool any_all = q_rows == nullptr || k_rows == nullptr;
    const bool any_list = q_rows != nullptr || k_rows != nullptr;
    if (any_list && (max_kept <= 0 || max_kept > N)) return SBP_ERR_INVALID_ARG;
    const int64_t most = any_all ? N : max_kept;
    if (most > attention_max_tokens()) return SBP_ERR_UNSUPPORTED;
    const cudaError_t e = launch_attention_backward(Q, K, V, ld_qkv, dA, ld_da, q_rows, q_offsets, k_rows, k_offs, B, N, heads, most,
                                                    dQ, dK, dV, ld_out, (flags & SBP_FLAG_ATTN_KEPT_ROWS_ONLY) == 0, status_word,
                                                    (cudaStream_t)stream);
    return e == cudaSuccess ? SBP_OK : SBP_ERR_CUDA;
}

namespace {
struct StepArena {
    size_t X, dY, W, rows, offs, Xk, dW, db, dX, status, ws, ws_bytes, total;
};
StepArena plan_step_arena(sbp_dtype dt, int64_t M, int64_t cap_total, int64_t B, int64_t C_in, int64_t C_out) {
    const size_t es = (dt == SBP_BF16) ? 2 : 4;
    StepArena a;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off += align_up(bytes, 256); return at; };
    a.X = take((size_t)M * C_in * es);
    a.dY = take((size_t)M * C_out * es);
    a.W = take((size_t)C_in * C_out * es);
    a.rows = take((size_t)cap_total * 4);
    a.offs = take((size_t)(B + 1) * 4);
    a.Xk = take((size_t)cap_total * C_in * es);
    a.dW = take((size_t)C_in * C_out * 4);
    a.db = take((size_t)C_out * 4);
    a.dX = take((size_t)M * C_in * es);
    a.status = take(4);
    a.ws_bytes = sbp_linear_backward_workspace_bytes(dt, M, cap_total, C_in, C_out);
    a.ws = take(a.ws_bytes);
    a.total = off;
    return a;
}
}  // namespace

size_t sbp_step_host_arena_bytes(sbp_dtype dt, sbp_mask_mode mode, int64_t B, int64_t H, int64_t W, int64_t C_in,
                                 int64_t C_out, double keep_ratio) {
    const int64_t cap = sbp_keep_count(mode, H, W, keep_ratio);
    if (cap < 0 || B <= 0 || C_in <= 0 || C_out <= 0) return 0;
    return plan_step_arena(dt, B * H * W, B * cap, B, C_in, C_out).total;
}

sbp_status sbp_step_host(sbp_dtype dt, sbp_mask_mode mode, int64_t B, int64_t H, int64_t W, int64_t C_in,
                         int64_t C_out, double keep_ratio, uint64_t seed, uint64_t step, int64_t sample_offset,
                         uint32_t flags, const void* X_host, const void* dY_host, const void* W_host,
                         float* dW_host, float* db_host, void* dX_host, int32_t* keep_rows_host,
                         int32_t* keep_offsets_host, int32_t* status_host, void* arena, size_t arena_bytes,
                         void* stream_v) {
    cudaStream_t stream = (cudaStream_t)stream_v;
    if (dt != SBP_F32 && dt != SBP_BF16) return SBP_ERR_INVALID_ARG;
    if (X_host == nullptr || dY_host == nullptr || W_host == nullptr || dW_host == nullptr || db_host == nullptr ||
        dX_host == nullptr)
        return SBP_ERR_INVALID_ARG;
    if (flags & SBP_FLAG_ACCUMULATE) return SBP_ERR_UNSUPPORTED;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || C_out <= 0) return SBP_ERR_INVALID_ARG;
    const int64_t cap = sbp_keep_count(mode, H, W, keep_ratio);
    if (cap < 0) return (mode == SBP_MASK_GRID && ratio_ok(keep_ratio)) ? SBP_ERR_UNSUPPORTED : SBP_ERR_INVALID_ARG;
    if (H * W >= (1ll << 31) || B * (H * W) >= (1ll << 31)) return SBP_ERR_INVALID_ARG;
    const int64_t M = B * H * W, cap_total = B * cap;
    const StepArena a = plan_step_arena(dt, M, cap_total, B, C_in, C_out);
    if (arena == nullptr || (reinterpret_cast<uintptr_t>(arena) & 255u) || arena_bytes < a.total)
        return SBP_ERR_WORKSPACE;
    const size_t es = (dt == SBP_BF16) ? 2 : 4;
    char* base = static_cast<char*>(arena);
    auto ok = [](cudaError_t e) { return e == cudaSuccess; };
    if (!ok(cudaMemcpyAsync(base + a.X, X_host, (size_t)M * C_in * es, cudaMemcpyHostToDevice, stream)) ||
        !ok(cudaMemcpyAsync(base + a.dY, dY_host, (size_t)M * C_out * es, cudaMemcpyHostToDevice, stream)) ||
        !ok(cudaMemcpyAsync(base + a.W, W_host, (size_t)C_in * C_out * es, cudaMemcpyHostToDevice, stream)) ||
        !ok(cudaMemsetAsync(base + a.status, 0, 4, stream)))
        return SBP_ERR_CUDA;
    int32_t* rows = reinterpret_cast<int32_t*>(base + a.rows);
    int32_t* offs = reinterpret_cast<int32_t*>(base + a.offs);
    int32_t* status = reinterpret_cast<int32_t*>(base + a.status);
    sbp_status s = sbp_sample_keep(mode, B, H, W, keep_ratio, seed, step, sample_offset, flags, rows, offs, stream);
    if (s != SBP_OK) return s;
    s = sbp_forward_cache(dt, base + a.X, M, C_in, rows, offs + B, cap_total, base + a.Xk, stream);
    if (s != SBP_OK) return s;
    s = sbp_linear_backward(dt, base + a.Xk, base + a.dY, base + a.W, rows, offs + B, M, cap_total, C_in, C_out,
                            reinterpret_cast<float*>(base + a.dW), reinterpret_cast<float*>(base + a.db), base + a.dX,
                            flags & (SBP_FLAG_VALIDATE | SBP_FLAG_PLAIN_FMA), base + a.ws, a.ws_bytes, status, stream);
    if (s != SBP_OK) return s;
    if (!ok(cudaMemcpyAsync(dW_host, base + a.dW, (size_t)C_in * C_out * 4, cudaMemcpyDeviceToHost, stream)) ||
        !ok(cudaMemcpyAsync(db_host, base + a.db, (size_t)C_out * 4, cudaMemcpyDeviceToHost, stream)) ||
        !ok(cudaMemcpyAsync(dX_host, base + a.dX, (size_t)M * C_in * es, cudaMemcpyDeviceToHost, stream)))
        return SBP_ERR_CUDA;
    if (keep_rows_host != nullptr &&
        !ok(cudaMemcpyAsync(keep_rows_host, rows, (size_t)cap_total * 4, cudaMemcpyDeviceToHost, stream)))
        return SBP_ERR_CUDA;
    if (keep_offsets_host != nullptr &&
        !ok(cudaMemcpyAsync(keep_offsets_host, offs, (size_t)(B + 1) * 4, cudaMemcpyDeviceToHost, stream)))
        return SBP_ERR_CUDA;
    if (status_host != nullptr && !ok(cudaMemcpyAsync(status_host, status, 4, cudaMemcpyDeviceToHost, stream)))
        return SBP_ERR_CUDA;
    return SBP_OK;
}

}  // extern "C"
