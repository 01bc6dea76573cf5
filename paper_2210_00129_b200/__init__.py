"""B200-native Stochastic Backpropagation (SBP) linear-layer hot path.

The compute lives in a C-ABI CUDA library (``include/sbp.h``, built in-tree as
``libsbp_b200.so``); this module is its thin Python binding: the functions below carry the
same names as the C entry points and only marshal arguments (torch tensors -> device
pointers, the current torch stream -> ``cudaStream_t``).  Every step of the path runs in the
library's kernels; there is no fallback - a missing library raises at the first call.

``synth`` (seeded input generators) is importable without the library.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsbp_b200.so")

# enums of include/sbp.h
SBP_OK, SBP_ERR_INVALID_ARG, SBP_ERR_UNSUPPORTED, SBP_ERR_WORKSPACE = 0, 1, 2, 3
SBP_ERR_CUDA, SBP_ERR_TIMEOUT, SBP_ERR_BAD_INDICES = 4, 5, 6
SBP_F32, SBP_BF16 = 0, 1
SBP_ACT_GELU = 0
SBP_MASK_RANDOM, SBP_MASK_GRID, SBP_MASK_TEMPORAL, SBP_MASK_TEMPORAL_GRID = 0, 1, 2, 3
SBP_FLAG_SHARE_MASK, SBP_FLAG_ACCUMULATE, SBP_FLAG_VALIDATE, SBP_FLAG_PLAIN_FMA = 1, 2, 4, 8
SBP_FLAG_DY_COMPACT, SBP_FLAG_DX_COMPACT, SBP_FLAG_W_OUT_IN, SBP_FLAG_ATTN_ALL_KEYS = 16, 32, 64, 128
SBP_FLAG_ATTN_KEPT_ROWS_ONLY = 256

EXPORTS = ("sbp_status_string", "sbp_keep_count", "sbp_sample_keep", "sbp_forward_cache", "sbp_linear_forward",
           "sbp_linear_backward_workspace_bytes", "sbp_linear_backward", "sbp_linear_backward_kernel_count",
           "sbp_plan_search_count", "sbp_act_backward", "sbp_attention_backward", "sbp_patch_cache", "sbp_patch_scatter_workspace_bytes",
           "sbp_patch_scatter", "sbp_step_host_arena_bytes", "sbp_step_host", "sbp_bias_grad_static",
           "sbp_selftest_bounded_wait", "sbp_probe_gather_ring", "sbp_probe_mma_rate", "sbp_probe_mma_pair_rate", "sbp_probe_operand_feed")

_lib = None


class SbpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (sbp_status {status})")


def load_library() -> ctypes.CDLL:
    """Load ``libsbp_b200.so``; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2210_00129_b200.build` "
                           "(the SBP path has no implementation outside this CUDA library)")
    lib = ctypes.CDLL(LIB_PATH)
    i64, u64, u32, dbl, vp, sz, ci = (ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_double,
                                      ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int)
    lib.sbp_status_string.argtypes = [ci]
    lib.sbp_status_string.restype = ctypes.c_char_p
    lib.sbp_keep_count.argtypes = [ci, i64, i64, dbl]
    lib.sbp_keep_count.restype = i64
    lib.sbp_sample_keep.argtypes = [ci, i64, i64, i64, dbl, u64, u64, i64, u32, vp, vp, vp]
    lib.sbp_sample_keep.restype = ci
    lib.sbp_forward_cache.argtypes = [ci, vp, i64, i64, vp, vp, i64, vp, vp]
    lib.sbp_forward_cache.restype = ci
    lib.sbp_selftest_bounded_wait.argtypes = [dbl, vp, vp, vp]
    lib.sbp_selftest_bounded_wait.restype = ci
    lib.sbp_linear_forward.argtypes = [ci, vp, vp, vp, i64, i64, i64, vp, vp, vp, i64, vp, u32, vp, vp]
    lib.sbp_linear_forward.restype = ci
    lib.sbp_linear_backward_workspace_bytes.argtypes = [ci, i64, i64, i64, i64]
    lib.sbp_linear_backward_workspace_bytes.restype = sz
    lib.sbp_linear_backward.argtypes = [ci, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp, vp, vp, u32, vp, sz, vp, vp]
    lib.sbp_linear_backward.restype = ci
    lib.sbp_linear_backward_kernel_count.argtypes = [ci, i64, i64, i64, i64, ci, ci, ci, u32]
    lib.sbp_linear_backward_kernel_count.restype = ci
    lib.sbp_attention_backward.argtypes = [ci, vp, vp, vp, i64, vp, i64, vp, vp, vp, vp, i64, i64, i64, i64, i64, vp, vp, vp, i64,
                                           u32, vp, vp]
    lib.sbp_attention_backward.restype = ci
    lib.sbp_patch_cache.argtypes = [ci, vp, i64, i64, i64, i64, i64, i64, vp, vp, i64, vp, vp]
    lib.sbp_patch_cache.restype = ci
    lib.sbp_patch_scatter_workspace_bytes.argtypes = [i64, i64, i64, i64, i64]
    lib.sbp_patch_scatter_workspace_bytes.restype = sz
    lib.sbp_patch_scatter.argtypes = [ci, vp, i64, i64, i64, i64, i64, i64, vp, vp, i64, vp, vp, sz, vp, vp]
    lib.sbp_patch_scatter.restype = ci
    lib.sbp_probe_gather_ring.argtypes = [vp, i64, vp, i64, ci, ci, ci, vp, vp]
    lib.sbp_probe_gather_ring.restype = ci
    lib.sbp_probe_mma_rate.argtypes = [ci, ci, ci, ci, ci, vp, vp, vp]
    lib.sbp_probe_mma_rate.restype = ci
    lib.sbp_probe_operand_feed.argtypes = [vp, i64, vp, i64, ci, vp, i64, i64, ci, ci, ci, ci, vp, vp]
    lib.sbp_probe_operand_feed.restype = ci
    lib.sbp_probe_mma_pair_rate.argtypes = [ci, ci, ci, ci, vp, vp, vp]
    lib.sbp_probe_mma_pair_rate.restype = ci
    lib.sbp_act_backward.argtypes = [ci, ci, vp, vp, vp, i64, i64, vp, vp, vp]
    lib.sbp_act_backward.restype = ci
    lib.sbp_plan_search_count.argtypes = []
    lib.sbp_plan_search_count.restype = i64
    lib.sbp_step_host_arena_bytes.argtypes = [ci, ci, i64, i64, i64, i64, i64, dbl]
    lib.sbp_step_host_arena_bytes.restype = sz
    lib.sbp_step_host.argtypes = [ci, ci, i64, i64, i64, i64, i64, dbl, u64, u64, i64, u32,
                                  vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sbp_step_host.restype = ci
    lib.sbp_bias_grad_static.argtypes = [ci, vp, vp, vp, i64, i64, i64, vp, u32, vp]
    lib.sbp_bias_grad_static.restype = ci
    _lib = lib
    return lib


def _ptr(t):
    """Device (or host) address of a torch tensor / raw integer address / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str):
    if status != SBP_OK:
        raise SbpError(status, where)


def status_string(status: int) -> str:
    return load_library().sbp_status_string(int(status)).decode()


def sbp_keep_count(mode: int, H: int, W: int, keep_ratio: float) -> int:
    return int(load_library().sbp_keep_count(mode, H, W, float(keep_ratio)))


def sbp_sample_keep(mode, B, H, W, keep_ratio, seed, step, sample_offset, flags, keep_rows, keep_offsets,
                    stream=None, check=True) -> int:
    """Fill ``keep_rows`` / ``keep_offsets`` (int32 CUDA tensors) on the current stream."""
    s = load_library().sbp_sample_keep(mode, B, H, W, float(keep_ratio), seed, step, sample_offset, flags,
                                       _ptr(keep_rows), _ptr(keep_offsets), _stream(stream))
    if check:
        _check(s, "sbp_sample_keep")
    return s


def sbp_forward_cache(dt, X, M, C, keep_rows, M_keep_dev, M_keep_cap, X_keep, stream=None, check=True) -> int:
    s = load_library().sbp_forward_cache(dt, _ptr(X), M, C, _ptr(keep_rows), _ptr(M_keep_dev), M_keep_cap,
                                         _ptr(X_keep), _stream(stream))
    if check:
        _check(s, "sbp_forward_cache")
    return s


def sbp_linear_forward(dt, X, W, bias, M, C_in, C_out, Y, keep_rows=None, M_keep_dev=None, M_keep_cap=0, X_keep=None,
                       flags=0, status_word=None, stream=None, check=True) -> int:
    """Y = X W + bias; with X_keep given the same launch also writes the forward cache."""
    s = load_library().sbp_linear_forward(dt, _ptr(X), _ptr(W), _ptr(bias), M, C_in, C_out, _ptr(Y), _ptr(keep_rows),
                                          _ptr(M_keep_dev), M_keep_cap, _ptr(X_keep), flags, _ptr(status_word),
                                          _stream(stream))
    if check:
        _check(s, "sbp_linear_forward")
    return s


def sbp_linear_backward_workspace_bytes(dt, M, M_keep_cap, C_in, C_out) -> int:
    return int(load_library().sbp_linear_backward_workspace_bytes(dt, M, M_keep_cap, C_in, C_out))


def sbp_linear_backward(dt, X_keep, dY, W, keep_rows, M_keep_dev, M, M_keep_cap, C_in, C_out, dW, db, dX,
                        flags, workspace, workspace_bytes, status_word=None, stream=None, check=True) -> int:
    s = load_library().sbp_linear_backward(dt, _ptr(X_keep), _ptr(dY), _ptr(W), _ptr(keep_rows), _ptr(M_keep_dev),
                                           M, M_keep_cap, C_in, C_out, _ptr(dW), _ptr(db), _ptr(dX), flags,
                                           _ptr(workspace), workspace_bytes, _ptr(status_word), _stream(stream))
    if check:
        _check(s, "sbp_linear_backward")
    return s


def sbp_linear_backward_kernel_count(dt, M, M_keep_cap, C_in, C_out, want_dW=True, want_db=True, want_dX=True,
                                     flags=0) -> int:
    return int(load_library().sbp_linear_backward_kernel_count(dt, M, M_keep_cap, C_in, C_out, int(want_dW),
                                                               int(want_db), int(want_dX), flags))


def sbp_attention_backward(dt, Q, K, V, ld_qkv, dA, ld_da, q_rows, q_offsets, kv_rows, kv_offsets, B, N, heads, head_dim,
                           max_kept, dQ, dK, dV, ld_out, flags=0, status_word=None, stream=None, check=True) -> int:
    """dQ, dK, dV of attention restricted to the listed query and key / value tokens (Drop QKV / Drop Query only)."""
    s = load_library().sbp_attention_backward(dt, _ptr(Q), _ptr(K), _ptr(V), ld_qkv, _ptr(dA), ld_da, _ptr(q_rows),
                                              _ptr(q_offsets), _ptr(kv_rows), _ptr(kv_offsets), B, N, heads, head_dim,
                                              max_kept, _ptr(dQ), _ptr(dK), _ptr(dV), ld_out, flags, _ptr(status_word),
                                              _stream(stream))
    if check:
        _check(s, "sbp_attention_backward")
    return s


def sbp_patch_cache(dt, X, B, H, W, C, k, stride, keep_rows, M_keep_dev, M_keep_cap, X_keep, stream=None, check=True) -> int:
    """Forward cache of a stride >= kernel convolution: the kept output positions' k x k patches as rows of k*k*C values."""
    s = load_library().sbp_patch_cache(dt, _ptr(X), B, H, W, C, k, stride, _ptr(keep_rows), _ptr(M_keep_dev), M_keep_cap,
                                       _ptr(X_keep), _stream(stream))
    if check:
        _check(s, "sbp_patch_cache")
    return s


def sbp_patch_scatter_workspace_bytes(B, H, W, k, stride) -> int:
    return int(load_library().sbp_patch_scatter_workspace_bytes(B, H, W, k, stride))


def sbp_patch_scatter(dt, dX_patches, B, H, W, C, k, stride, keep_rows, M_keep_dev, M_keep_cap, dX, workspace, workspace_bytes,
                      status_word=None, stream=None, check=True) -> int:
    """Packed patch gradients [M_keep_cap, k*k*C] back into dX [B, H, W, C], zeros everywhere else."""
    s = load_library().sbp_patch_scatter(dt, _ptr(dX_patches), B, H, W, C, k, stride, _ptr(keep_rows), _ptr(M_keep_dev),
                                         M_keep_cap, _ptr(dX), _ptr(workspace), workspace_bytes, _ptr(status_word),
                                         _stream(stream))
    if check:
        _check(s, "sbp_patch_scatter")
    return s


def sbp_act_backward(dt, act, Z_keep, dH, M_keep_dev, M_keep_cap, C, dZ, status_word=None, stream=None, check=True) -> int:
    """dZ = dH * act'(Z_keep) on packed kept rows (the activation between two layers of a packed block)."""
    s = load_library().sbp_act_backward(dt, act, _ptr(Z_keep), _ptr(dH), _ptr(M_keep_dev), M_keep_cap, C, _ptr(dZ),
                                        _ptr(status_word), _stream(stream))
    if check:
        _check(s, "sbp_act_backward")
    return s


def sbp_plan_search_count() -> int:
    return int(load_library().sbp_plan_search_count())


def sbp_step_host_arena_bytes(dt, mode, B, H, W, C_in, C_out, keep_ratio) -> int:
    return int(load_library().sbp_step_host_arena_bytes(dt, mode, B, H, W, C_in, C_out, float(keep_ratio)))


def sbp_step_host(dt, mode, B, H, W, C_in, C_out, keep_ratio, seed, step, sample_offset, flags, X_host, dY_host,
                  W_host, dW_host, db_host, dX_host, keep_rows_host, keep_offsets_host, status_host, arena,
                  arena_bytes, stream=None, check=True) -> int:
    """Whole step from host (ideally pinned) tensors; results land in the host outputs once the stream is synced."""
    s = load_library().sbp_step_host(dt, mode, B, H, W, C_in, C_out, float(keep_ratio), seed, step, sample_offset,
                                     flags, _ptr(X_host), _ptr(dY_host), _ptr(W_host), _ptr(dW_host), _ptr(db_host),
                                     _ptr(dX_host), _ptr(keep_rows_host), _ptr(keep_offsets_host), _ptr(status_host),
                                     _ptr(arena), arena_bytes, _stream(stream))
    if check:
        _check(s, "sbp_step_host")
    return s


def sbp_bias_grad_static(dt, dY, keep_rows, M_keep_dev, M, M_keep_cap, C_out, db, flags=0, stream=None,
                         check=True) -> int:
    """Bias gradient with the library's built-in scratch: for callers that cannot allocate a workspace."""
    s = load_library().sbp_bias_grad_static(dt, _ptr(dY), _ptr(keep_rows), _ptr(M_keep_dev), M, M_keep_cap, C_out,
                                            _ptr(db), flags, _stream(stream))
    if check:
        _check(s, "sbp_bias_grad_static")
    return s


def sbp_probe_gather_ring(src, row_bytes, rows, n_rows, threads, stages, blocks, status_word=None, stream=None, check=True) -> int:
    """Diagnostic: gather rows through a shared-memory ring as the tensor-core kernels do; time it with events."""
    s = load_library().sbp_probe_gather_ring(_ptr(src), row_bytes, _ptr(rows), n_rows, threads, stages, blocks, _ptr(status_word),
                                             _stream(stream))
    if check:
        _check(s, "sbp_probe_gather_ring")
    return s


def sbp_probe_mma_rate(N, mn_major, accumulators, iters, blocks, cycles_out, status_word=None, stream=None, check=True) -> int:
    """Diagnostic: clocks of a stream of tcgen05.mma instructions of width N (int64 CUDA tensor receives the count)."""
    s = load_library().sbp_probe_mma_rate(N, int(mn_major), accumulators, iters, blocks, _ptr(cycles_out), _ptr(status_word),
                                          _stream(stream))
    if check:
        _check(s, "sbp_probe_mma_rate")
    return s


def sbp_probe_operand_feed(src, row_bytes, rows, n_rows, gather_rows, dense, dense_rows, dense_cols, tma_boxes, stages, steps, blocks,
                           status_word=None, stream=None, check=True) -> int:
    """Diagnostic: the gather ring fed by cp.async gathers and TMA loads of a dense matrix together (nothing is computed)."""
    s = load_library().sbp_probe_operand_feed(_ptr(src), row_bytes, _ptr(rows), n_rows, gather_rows, _ptr(dense), dense_rows, dense_cols,
                                              tma_boxes, stages, steps, blocks, _ptr(status_word), _stream(stream))
    if check:
        _check(s, "sbp_probe_operand_feed")
    return s


def sbp_probe_mma_pair_rate(N, mn_major, iters, pairs, cycles_out, status_word=None, stream=None, check=True) -> int:
    """Diagnostic: clocks of a stream of two-SM tcgen05.mma instructions (M = 256 over a pair of SMs) of width N."""
    s = load_library().sbp_probe_mma_pair_rate(N, int(mn_major), iters, pairs, _ptr(cycles_out), _ptr(status_word), _stream(stream))
    if check:
        _check(s, "sbp_probe_mma_pair_rate")
    return s


def sbp_selftest_bounded_wait(limit_ms, status_word, completed, stream=None, check=True) -> int:
    """Runs a device-side wait that cannot complete; it must give up after limit_ms and report SBP_ERR_TIMEOUT."""
    s = load_library().sbp_selftest_bounded_wait(float(limit_ms), _ptr(status_word), _ptr(completed), _stream(stream))
    if check:
        _check(s, "sbp_selftest_bounded_wait")
    return s
