"""ctypes front end of the fp64 CPU oracle (``oracle/sbp_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  It shares nothing with the CUDA library and
never imports it.  ``build()`` compiles the C file with gcc; every wrapper only
marshals numpy arrays, the arithmetic lives in the C file.

Paper passages each wrapped function follows are cited in the C source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sbp_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libsbp_oracle.so")

MASK_RANDOM = 0
MASK_GRID = 1
MASK_TEMPORAL = 2
MASK_TEMPORAL_GRID = 3
FLAG_SHARE_MASK = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle shared object beside its source (gcc -O2 -fopenmp)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
           "-ffp-contract=off", "-o", _LIB_PATH, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB_PATH)
    i64, u64, u32, dbl, vp = (ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32,
                              ctypes.c_double, ctypes.c_void_p)
    lib.oracle_philox4x32_10.argtypes = [vp, vp, vp]
    lib.oracle_philox4x32_10.restype = None
    lib.oracle_keep_count.argtypes = [ctypes.c_int, i64, i64, dbl]
    lib.oracle_keep_count.restype = i64
    lib.oracle_sample_keep.argtypes = [ctypes.c_int, i64, i64, i64, dbl, u64, u64, i64, u32, vp, vp]
    lib.oracle_sample_keep.restype = i64
    lib.oracle_forward_cache.argtypes = [vp, i64, vp, i64, vp]
    lib.oracle_forward_cache.restype = None
    lib.oracle_linear_backward.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, vp, vp, vp]
    lib.oracle_linear_backward.restype = None
    lib.oracle_full_backward.argtypes = [vp, vp, vp, i64, i64, i64, vp, vp, vp]
    lib.oracle_full_backward.restype = None
    lib.oracle_linear_forward.argtypes = [vp, vp, vp, i64, i64, i64, vp]
    lib.oracle_linear_forward.restype = None
    lib.oracle_attention_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp]
    lib.oracle_attention_forward.restype = None
    lib.oracle_attention_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, vp, vp, vp]
    lib.oracle_attention_backward.restype = None
    lib.oracle_attention_memory_ratio.argtypes = [ctypes.c_int, dbl, dbl, dbl]
    lib.oracle_attention_memory_ratio.restype = dbl
    lib.oracle_patch_conv_forward.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i64, i64, vp]
    lib.oracle_patch_conv_forward.restype = None
    lib.oracle_patch_conv_backward.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, i64, i64, vp, vp, vp]
    lib.oracle_patch_conv_backward.restype = None
    lib.oracle_gelu.argtypes = [vp, i64, vp]
    lib.oracle_gelu.restype = None
    lib.oracle_act_backward_gelu.argtypes = [vp, vp, i64, vp]
    lib.oracle_act_backward_gelu.restype = None
    lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
    lib.oracle_set_num_threads.restype = None
    lib.oracle_num_threads.argtypes = []
    lib.oracle_num_threads.restype = ctypes.c_int
    _lib = lib
    return lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def philox4x32_10(counter, key):
    """One Philox4x32-10 block: 4 counter words, 2 key words -> 4 output words."""
    c = np.asarray(counter, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    assert c.shape == (4,) and k.shape == (2,)
    out = np.zeros(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def keep_count(mode: int, H: int, W: int, keep_ratio: float) -> int:
    return int(_load().oracle_keep_count(mode, H, W, float(keep_ratio)))


def sample_keep(mode: int, B: int, H: int, W: int, keep_ratio: float, seed: int = 0,
                step: int = 0, sample_offset: int = 0, flags: int = 0):
    """Returns (keep_rows int32 [M_keep], keep_offsets int32 [B+1])."""
    cap = keep_count(mode, H, W, keep_ratio)
    if cap < 0:
        raise ValueError("arguments outside the sampler's domain")
    rows = np.zeros(max(B * cap, 1), dtype=np.int32)
    offs = np.zeros(B + 1, dtype=np.int32)
    n = _load().oracle_sample_keep(mode, B, H, W, float(keep_ratio), seed, step,
                                   sample_offset, flags, _ptr(rows), _ptr(offs))
    if n < 0:
        raise ValueError("arguments outside the sampler's domain")
    return rows[:n].copy(), offs


def forward_cache(X: np.ndarray, keep_rows: np.ndarray) -> np.ndarray:
    """Byte-exact gather of the kept rows of a 2-D array of any dtype."""
    X = np.ascontiguousarray(X)
    assert X.ndim == 2
    rows = np.ascontiguousarray(keep_rows, dtype=np.int32)
    out = np.empty((rows.shape[0], X.shape[1]), dtype=X.dtype)
    _load().oracle_forward_cache(_ptr(X), X.shape[1] * X.dtype.itemsize, _ptr(rows),
                                 rows.shape[0], _ptr(out))
    return out


def linear_forward(X, W, bias=None):
    """Y = X W (+ bias) in fp64 (Eq. 2)."""
    X, W = _f64(X), _f64(W)
    M, C_in = X.shape
    C_out = W.shape[1]
    assert W.shape == (C_in, C_out)
    b = _f64(bias) if bias is not None else None
    Y = np.empty((M, C_out))
    _load().oracle_linear_forward(_ptr(X), _ptr(W), _ptr(b), M, C_in, C_out, _ptr(Y))
    return Y


def linear_backward(X_keep, dY, W, keep_rows, want=("dW", "db", "dX")):
    """SBP backward of one linear layer in fp64.  Returns dict of requested outputs."""
    X_keep, dY, W = _f64(X_keep), _f64(dY), _f64(W)
    rows = np.ascontiguousarray(keep_rows, dtype=np.int32)
    M, C_out = dY.shape
    C_in = W.shape[0]
    M_keep = rows.shape[0]
    assert W.shape == (C_in, C_out) and X_keep.shape == (M_keep, C_in)
    dW = np.empty((C_in, C_out)) if "dW" in want else None
    db = np.empty(C_out) if "db" in want else None
    dX = np.empty((M, C_in)) if "dX" in want else None
    _load().oracle_linear_backward(_ptr(X_keep), _ptr(dY), _ptr(W), _ptr(rows), M_keep, M,
                                   C_in, C_out, _ptr(dW), _ptr(db), _ptr(dX))
    return {k: v for k, v in (("dW", dW), ("db", db), ("dX", dX)) if v is not None}


def full_backward(X, dY, W, want=("dW", "db", "dX")):
    """Full (no SBP) backward of the same layer in fp64."""
    X, dY, W = _f64(X), _f64(dY), _f64(W)
    M, C_out = dY.shape
    C_in = W.shape[0]
    assert X.shape == (M, C_in) and W.shape == (C_in, C_out)
    dW = np.empty((C_in, C_out)) if "dW" in want else None
    db = np.empty(C_out) if "db" in want else None
    dX = np.empty((M, C_in)) if "dX" in want else None
    _load().oracle_full_backward(_ptr(X), _ptr(dY), _ptr(W), M, C_in, C_out,
                                 _ptr(dW), _ptr(db), _ptr(dX))
    return {k: v for k, v in (("dW", dW), ("db", db), ("dX", dX)) if v is not None}


ATTN_DROP_QUERY = 0
ATTN_DROP_QKV = 1


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def attention_forward(Q, K, V, q_rows, q_offs, k_rows, k_offs, heads):
    """Attention output A [M, heads*d] in fp64 for queries in the q lists against keys in the k lists
    (per-sample lists of global row ids with their offsets); rows outside the q lists are zero."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    M, C = Q.shape
    d = C // heads
    qr, qo, kr, ko = _i32(q_rows), _i32(q_offs), _i32(k_rows), _i32(k_offs)
    A = np.empty((M, C))
    _load().oracle_attention_forward(_ptr(Q), _ptr(K), _ptr(V), _ptr(qr), _ptr(qo), _ptr(kr), _ptr(ko),
                                     len(qo) - 1, M, heads, d, _ptr(A))
    return A


def attention_backward(Q, K, V, dA, q_rows, q_offs, k_rows, k_offs, heads):
    """(dQ, dK, dV), each [M, heads*d] in fp64, zero outside the chosen token lists."""
    Q, K, V, dA = _f64(Q), _f64(K), _f64(V), _f64(dA)
    M, C = Q.shape
    d = C // heads
    qr, qo, kr, ko = _i32(q_rows), _i32(q_offs), _i32(k_rows), _i32(k_offs)
    dQ, dK, dV = np.empty((M, C)), np.empty((M, C)), np.empty((M, C))
    _load().oracle_attention_backward(_ptr(Q), _ptr(K), _ptr(V), _ptr(dA), _ptr(qr), _ptr(qo), _ptr(kr), _ptr(ko),
                                      len(qo) - 1, M, heads, d, _ptr(dQ), _ptr(dK), _ptr(dV))
    return dQ, dK, dV


def attention_memory_ratio(mode: int, d: float, n: float, r: float) -> float:
    return float(_load().oracle_attention_memory_ratio(mode, float(d), float(n), float(r)))


def patch_conv_forward(X, Wt, bias, k, stride):
    """Y [B, Ho, Wo, Co] of a k x k convolution with stride >= k, channels last, no padding (fp64)."""
    X, Wt = _f64(X), _f64(Wt)
    B, H, W, C = X.shape
    Co = Wt.shape[3]
    assert Wt.shape == (k, k, C, Co) and stride >= k
    b = _f64(bias) if bias is not None else None
    Y = np.empty((B, (H - k) // stride + 1, (W - k) // stride + 1, Co))
    _load().oracle_patch_conv_forward(_ptr(X), _ptr(Wt), _ptr(b), B, H, W, C, Co, k, stride, _ptr(Y))
    return Y


def patch_conv_backward(X, dY, Wt, keep_rows, k, stride, want=("dW", "db", "dX")):
    """SBP backward of that layer with dY kept on the listed output positions (ids (b*Ho + ho)*Wo + wo)."""
    X, dY, Wt = _f64(X), _f64(dY), _f64(Wt)
    B, H, W, C = X.shape
    Co = Wt.shape[3]
    rows = np.ascontiguousarray(keep_rows, dtype=np.int32)
    assert dY.shape == (B, (H - k) // stride + 1, (W - k) // stride + 1, Co) and stride >= k
    dW = np.empty((k, k, C, Co)) if "dW" in want else None
    db = np.empty(Co) if "db" in want else None
    dX = np.empty((B, H, W, C)) if "dX" in want else None
    _load().oracle_patch_conv_backward(_ptr(X), _ptr(dY), _ptr(Wt), _ptr(rows), rows.shape[0], B, H, W, C, Co, k, stride,
                                       _ptr(dW), _ptr(db), _ptr(dX))
    return {n: v for n, v in (("dW", dW), ("db", db), ("dX", dX)) if v is not None}


def gelu(z):
    """Exact GELU, z Phi(z), in fp64."""
    z = _f64(z)
    out = np.empty_like(z)
    _load().oracle_gelu(_ptr(z), z.size, _ptr(out))
    return out


def act_backward_gelu(z, dh):
    """dz = dh * gelu'(z) in fp64 (element-wise; the caller passes the kept rows)."""
    z, dh = _f64(z), _f64(dh)
    assert z.shape == dh.shape
    out = np.empty_like(z)
    _load().oracle_act_backward_gelu(_ptr(z), _ptr(dh), z.size, _ptr(out))
    return out
