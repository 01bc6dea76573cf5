"""Packed-gradient forms of sbp_linear_backward for chained layers (Sec. 3.3.1, Eq. 9), against the oracle.

With the same keep set on consecutive point-wise layers the gradient between them is non-zero only in the
kept rows, so a block can hand it on packed: SBP_FLAG_DX_COMPACT writes [M_keep_cap, C_in] rows,
SBP_FLAG_DY_COMPACT reads [M_keep_cap, C_out] rows.  The oracle has no packed form: the expected values
are its scattered results, gathered or scattered by the test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, host, run_backward, run_forward_cache

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-5, "bf16": 5e-3}


def relerr(a, b):
    d = np.linalg.norm(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64))
    n = np.linalg.norm(np.asarray(b, dtype=np.float64))
    return d / n if n > 0 else d


def _bits(a, dtype):
    return a.view(np.uint16 if dtype == "bf16" else np.uint32)


def _nan_like(shape, dtype):
    if dtype == "bf16":
        return np.full(shape, 0x7FC0, dtype=np.uint16)          # bf16 quiet NaN bit pattern
    return np.full(shape, np.nan, dtype=np.float32)


def _packed(dY, keep, cap, dtype):
    """Kept rows of dY packed to the front; the padding rows hold NaN: they must never reach a result."""
    out = _nan_like((max(cap, 1), dY.shape[1]), dtype)
    out[:len(keep)] = dY[keep]
    return out


@pytest.mark.parametrize("dtype,B,H,W,C_in,C_out,r,extra", [
    ("f32", 3, 9, 7, 36, 68, 0.5, 0),            # CUDA-core kernels, ragged tiles
    ("bf16", 2, 14, 14, 64, 32, 0.5, 0),         # bf16 shapes too small for the tensor-core kernel
    ("bf16", 5, 14, 14, 256, 384, 0.5, 0),       # tensor-core kernel, several tiles, ragged last row tile
    ("bf16", 3, 14, 14, 384, 136, 0.25, 37),     # capacity larger than the device-side count
    ("bf16", 9, 7, 7, 128, 512, 0.75, 5),
    ("bf16", 100, 14, 14, 512, 776, 0.5, 29),    # enough kept rows for pairs of blocks; 7 column tiles of dY: a dead half
])
def test_packed_forms_match_the_scattered_result(dtype, B, H, W, C_in, C_out, r, extra):
    M = B * H * W
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, 21)
    keep, _ = oracle.sample_keep(0, B, H, W, r, 3)
    M_keep, cap = len(keep), len(keep) + extra
    rows = np.zeros(cap, dtype=np.int32)
    rows[:M_keep] = keep
    rows_d = torch.from_numpy(rows).cuda()
    cnt = torch.tensor([M_keep], dtype=torch.int32, device="cuda") if extra else None
    Xk_d = run_forward_cache(dtype, dev(X, dtype), rows_d, cap, cnt)
    Xk = oracle.forward_cache(X, keep)
    want = oracle.linear_backward(synth.to_f64(Xk, dtype), synth.to_f64(dY, dtype), synth.to_f64(Wt, dtype), keep)
    tol = TOL[dtype]
    dY_full_d, dY_pack_d, W_d = dev(dY, dtype), dev(_packed(dY, keep, cap, dtype), dtype), dev(Wt, dtype)
    drop = np.setdiff1d(np.arange(M), keep)

    def check(got, packed_dx):
        assert got["status"] == 0
        assert relerr(host(got["dW"]), want["dW"]) <= tol
        assert relerr(host(got["db"]), want["db"]) <= tol
        dX_bits = host(got["dX"])
        if packed_dx:
            assert dX_bits.shape == (cap, C_in)
            assert relerr(synth.to_f64(dX_bits[:M_keep], dtype), want["dX"][keep]) <= tol
            assert not np.any(_bits(dX_bits[M_keep:], dtype))              # padding rows: +0.0
        else:
            assert relerr(synth.to_f64(dX_bits, dtype), want["dX"]) <= tol
            assert not np.any(_bits(dX_bits[drop], dtype))

    # packed dY in, scattered dX out (the layer at the lower boundary of a block)
    check(run_backward(dtype, Xk_d, dY_pack_d, W_d, rows_d, cap, cnt, flags=sbp.SBP_FLAG_DY_COMPACT, M=M, dX_rows=M), False)
    # full dY in, packed dX out (the layer at the upper boundary)
    check(run_backward(dtype, Xk_d, dY_full_d, W_d, rows_d, cap, cnt, flags=sbp.SBP_FLAG_DX_COMPACT, M=M, dX_rows=cap), True)
    # packed on both sides (a layer inside the block): the index list is not needed at all
    check(run_backward(dtype, Xk_d, dY_pack_d, W_d, None, cap, cnt,
                       flags=sbp.SBP_FLAG_DY_COMPACT | sbp.SBP_FLAG_DX_COMPACT, M=M, dX_rows=cap), True)


@pytest.mark.parametrize("dtype,B,H,W,C0,C1,C2", [("f32", 2, 8, 8, 32, 64, 32), ("bf16", 6, 14, 14, 256, 1024, 256)])
def test_two_layer_block_keeps_the_gradient_packed(dtype, B, H, W, C0, C1, C2):
    # Eq. 9: X1 = X0 W1, X2 = X1 W2, the same keep set on both layers.  The upper layer writes dX1 packed, the
    # lower one reads it packed; the results must equal two scattered oracle backward passes, and
    # dX0[keep] = dY[keep] W2^T W1^T with zeros elsewhere.
    M = B * H * W
    X0, W1, _ = synth.layer_inputs(dtype, M, C0, C1, 31)
    X1, W2, dY = synth.layer_inputs(dtype, M, C1, C2, 32)          # X1 stands for the cached input of the upper layer
    keep, _ = oracle.sample_keep(0, B, H, W, 0.5, 8)
    M_keep = len(keep)
    rows_d = torch.from_numpy(keep.astype(np.int32)).cuda()
    X0k_d = run_forward_cache(dtype, dev(X0, dtype), rows_d, M_keep)
    X1k_d = run_forward_cache(dtype, dev(X1, dtype), rows_d, M_keep)
    upper = run_backward(dtype, X1k_d, dev(dY, dtype), dev(W2, dtype), rows_d, M_keep, flags=sbp.SBP_FLAG_DX_COMPACT,
                         M=M, dX_rows=M_keep)
    lower = run_backward(dtype, X0k_d, upper["dX"], dev(W1, dtype), rows_d, M_keep, flags=sbp.SBP_FLAG_DY_COMPACT,
                         M=M, dX_rows=M)
    assert upper["status"] == 0 and lower["status"] == 0

    f64 = lambda a: synth.to_f64(a, dtype)
    want_u = oracle.linear_backward(f64(oracle.forward_cache(X1, keep)), f64(dY), f64(W2), keep)
    dX1 = want_u["dX"]
    if dtype == "bf16":                                               # the path hands dX1 on in bf16
        dX1 = synth.bf16_bits_to_f64(synth.f64_to_bf16_bits(dX1))
    want_l = oracle.linear_backward(f64(oracle.forward_cache(X0, keep)), dX1, f64(W1), keep)
    tol = TOL[dtype]
    assert relerr(host(upper["dW"]), want_u["dW"]) <= tol and relerr(host(upper["db"]), want_u["db"]) <= tol
    assert relerr(f64(host(upper["dX"])), want_u["dX"][keep]) <= tol
    assert relerr(host(lower["dW"]), want_l["dW"]) <= tol and relerr(host(lower["db"]), want_l["db"]) <= tol
    dX0_bits = host(lower["dX"])
    assert relerr(f64(dX0_bits), want_l["dX"]) <= tol
    drop = np.setdiff1d(np.arange(M), keep)
    assert not np.any(_bits(dX0_bits[drop], dtype))
    closed = np.zeros((M, C0))
    closed[keep] = f64(dY)[keep] @ f64(W2).T @ f64(W1).T             # Eq. 9, written out
    assert relerr(f64(dX0_bits), closed) <= 2 * tol


def test_packed_flags_still_need_the_index_list_where_it_is_used():
    M, cap, C = 64, 32, 32
    z = lambda *s: torch.zeros(*s, device="cuda")
    nb = sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_F32, M, cap, C, C)
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    call = lambda flags, dY_rows, dX_rows: sbp.sbp_linear_backward(
        sbp.SBP_F32, z(cap, C), z(dY_rows, C), z(C, C), None, None, M, cap, C, C, z(C, C), z(C), z(dX_rows, C), flags,
        ws, nb, None, check=False)
    assert call(sbp.SBP_FLAG_DY_COMPACT, cap, M) == sbp.SBP_ERR_INVALID_ARG      # scattered dX needs keep_rows
    assert call(sbp.SBP_FLAG_DX_COMPACT, M, cap) == sbp.SBP_ERR_INVALID_ARG      # full dY needs keep_rows
    assert call(sbp.SBP_FLAG_DY_COMPACT | sbp.SBP_FLAG_DX_COMPACT, cap, cap) == sbp.SBP_OK
    torch.cuda.synchronize()
