"""SBP_FLAG_W_OUT_IN: W and dW stored [C_out, C_in] (the layout of framework linear layers) give the same numbers
as the paper's [C_in, C_out] layout (Sec. 3.2.1), transposed.  Expected values come from the oracle in its own
layout; the test only transposes them."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, dt_code, host, run_forward_cache

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-5, "bf16": 5e-3}


def relerr(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / max(np.linalg.norm(b), 1e-300))


@pytest.mark.parametrize("dtype,B,H,W,C_in,C_out,accumulate", [
    ("f32", 3, 9, 7, 36, 68, False),
    ("f32", 2, 8, 8, 32, 64, True),
    ("bf16", 2, 14, 14, 64, 32, False),          # CUDA-core path
    ("bf16", 5, 14, 14, 256, 384, False),        # tensor cores
    ("bf16", 3, 14, 14, 264, 136, True),         # ragged edges, accumulation through the transpose
    ("bf16", 9, 7, 7, 128, 512, True),
])
def test_backward_with_out_in_weights(dtype, B, H, W, C_in, C_out, accumulate):
    M = B * H * W
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, 51)
    keep, _ = oracle.sample_keep(0, B, H, W, 0.5, 2)
    M_keep = len(keep)
    rows_d = torch.from_numpy(keep.astype(np.int32)).cuda()
    Xk_d = run_forward_cache(dtype, dev(X, dtype), rows_d, M_keep)
    want = oracle.linear_backward(synth.to_f64(oracle.forward_cache(X, keep), dtype), synth.to_f64(dY, dtype),
                                  synth.to_f64(Wt, dtype), keep)
    W_oi = dev(np.ascontiguousarray(Wt.T), dtype)                                   # [C_out, C_in]
    code = dt_code(dtype)
    nb = sbp.sbp_linear_backward_workspace_bytes(code, M, M_keep, C_in, C_out)
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW0 = np.linspace(-1, 1, C_in * C_out, dtype=np.float32).reshape(C_out, C_in)
    db0 = np.linspace(2, 3, C_out, dtype=np.float32)
    dW = torch.from_numpy(dW0.copy()).cuda() if accumulate else torch.full((C_out, C_in), float("nan"), device="cuda")
    db = torch.from_numpy(db0.copy()).cuda() if accumulate else torch.full((C_out,), float("nan"), device="cuda")
    dX = torch.full((M, C_in), float("nan"), dtype=W_oi.dtype, device="cuda")
    flags = sbp.SBP_FLAG_W_OUT_IN | (sbp.SBP_FLAG_ACCUMULATE if accumulate else 0)
    sbp.sbp_linear_backward(code, Xk_d, dev(dY, dtype), W_oi, rows_d, None, M, M_keep, C_in, C_out, dW, db, dX, flags, ws, nb,
                            status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    tol = TOL[dtype]
    want_dW = want["dW"].T + (dW0 if accumulate else 0.0)
    want_db = want["db"] + (db0 if accumulate else 0.0)
    assert relerr(host(dW), want_dW) <= tol
    assert relerr(host(db), want_db) <= tol
    dX_bits = host(dX)
    assert relerr(synth.to_f64(dX_bits, dtype), want["dX"]) <= tol
    drop = np.setdiff1d(np.arange(M), keep)
    assert not np.any(dX_bits[drop].view(np.uint16 if dtype == "bf16" else np.uint32))
    plain = sbp.sbp_linear_backward_kernel_count(code, M, M_keep, C_in, C_out, flags=flags & ~sbp.SBP_FLAG_W_OUT_IN)
    assert sbp.sbp_linear_backward_kernel_count(code, M, M_keep, C_in, C_out, flags=flags) == plain + 2


@pytest.mark.parametrize("dtype,M,C_in,C_out,flags", [
    ("f32", 130, 36, 68, 0), ("bf16", 200, 64, 32, 0), ("bf16", 980, 256, 384, 0), ("bf16", 441, 264, 136, 0),
    ("bf16", 700, 256, 256, 8),       # SBP_FLAG_PLAIN_FMA
])
def test_forward_with_out_in_weights(dtype, M, C_in, C_out, flags):
    X, Wt, _ = synth.layer_inputs(dtype, M, C_in, C_out, 52)
    bias = np.linspace(-1, 1, C_out, dtype=np.float32)
    want = oracle.linear_forward(synth.to_f64(X, dtype), synth.to_f64(Wt, dtype), bias)
    X_d, W_oi = dev(X, dtype), dev(np.ascontiguousarray(Wt.T), dtype)
    Y = torch.full((M, C_out), float("nan"), dtype=X_d.dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sbp.sbp_linear_forward(dt_code(dtype), X_d, W_oi, torch.from_numpy(bias).cuda(), M, C_in, C_out, Y,
                           flags=flags | sbp.SBP_FLAG_W_OUT_IN, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert relerr(synth.to_f64(host(Y), dtype), want) <= TOL[dtype]
