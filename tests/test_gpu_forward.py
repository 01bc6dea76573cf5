"""sbp_linear_forward (Eq. 2 with the cache of Algorithm 1 fused in) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, dt_code, host

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-5, "bf16": 5e-3}


def relerr(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def _forward(dtype, X, Wt, bias, keep=None, cap=None, count_on_device=False, flags=0):
    M, C_in = X.shape
    C_out = Wt.shape[1]
    X_d, W_d = dev(X, dtype), dev(Wt, dtype)
    b_d = torch.from_numpy(bias).cuda() if bias is not None else None
    Y = torch.full((M, C_out), float("nan"), dtype=X_d.dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rows_d = cnt = Xk = None
    if keep is not None:
        cap = len(keep) if cap is None else cap
        rows = np.zeros(max(cap, 1), dtype=np.int32)
        rows[:len(keep)] = keep
        rows_d = torch.from_numpy(rows).cuda()
        cnt = torch.tensor([len(keep)], dtype=torch.int32, device="cuda") if count_on_device else None
        Xk = torch.full((max(cap, 1), C_in), 7.0, dtype=X_d.dtype, device="cuda")
    sbp.sbp_linear_forward(dt_code(dtype), X_d, W_d, b_d, M, C_in, C_out, Y, rows_d, cnt, cap or 0, Xk, flags, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return Y, Xk


@pytest.mark.parametrize("dtype,B,H,W,C_in,C_out,with_bias,extra", [
    ("f32", 2, 16, 1, 32, 64, True, 0),
    ("f32", 3, 9, 7, 36, 68, False, 0),            # ragged tiles in every direction
    ("bf16", 2, 14, 14, 64, 32, True, 0),          # too small for the tensor-core kernel
    ("bf16", 5, 14, 14, 256, 384, True, 0),        # tensor cores: ragged last row tile, two column tiles
    ("bf16", 3, 14, 14, 264, 136, True, 29),       # reduction and columns not multiples of 64; device-side count
    ("bf16", 9, 7, 7, 128, 512, False, 3),
    ("bf16", 1, 128, 1, 768, 128, True, 0),        # one row tile exactly
])
def test_forward_and_cache_match_the_oracle(dtype, B, H, W, C_in, C_out, with_bias, extra):
    M = B * H * W
    X, Wt, _ = synth.layer_inputs(dtype, M, C_in, C_out, 41)
    bias = (synth.to_f64(synth.gaussian_tensor((C_out,), "f32", 41, 9, 0.5), "f32")).astype(np.float32) if with_bias else None
    keep, _ = oracle.sample_keep(0, B, H, W, 0.5, 5)
    cap = len(keep) + extra
    Y, Xk = _forward(dtype, X, Wt, bias, keep, cap, count_on_device=extra > 0)
    want = oracle.linear_forward(synth.to_f64(X, dtype), synth.to_f64(Wt, dtype), bias)
    assert relerr(synth.to_f64(host(Y), dtype), want) <= TOL[dtype]
    Xk_h = host(Xk)
    assert Xk_h[:len(keep)].tobytes() == oracle.forward_cache(X, keep).tobytes()       # the cache is a bit-exact gather
    assert not np.any(Xk_h[len(keep):cap].view(np.uint16 if dtype == "bf16" else np.uint32))   # padding rows cleared


def test_forward_without_cache_and_plain_fma_flag():
    dtype, M, C_in, C_out = "bf16", 700, 256, 256
    X, Wt, _ = synth.layer_inputs(dtype, M, C_in, C_out, 42)
    want = oracle.linear_forward(synth.to_f64(X, dtype), synth.to_f64(Wt, dtype))
    Y_tc, none = _forward(dtype, X, Wt, None)
    assert none is None
    Y_fma, _ = _forward(dtype, X, Wt, None, flags=sbp.SBP_FLAG_PLAIN_FMA)
    assert relerr(synth.to_f64(host(Y_tc), dtype), want) <= TOL[dtype]
    assert relerr(synth.to_f64(host(Y_fma), dtype), want) <= TOL[dtype]


def test_forward_full_size_vit_fc1_on_sampled_rows():
    # ViT-B/16 fc1 at B=64 (12544 x 768 -> 3072): the oracle computes a sample of the rows
    dtype, B, C_in, C_out = "bf16", 64, 768, 3072
    M = B * 196
    X, Wt, _ = synth.layer_inputs(dtype, M, C_in, C_out, 1002)
    bias = np.linspace(-1, 1, C_out, dtype=np.float32)
    keep, _ = oracle.sample_keep(0, B, 14, 14, 0.5, 0)
    Y, Xk = _forward(dtype, X, Wt, bias, keep)
    pick = np.unique(np.concatenate([np.arange(0, M, 97), np.arange(M - 130, M)]))
    want = oracle.linear_forward(synth.to_f64(X[pick], dtype), synth.to_f64(Wt, dtype), bias)
    assert relerr(synth.to_f64(host(Y)[pick], dtype), want) <= TOL[dtype]
    assert host(Xk).tobytes() == oracle.forward_cache(X, keep).tobytes()


def test_forward_then_backward_of_one_layer():
    # the whole SBP layer through the library: forward with cache, then the backward of Eq. 5 from that cache
    dtype, B, H, W, C_in, C_out = "bf16", 4, 14, 14, 256, 512
    M = B * H * W
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, 43)
    keep, _ = oracle.sample_keep(0, B, H, W, 0.5, 1)
    Y, Xk = _forward(dtype, X, Wt, None, keep)
    from gpu_harness import run_backward
    rows_d = torch.from_numpy(keep.astype(np.int32)).cuda()
    got = run_backward(dtype, Xk, dev(dY, dtype), dev(Wt, dtype), rows_d, len(keep))
    want = oracle.linear_backward(synth.to_f64(oracle.forward_cache(X, keep), dtype), synth.to_f64(dY, dtype),
                                  synth.to_f64(Wt, dtype), keep)
    for k in ("dW", "db"):
        assert relerr(host(got[k]), want[k]) <= TOL[dtype]
    assert relerr(synth.to_f64(host(got["dX"]), dtype), want["dX"]) <= TOL[dtype]
