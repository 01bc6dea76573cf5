"""`sbp_act_backward` against the oracle, alone and inside a packed MLP block (linear, GELU, linear with one keep set:
the gradient stays packed from the upper layer's dX through the activation into the lower layer's dY, Sec. 3.3.1)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, host, run_forward_cache, run_backward, dt_code

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,cap,valid,C", [("bf16", 500, 500, 768), ("bf16", 333, 200, 136), ("f32", 257, 257, 36), ("f32", 64, 10, 4)])
def test_gelu_backward_on_packed_rows(dtype, cap, valid, C):
    Z = synth.gaussian_tensor((cap, C), dtype, 91, 0, 1.5)
    dH = synth.gaussian_tensor((cap, C), dtype, 91, 1, 1e-2)
    cnt = torch.tensor([valid], dtype=torch.int32, device="cuda") if valid < cap else None
    out = torch.full((cap, C), float("nan"), dtype=torch.bfloat16 if dtype == "bf16" else torch.float32, device="cuda")
    sbp.sbp_act_backward(dt_code(dtype), sbp.SBP_ACT_GELU, dev(Z, dtype), dev(dH, dtype), cnt, cap, C, out)
    torch.cuda.synchronize()
    got_bits = host(out)
    got = synth.to_f64(got_bits, dtype)
    want = oracle.act_backward_gelu(synth.to_f64(Z, dtype)[:valid], synth.to_f64(dH, dtype)[:valid])
    tol = 5e-3 if dtype == "bf16" else 1e-5
    assert np.linalg.norm(got[:valid] - want) <= tol * np.linalg.norm(want)
    el = (2.0 ** -8, 1e-6) if dtype == "bf16" else (1e-5, 1e-9)
    assert (np.abs(got[:valid] - want) <= el[0] * np.abs(want) + el[1]).all()
    assert not got_bits[valid:].view(np.uint8).any()             # padding rows are zero
    assert sbp.sbp_act_backward(dt_code(dtype), 7, out, out, None, cap, C, out, check=False) == sbp.SBP_ERR_UNSUPPORTED
    assert sbp.sbp_act_backward(dt_code(dtype), 0, out, None, None, cap, C, out, check=False) == sbp.SBP_ERR_INVALID_ARG


def test_packed_mlp_block_with_gelu_matches_the_oracle_chain():
    # h = X0 W1 (+b), a = gelu(h), y = a W2: backward from dY with one keep set on both layers
    B, H, W, d, hdim, r = 6, 14, 14, 256, 1024, 0.5
    M = B * H * W
    X0 = synth.gaussian_tensor((M, d), "bf16", 71, 0, 1.0)
    W1 = synth.gaussian_tensor((d, hdim), "bf16", 71, 1, 0.05)
    W2 = synth.gaussian_tensor((hdim, d), "bf16", 71, 2, 0.02)
    dY = synth.gaussian_tensor((M, d), "bf16", 71, 3, 1e-2)
    f = synth.bf16_bits_to_f64
    keep, _ = oracle.sample_keep(0, B, H, W, r, 5)
    n = len(keep)
    # forward values the caches hold (computed by the oracle, rounded to bf16 as a bf16 forward would store them)
    Hk = synth.f64_to_bf16_bits(oracle.linear_forward(f(X0[keep]), f(W1)))            # pre-activation, kept rows
    Ak = synth.f64_to_bf16_bits(oracle.gelu(f(Hk)))                                   # input of the upper layer, kept rows
    rows_d = torch.from_numpy(keep).cuda()
    # GPU: upper layer with packed dX, activation, lower layer with packed dY
    up = run_backward("bf16", dev(Ak, "bf16"), dev(dY, "bf16"), dev(W2, "bf16"), rows_d, n, flags=sbp.SBP_FLAG_DX_COMPACT, dX_rows=n)
    dZ = torch.empty((n, hdim), dtype=torch.bfloat16, device="cuda")
    sbp.sbp_act_backward(sbp.SBP_BF16, sbp.SBP_ACT_GELU, dev(Hk, "bf16"), up["dX"], None, n, hdim, dZ)
    X0k = run_forward_cache("bf16", dev(X0, "bf16"), rows_d, n)
    low = run_backward("bf16", X0k, dZ, dev(W1, "bf16"), rows_d, n, flags=sbp.SBP_FLAG_DY_COMPACT, M=M)
    assert up["status"] == 0 and low["status"] == 0
    # oracle chain in fp64 on the same stored values
    o_up = oracle.linear_backward(f(Ak), f(dY), f(W2), keep)
    dZ_o = oracle.act_backward_gelu(f(Hk), o_up["dX"][keep])
    dZ_full = np.zeros((M, hdim)); dZ_full[keep] = dZ_o
    o_low = oracle.linear_backward(f(X0[keep]), dZ_full, f(W1), keep)
    rel = lambda g, w: float(np.linalg.norm(g - w) / np.linalg.norm(w))
    assert rel(host(up["dW"]).astype(np.float64), o_up["dW"]) <= 5e-3
    assert rel(f(host(dZ)), dZ_o) <= 5e-3
    # the lower layer sees a bf16-rounded packed gradient (two roundings on the way): still within the path's tolerance
    assert rel(host(low["dW"]).astype(np.float64), o_low["dW"]) <= 5e-3
    assert rel(host(low["db"]).astype(np.float64), o_low["db"]) <= 5e-3
    dX_bits = host(low["dX"])
    assert rel(f(dX_bits), o_low["dX"]) <= 5e-3
    dropped = np.ones(M, dtype=bool); dropped[keep] = False
    assert not dX_bits[dropped].any()
