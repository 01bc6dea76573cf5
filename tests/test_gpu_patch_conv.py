"""Stride >= kernel convolutions on the row-gather path (`sbp_patch_cache`, `sbp_linear_backward` on patch rows with
the packed input gradient, `sbp_patch_scatter`) against the fp64 oracle of the convolution itself: the cache bit for
bit, dW / db / dX within the path's tolerance and element by element, all-zero bits outside the kept patches."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, host, run_sample_keep, dt_code

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 5e-3}


def _patch_rows(X, k, s, Ho, Wo, keep):
    """The kept patches as rows (numpy indexing, no arithmetic): [len(keep), k*k*C] ordered (dh, dw, c)."""
    B, H, W, C = X.shape
    out = np.empty((len(keep), k * k * C), dtype=X.dtype)
    for i, g in enumerate(keep):
        b, ho, wo = g // (Ho * Wo), (g // Wo) % Ho, g % Wo
        out[i] = X[b, s * ho:s * ho + k, s * wo:s * wo + k, :].reshape(-1)
    return out


@pytest.mark.parametrize("dtype,B,H,W,C,Co,k,s,r,mode", [
    ("bf16", 4, 56, 56, 128, 256, 2, 2, 0.5, 0),      # ConvNeXt-B down-sampling between stages 1 and 2
    ("bf16", 3, 28, 28, 256, 512, 2, 2, 0.5, 1),      # stages 2 -> 3, grid mask
    ("bf16", 2, 14, 14, 512, 1024, 2, 2, 0.25, 0),    # stages 3 -> 4 (7 x 7 output map)
    ("bf16", 2, 15, 17, 128, 128, 2, 3, 0.5, 0),      # stride larger than the kernel: uncovered input positions
    ("bf16", 1, 64, 64, 8, 256, 4, 4, 0.5, 0),        # a 4 x 4 / stride 4 patch embedding on few channels
    ("f32", 2, 8, 8, 4, 12, 2, 2, 0.5, 0),
])
def test_patch_convolution_backward_matches_the_oracle(dtype, B, H, W, C, Co, k, s, r, mode):
    Ho, Wo = (H - k) // s + 1, (W - k) // s + 1
    Mo, Kc = B * Ho * Wo, k * k * C
    X = synth.gaussian_tensor((B, H, W, C), dtype, 500 + C, 0, 1.0)
    Wt = synth.gaussian_tensor((k, k, C, Co), dtype, 500 + C, 1, 0.05)
    dY = synth.gaussian_tensor((B, Ho, Wo, Co), dtype, 500 + C, 2, 1e-2)
    rows_d, offs_d, cap = run_sample_keep(mode, B, Ho, Wo, r, seed=2, step=5)
    keep, offs = oracle.sample_keep(mode, B, Ho, Wo, r, 2, 5, 0)
    n = len(keep)
    cap_total = B * cap
    cnt = offs_d[B:B + 1]
    code = dt_code(dtype)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    Xd, Wd, dYd = dev(X, dtype), dev(Wt.reshape(Kc, Co), dtype), dev(dY.reshape(Mo, Co), dtype)
    Xk = torch.full((cap_total, Kc), 7.0, dtype=tdt, device="cuda")
    sbp.sbp_patch_cache(code, Xd, B, H, W, C, k, s, rows_d, cnt, cap_total, Xk)
    torch.cuda.synchronize()
    got_cache = host(Xk)
    assert got_cache[:n].tobytes() == _patch_rows(X, k, s, Ho, Wo, keep).tobytes()
    assert not got_cache[n:].view(np.uint8).any()
    # the products on patch rows, input gradient kept packed
    nbytes = sbp.sbp_linear_backward_workspace_bytes(code, Mo, cap_total, Kc, Co)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW = torch.full((Kc, Co), float("nan"), dtype=torch.float32, device="cuda")
    db = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
    dXp = torch.full((cap_total, Kc), float("nan"), dtype=tdt, device="cuda")
    sbp.sbp_linear_backward(code, Xk, dYd, Wd, rows_d, cnt, Mo, cap_total, Kc, Co, dW, db, dXp, sbp.SBP_FLAG_DX_COMPACT, ws, nbytes, st)
    wsb = sbp.sbp_patch_scatter_workspace_bytes(B, H, W, k, s)
    ws2 = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    dX = torch.full((B, H, W, C), float("nan"), dtype=tdt, device="cuda")
    sbp.sbp_patch_scatter(code, dXp, B, H, W, C, k, s, rows_d, cnt, cap_total, dX, ws2, wsb, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f = lambda a: synth.to_f64(a, dtype)
    want = oracle.patch_conv_backward(f(X), f(dY), f(Wt), keep, k, s)
    rel = lambda g_, w_: float(np.linalg.norm(g_.astype(np.float64) - w_) / np.linalg.norm(w_))
    rms = lambda a: float(np.sqrt(np.mean(a * a)))
    acc = 1e-3 if dtype == "bf16" else 1e-4
    gW, gb = host(dW).reshape(k, k, C, Co), host(db)
    assert rel(gW, want["dW"]) <= TOL[dtype] and rel(gb, want["db"]) <= TOL[dtype]
    assert np.abs(gW - want["dW"]).max() <= acc * rms(want["dW"]) and np.abs(gb - want["db"]).max() <= acc * rms(want["db"])
    dX_bits = host(dX)
    gX = f(dX_bits)
    assert rel(gX, want["dX"]) <= TOL[dtype]
    zero = want["dX"] == 0.0                                      # outside the kept patches the oracle holds exact zeros
    inside = np.zeros((B, H, W), dtype=bool)
    for g_ in keep:
        b, ho, wo = g_ // (Ho * Wo), (g_ // Wo) % Ho, g_ % Wo
        inside[b, s * ho:s * ho + k, s * wo:s * wo + k] = True
    assert not dX_bits[~inside].view(np.uint16 if dtype == "bf16" else np.uint32).any()
    assert np.array_equal(zero.all(axis=3), ~inside) or dtype == "f32"


def test_patch_calls_check_their_arguments():
    t = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    r = torch.zeros(16, dtype=torch.int32, device="cuda")
    assert sbp.sbp_patch_cache(sbp.SBP_BF16, t, 1, 8, 8, 8, 2, 1, r, None, 4, t, check=False) == sbp.SBP_ERR_INVALID_ARG      # stride < k
    assert sbp.sbp_patch_cache(sbp.SBP_BF16, t, 1, 8, 8, 4, 2, 2, r, None, 4, t, check=False) == sbp.SBP_ERR_UNSUPPORTED     # 8-byte positions
    assert sbp.sbp_patch_cache(sbp.SBP_BF16, t, 1, 8, 8, 8, 2, 2, r, None, 17, t, check=False) == sbp.SBP_ERR_INVALID_ARG    # more rows than outputs
    need = sbp.sbp_patch_scatter_workspace_bytes(1, 8, 8, 2, 2)
    assert need >= 16 * 4 and need % 256 == 0
    w = torch.zeros(need, dtype=torch.uint8, device="cuda")
    assert sbp.sbp_patch_scatter(sbp.SBP_BF16, t, 1, 8, 8, 8, 2, 2, r, None, 4, t, w, need - 1, None, check=False) == sbp.SBP_ERR_WORKSPACE
    assert sbp.sbp_patch_scatter(sbp.SBP_BF16, t, 1, 8, 8, 8, 2, 2, r, None, 4, t, None, need, None, check=False) == sbp.SBP_ERR_WORKSPACE
