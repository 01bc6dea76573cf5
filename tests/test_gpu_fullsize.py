"""Full-size workloads (the shapes the benchmark times), every output element against the fp64 oracle.

Beside the relative Frobenius bound of the small cases, each element has its own bound, so that one
wrong entry (a clipped tile edge, a k-block left out, a row stored twice) fails even where it would
drown in the norm of a 768 x 3072 matrix:
  dW, db (fp32 out of fp32 accumulators):  |got - want| <= 1e-3 * rms(want)
      (one row of 6272 left out of a sum moves an entry by about 1e-2 rms; the arithmetic's own error is
      a few 1e-6 rms per thousand accumulator updates)
  dX (one rounding to bf16):               |got - want| <= 2^-8 |want| + 1e-3 * rms(want)
The shapes are chosen so that every block of the persistent kernels runs several tiles (five and more on
the ConvNeXt and detection maps), with ragged last tiles and ragged per-sample counts among them; the last two run
the form that pairs blocks on the two-SM tensor-core instructions.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, host, run_sample_keep, run_forward_cache, run_backward

pytestmark = pytest.mark.gpu

CASES = [
    # name, B, H, W, C_in, C_out, keep ratio, mask mode
    ("vit_b16_fc1", 64, 14, 14, 768, 3072, 0.5, 0),
    ("vit_b16_fc2_b128_r025", 128, 14, 14, 3072, 768, 0.25, 0),
    ("vit_b16_proj_b128_r075", 128, 14, 14, 768, 768, 0.75, 0),
    ("convnext_s1_pw1_grid", 64, 56, 56, 128, 512, 0.5, 1),
    ("convnext_s2_pw2_random", 64, 28, 28, 1024, 256, 0.5, 0),
    ("convnext_s4_pw2_grid_ragged", 64, 7, 7, 4096, 1024, 0.5, 1),
    ("detection_s1_pw1", 2, 200, 334, 128, 512, 0.5, 0),
    ("detection_s1_pw2", 2, 200, 334, 512, 128, 0.5, 0),
    # from 8192 kept rows on wide layers run on pairs of SMs (256-row tiles, half of the dense operand per block)
    ("vit_b16_fc1_b128_pairs", 128, 14, 14, 768, 3072, 0.5, 0),
    ("pairs_odd_row_tiles_ragged_columns", 100, 14, 14, 768, 1160, 0.5, 0),     # 77 row tiles: the last pair has a dead half
]


def check_against_oracle(got, want, dX_bits, keep, M, tag=""):
    rel = lambda g, w: float(np.linalg.norm(g - w) / np.linalg.norm(w))
    rms = lambda a: float(np.sqrt(np.mean(a * a)))
    report = {}
    for k in ("dW", "db"):
        if k not in want:
            continue
        g = host(got[k]).astype(np.float64)
        report[k] = (rel(g, want[k]), float(np.abs(g - want[k]).max() / rms(want[k])))
        assert report[k][0] <= 5e-3, (tag, k, report[k])
        assert report[k][1] <= 1e-3, (tag, k, report[k])
    if "dX" in want:
        g = synth.bf16_bits_to_f64(dX_bits)
        w = want["dX"]
        report["dX"] = rel(g, w)
        assert report["dX"] <= 5e-3, (tag, report)
        kept = w[keep]
        assert (np.abs(g[keep] - kept) <= 2.0 ** -8 * np.abs(kept) + 1e-3 * rms(kept)).all(), (tag, "dX element")
        dropped = np.ones(M, dtype=bool)
        dropped[keep] = False
        assert not dX_bits[dropped].any(), (tag, "dropped rows must be +0.0")
    return report


@pytest.mark.parametrize("name,B,H,W,C_in,C_out,r,mode", CASES)
def test_full_size_every_element_against_the_oracle(name, B, H, W, C_in, C_out, r, mode):
    M = B * H * W
    X, Wt, dY = synth.layer_inputs("bf16", M, C_in, C_out, 1000 + len(name))
    rows_d, offs_d, cap = run_sample_keep(mode, B, H, W, r, seed=0, step=3)
    keep, offs = oracle.sample_keep(mode, B, H, W, r, 0, 3, 0)
    M_keep = len(keep)
    assert np.array_equal(host(offs_d), offs) and np.array_equal(host(rows_d)[:M_keep], keep)
    cnt = offs_d[B:B + 1]
    Xk_d = run_forward_cache("bf16", dev(X, "bf16"), rows_d, B * cap, cnt)
    got = run_backward("bf16", Xk_d, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, B * cap, cnt)
    assert got["status"] == 0
    Xk = oracle.forward_cache(X, keep)
    assert host(Xk_d)[:M_keep].tobytes() == Xk.tobytes()
    want = oracle.linear_backward(synth.bf16_bits_to_f64(Xk), synth.bf16_bits_to_f64(dY), synth.bf16_bits_to_f64(Wt), keep)
    report = check_against_oracle(got, want, host(got["dX"]), keep, M, name)
    print(name, report)
