"""Full-size workloads (the shapes the benchmark times), checked on sampled outputs.

The fp64 oracle is too slow to produce whole gradients at these sizes, so every check below
computes individual outputs one by one in fp64 from their definition (Eq. 5) - sampled entries of
dW, sampled rows of dX - plus what is cheap in full: the keep indices, db, and the all-zero
bit pattern of every dropped row of dX.
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
    ("convnext_s1_pw1_grid", 64, 56, 56, 128, 512, 0.5, 1),
    ("convnext_s4_pw2_grid_ragged", 64, 7, 7, 4096, 1024, 0.5, 1),
    ("detection_s1_pw2", 2, 200, 334, 512, 128, 0.5, 0),
]


@pytest.mark.parametrize("name,B,H,W,C_in,C_out,r,mode", CASES)
def test_full_size_sampled_outputs(name, B, H, W, C_in, C_out, r, mode):
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
    assert host(Xk_d)[:M_keep].tobytes() == X[keep].tobytes()

    rng = np.random.default_rng(7)
    Xk64 = synth.bf16_bits_to_f64(X[keep])
    # db: every column, exact definition
    dYk64 = synth.bf16_bits_to_f64(dY[keep])
    db_want = dYk64.sum(axis=0)
    db_got = host(got["db"]).astype(np.float64)
    assert np.linalg.norm(db_got - db_want) <= 5e-3 * np.linalg.norm(db_want)
    # dW: sampled entries, each a dot product over the kept rows
    ii = rng.integers(0, C_in, 48); jj = rng.integers(0, C_out, 48)
    ii[:4] = [0, C_in - 1, 0, C_in - 1]; jj[:4] = [0, C_out - 1, C_out - 1, 0]
    dW_got = host(got["dW"]).astype(np.float64)[ii, jj]
    dW_want = np.einsum("mk,mk->k", Xk64[:, ii], dYk64[:, jj])
    assert np.linalg.norm(dW_got - dW_want) <= 5e-3 * np.linalg.norm(dW_want)
    # dX: sampled kept rows (first, last, random) against dY_row . W^T; all dropped rows all-zero bits
    W64 = synth.bf16_bits_to_f64(Wt)
    dX_bits = host(got["dX"])
    pick = np.unique(np.concatenate([[0, M_keep - 1], rng.integers(0, M_keep, 24)]))
    want_rows = dYk64[pick] @ W64.T
    got_rows = synth.bf16_bits_to_f64(dX_bits[keep[pick]])
    assert np.linalg.norm(got_rows - want_rows) <= 5e-3 * np.linalg.norm(want_rows)
    dropped = np.ones(M, dtype=bool); dropped[keep] = False
    assert not dX_bits[dropped].any()
    assert dX_bits[keep].any(axis=1).all()          # no kept row was left as zeros
