"""Pins for the oracle's stride >= kernel convolution under SBP (Sec. 3.2.2: with s >= k the layer behaves like a
point-wise one).  Checked against: a hand-worked 4 x 4 map with small integers, the already pinned point-wise oracle
after a space-to-depth rearrangement done here in numpy, central differences of the forward, and the convolution
gradient written as tensor contractions (Eq. 6 for this case)."""
import numpy as np

import oracle


def _space_to_depth(X, k):
    """[B, H, W, C] -> [B * H/k * W/k, k * k * C]: row = output position, columns ordered (dh, dw, c)."""
    B, H, W, C = X.shape
    return X.reshape(B, H // k, k, W // k, k, C).transpose(0, 1, 3, 2, 4, 5).reshape(B * (H // k) * (W // k), k * k * C)


def test_hand_worked_4x4_map():
    # one sample, one input channel, one output channel, 2 x 2 kernel, stride 2: outputs (0,0), (0,1), (1,0), (1,1)
    X = np.arange(16, dtype=np.float64).reshape(1, 4, 4, 1)
    Wt = np.array([1.0, 2.0, 3.0, 4.0]).reshape(2, 2, 1, 1)
    assert oracle.patch_conv_forward(X, Wt, None, 2, 2).reshape(-1).tolist() == [0 + 2 + 12 + 20, 2 + 6 + 18 + 28, 8 + 18 + 36 + 52, 10 + 22 + 42 + 60]
    dY = np.array([1.0, 10.0, 100.0, 1000.0]).reshape(1, 2, 2, 1)
    g = oracle.patch_conv_backward(X, dY, Wt, np.array([1, 2], dtype=np.int32), 2, 2)      # keep outputs (0,1) and (1,0)
    # dW[dh, dw] = 10 * X[patch (0,1)] + 100 * X[patch (1,0)]
    assert g["dW"].reshape(-1).tolist() == [10 * 2 + 100 * 8, 10 * 3 + 100 * 9, 10 * 6 + 100 * 12, 10 * 7 + 100 * 13]
    assert g["db"].tolist() == [110.0]
    want = np.zeros((4, 4))
    want[0:2, 2:4] = 10 * Wt.reshape(2, 2)
    want[2:4, 0:2] = 100 * Wt.reshape(2, 2)
    assert np.array_equal(g["dX"].reshape(4, 4), want)


def test_equals_the_pointwise_oracle_after_space_to_depth():
    rng = np.random.default_rng(0)
    B, H, W, C, Co, k = 2, 6, 8, 3, 5, 2
    X, Wt = rng.standard_normal((B, H, W, C)), rng.standard_normal((k, k, C, Co))
    dY = rng.standard_normal((B, H // k, W // k, Co))
    keep = np.sort(rng.choice(B * (H // k) * (W // k), 11, replace=False)).astype(np.int32)
    g = oracle.patch_conv_backward(X, dY, Wt, keep, k, k)
    Xr = _space_to_depth(X, k)
    pw = oracle.linear_backward(Xr[keep], dY.reshape(-1, Co), Wt.reshape(k * k * C, Co), keep)
    assert np.allclose(g["dW"].reshape(k * k * C, Co), pw["dW"], rtol=1e-13, atol=1e-13)
    assert np.allclose(g["db"], pw["db"], rtol=1e-13, atol=1e-13)
    assert np.allclose(_space_to_depth(g["dX"], k), pw["dX"], rtol=1e-13, atol=1e-13)
    # and the forward is the point-wise forward on the rearranged input
    assert np.allclose(oracle.patch_conv_forward(X, Wt, None, k, k).reshape(-1, Co), oracle.linear_forward(Xr, Wt.reshape(k * k * C, Co)))


def test_full_keep_is_the_gradient_of_the_forward_and_stride_may_exceed_the_kernel():
    rng = np.random.default_rng(1)
    B, H, W, C, Co, k, s = 1, 7, 8, 2, 3, 2, 3            # stride 3 > kernel 2: some input positions feed no output
    X, Wt, bias = rng.standard_normal((B, H, W, C)), rng.standard_normal((k, k, C, Co)), rng.standard_normal(Co)
    Ho, Wo = (H - k) // s + 1, (W - k) // s + 1
    G = rng.standard_normal((B, Ho, Wo, Co))
    keep = np.arange(B * Ho * Wo, dtype=np.int32)
    g = oracle.patch_conv_backward(X, G, Wt, keep, k, s)
    loss = lambda x, w, b_: float((oracle.patch_conv_forward(x, w, b_, k, s) * G).sum())
    eps = 1e-6
    for T, dT, which in ((X, g["dX"], 0), (Wt, g["dW"], 1), (bias, g["db"], 2)):
        num = np.zeros_like(T)
        for idx in np.ndindex(*T.shape):
            args = [X.copy(), Wt.copy(), bias.copy()]
            args[which][idx] += eps
            up = loss(*args)
            args[which][idx] -= 2 * eps
            num[idx] = (up - loss(*args)) / (2 * eps)
        assert np.allclose(dT, num, rtol=1e-6, atol=1e-8), which
    # input positions outside every patch (row 6 since rows 0-1 and 3-4 are covered; columns 2, 5) get no gradient
    assert not g["dX"][0, 2].any() and not g["dX"][0, :, 2].any() and not g["dX"][0, 5:].any()
    # the same gradient as tensor contractions over the patches (Eq. 6 for non-overlapping patches)
    P = np.stack([[X[0, s * ho:s * ho + k, s * wo:s * wo + k] for wo in range(Wo)] for ho in range(Ho)])    # [Ho, Wo, k, k, C]
    assert np.allclose(g["dW"], np.einsum("hwabc,hwj->abcj", P, G[0]), rtol=1e-12, atol=1e-12)


def test_dropped_output_positions_leave_their_patches_zero_and_kept_ones_exact():
    rng = np.random.default_rng(2)
    B, H, W, C, Co, k = 2, 4, 4, 2, 3, 2
    X, Wt = rng.standard_normal((B, H, W, C)), rng.standard_normal((k, k, C, Co))
    dY = rng.standard_normal((B, 2, 2, Co))
    keep = np.array([0, 3, 5], dtype=np.int32)
    part = oracle.patch_conv_backward(X, dY, Wt, keep, k, k)
    full = oracle.patch_conv_backward(X, dY, Wt, np.arange(8, dtype=np.int32), k, k)
    sd_p, sd_f = _space_to_depth(part["dX"], k), _space_to_depth(full["dX"], k)
    assert np.array_equal(sd_p[keep], sd_f[keep])                       # exact on the kept patches
    assert not sd_p[np.setdiff1d(np.arange(8), keep)].any()             # zero on the dropped ones
    rest = oracle.patch_conv_backward(X, dY, Wt, np.setdiff1d(np.arange(8), keep).astype(np.int32), k, k)
    assert np.allclose(part["dW"] + rest["dW"], full["dW"]) and np.allclose(part["db"] + rest["db"], full["db"])
