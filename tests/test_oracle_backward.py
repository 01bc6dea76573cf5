"""Pins for the oracle's forward cache and SBP linear backward (CPU only).

The oracle is plain C loops; these checks hold it to things fixed outside it:
an integer case worked by hand from Eq. 5, numpy matrix products on the special
cases the paper states (keep ratio 1 = Eq. 3; SBP = full backward with dY zeroed
on dropped rows; the keep/drop partition of Eq. 5), enumeration of all masks
for the expectation, and the two-layer chain of Eq. 9.
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_2210_00129_b200 import synth


def _rand_layer(M, C_in, C_out, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((M, C_in)), rng.standard_normal((C_in, C_out)),
            rng.standard_normal((M, C_out)))


def _relerr(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def test_hand_worked_integer_case():
    # B=1, N=4, C_in=2, C_out=3, kept rows {1, 3}.  All values are small integers,
    # so every product and sum below is exact in any float format.
    X = np.array([[1, 2], [3, 4], [5, 6], [7, 8]], dtype=np.float64)
    W = np.array([[1, 0, -1], [2, 1, 0]], dtype=np.float64)          # [C_in, C_out]
    dY = np.array([[1, 2, 3], [4, 5, 6], [7, 8, 9], [10, 11, 12]], dtype=np.float64)
    keep = np.array([1, 3], dtype=np.int32)
    Xk = oracle.forward_cache(X, keep)
    assert Xk.tolist() == [[3, 4], [7, 8]]
    out = oracle.linear_backward(Xk, dY, W, keep)
    # dW[i,:] = 3or4 * dY[1] + 7or8 * dY[3]
    #   i=0: 3*[4,5,6] + 7*[10,11,12] = [82, 92, 102]
    #   i=1: 4*[4,5,6] + 8*[10,11,12] = [96, 108, 120]
    assert out["dW"].tolist() == [[82, 92, 102], [96, 108, 120]]
    # db = dY[1] + dY[3]
    assert out["db"].tolist() == [14, 16, 18]
    # dX[1] = [4*1 + 6*(-1), 4*2 + 5*1] = [-2, 13];  dX[3] = [10 - 12, 20 + 11] = [-2, 31]
    assert out["dX"].tolist() == [[0, 0], [-2, 13], [0, 0], [-2, 31]]
    # an asymmetric case catches a transposed W: W is not square and not symmetric
    assert out["dW"].shape == (2, 3) and out["dX"].shape == (4, 2)


def test_forward_cache_is_a_bitwise_row_gather():
    for dtype in ("f32", "bf16"):
        X = synth.gaussian_tensor((37, 24), dtype, 5, 0, 1.0)
        keep = np.array([0, 3, 4, 17, 36], dtype=np.int32)
        got = oracle.forward_cache(X, keep)
        assert got.dtype == X.dtype and got.shape == (5, 24)
        assert got.tobytes() == X[keep].tobytes()
    empty = oracle.forward_cache(X, np.zeros(0, dtype=np.int32))
    assert empty.shape == (0, 24)


def test_keep_ratio_one_is_full_backprop():
    # Eq. 3 with numpy as the library routine
    M, C_in, C_out = 24, 5, 7
    X, W, dY = _rand_layer(M, C_in, C_out, 0)
    keep = np.arange(M, dtype=np.int32)
    out = oracle.linear_backward(X, dY, W, keep)
    assert _relerr(out["dW"], X.T @ dY) < 1e-14
    assert _relerr(out["db"], dY.sum(0)) < 1e-14
    assert _relerr(out["dX"], dY @ W.T) < 1e-14
    full = oracle.full_backward(X, dY, W)
    for k in ("dW", "db", "dX"):
        assert np.array_equal(full[k], out[k])


@pytest.mark.parametrize("M,C_in,C_out,r", [(32, 32, 64, 0.5), (60, 9, 4, 0.25), (45, 3, 17, 0.75)])
def test_sbp_equals_full_backward_with_dy_zeroed_on_dropped_rows(M, C_in, C_out, r):
    # text after Eq. 5: SBP is the full backward with dX_{i+1}^{drop} = 0
    X, W, dY = _rand_layer(M, C_in, C_out, 1)
    keep, _ = oracle.sample_keep(oracle.MASK_RANDOM, 1, M, 1, r, seed=3)
    out = oracle.linear_backward(oracle.forward_cache(X, keep), dY, W, keep)
    dYm = np.zeros_like(dY)
    dYm[keep] = dY[keep]
    assert _relerr(out["dW"], X.T @ dYm) < 1e-13
    assert _relerr(out["db"], dYm.sum(0)) < 1e-13
    assert _relerr(out["dX"], dYm @ W.T) < 1e-13


def test_dropped_rows_are_positive_zero_and_kept_rows_are_exact():
    # "either 0 or exact" (Sec. 3.2.3)
    M, C_in, C_out = 40, 6, 10
    X, W, dY = _rand_layer(M, C_in, C_out, 2)
    keep, _ = oracle.sample_keep(oracle.MASK_RANDOM, 2, 20, 1, 0.5, seed=8)
    out = oracle.linear_backward(X[keep], dY, W, keep)
    full = oracle.full_backward(X, dY, W)
    drop = np.setdiff1d(np.arange(M), keep)
    assert np.all(out["dX"][drop].view(np.uint64) == 0)          # +0.0 bit pattern
    assert np.array_equal(out["dX"][keep], full["dX"][keep])      # same sums, same order
    assert np.all(np.abs(out["dX"][keep]).sum(1) > 0)


def test_keep_plus_drop_partition_gives_the_full_gradient():
    # last line of Eq. 5
    M, C_in, C_out = 36, 8, 5
    X, W, dY = _rand_layer(M, C_in, C_out, 3)
    keep, _ = oracle.sample_keep(oracle.MASK_RANDOM, 1, 6, 6, 0.5, seed=5)
    drop = np.setdiff1d(np.arange(M), keep).astype(np.int32)
    a = oracle.linear_backward(X[keep], dY, W, keep)
    b = oracle.linear_backward(X[drop], dY, W, drop)
    full = oracle.full_backward(X, dY, W)
    assert _relerr(a["dW"] + b["dW"], full["dW"]) < 1e-13
    assert _relerr(a["db"] + b["db"], full["db"]) < 1e-13
    assert np.array_equal(a["dX"] + b["dX"], full["dX"])


def test_expectation_over_all_masks_is_keep_fraction_times_full_gradient():
    # dW^{keep} is a "stochastic approximation" of dW (text after Eq. 5); with every
    # K-subset equally likely and no rescaling (Eq. 1), E[dW_SBP] = (K/N) dW_full.
    N, K, C_in, C_out = 6, 3, 3, 4
    X, W, dY = _rand_layer(N, C_in, C_out, 4)
    acc_w = np.zeros((C_in, C_out))
    acc_b = np.zeros(C_out)
    acc_x = np.zeros((N, C_in))
    subsets = list(itertools.combinations(range(N), K))
    for s in subsets:
        keep = np.array(s, dtype=np.int32)
        o = oracle.linear_backward(X[keep], dY, W, keep)
        acc_w += o["dW"]; acc_b += o["db"]; acc_x += o["dX"]
    full = oracle.full_backward(X, dY, W)
    f = K / N
    assert np.allclose(acc_w / len(subsets), f * full["dW"], rtol=0, atol=1e-12)
    assert np.allclose(acc_b / len(subsets), f * full["db"], rtol=0, atol=1e-12)
    assert np.allclose(acc_x / len(subsets), f * full["dX"], rtol=0, atol=1e-12)


def test_two_stacked_layers_with_the_same_keep_set():
    # Eq. 9: dX_{i-1}^{keep} = dX_{i+1}^{keep} W_i^T W_{i-1}^T, dropped rows 0,
    #        dW_{i-1} = X_{i-1}^{keep T} dX_{i+1}^{keep} W_i^T
    M, C0, C1, C2 = 30, 4, 6, 5
    rng = np.random.default_rng(6)
    X0 = rng.standard_normal((M, C0))
    W0 = rng.standard_normal((C0, C1))
    W1 = rng.standard_normal((C1, C2))
    dY = rng.standard_normal((M, C2))
    X1 = X0 @ W0
    keep, _ = oracle.sample_keep(oracle.MASK_RANDOM, 1, M, 1, 0.5, seed=12)
    top = oracle.linear_backward(X1[keep], dY, W1, keep)
    bot = oracle.linear_backward(X0[keep], top["dX"], W0, keep)
    assert _relerr(bot["dW"], X0[keep].T @ dY[keep] @ W1.T) < 1e-13
    want = np.zeros((M, C0))
    want[keep] = dY[keep] @ W1.T @ W0.T
    assert _relerr(bot["dX"], want) < 1e-13
    drop = np.setdiff1d(np.arange(M), keep)
    assert np.all(bot["dX"][drop] == 0)


def test_different_keep_sets_intersect():
    # Eq. 10: the keep set reaching layer i-1 is the intersection of the two layers' sets
    M, C0, C1, C2 = 24, 3, 4, 3
    rng = np.random.default_rng(7)
    X0 = rng.standard_normal((M, C0))
    W0 = rng.standard_normal((C0, C1))
    W1 = rng.standard_normal((C1, C2))
    dY = rng.standard_normal((M, C2))
    ka, _ = oracle.sample_keep(oracle.MASK_RANDOM, 1, M, 1, 0.5, seed=1)
    kb, _ = oracle.sample_keep(oracle.MASK_RANDOM, 1, M, 1, 0.5, seed=2)
    top = oracle.linear_backward((X0 @ W0)[ka], dY, W1, ka)
    bot = oracle.linear_backward(X0[kb], top["dX"], W0, kb)
    both = np.intersect1d(ka, kb)
    nz = np.nonzero(np.abs(bot["dX"]).sum(1))[0]
    assert nz.tolist() == both.tolist()
    assert _relerr(bot["dW"], X0[both].T @ dY[both] @ W1.T) < 1e-13


def test_outputs_can_be_requested_separately_and_nothing_is_rescaled():
    M, C_in, C_out = 16, 4, 4
    X, W, dY = _rand_layer(M, C_in, C_out, 9)
    keep = np.array([2, 5, 11], dtype=np.int32)
    all3 = oracle.linear_backward(X[keep], dY, W, keep)
    only = oracle.linear_backward(X[keep], dY, W, keep, want=("dW",))
    assert list(only) == ["dW"] and np.array_equal(only["dW"], all3["dW"])
    # one kept row: dW is exactly the outer product, no 1/r factor anywhere (Eq. 1)
    one = oracle.linear_backward(X[[7]], dY, W, np.array([7], dtype=np.int32))
    assert np.array_equal(one["dW"], np.outer(X[7], dY[7]))
    assert np.array_equal(one["db"], dY[7])


def test_synthetic_inputs_are_reproducible_gaussians():
    a = synth.gaussian_f64(100001, 42, 2.0)
    b = synth.gaussian_f64(100001, 42, 2.0)
    assert np.array_equal(a, b)
    assert np.array_equal(a[:1001], synth.gaussian_f64(1001, 42, 2.0))
    assert abs(a.mean()) < 0.03 and abs(a.std() - 2.0) < 0.03
    bits = synth.f64_to_bf16_bits(np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0]))
    # 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 is a tie -> even (1 + 2^-6)
    assert bits.tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x0000]
    assert synth.bf16_bits_to_f64(bits).tolist() == [1.0, 1.0, 1.015625, -2.5, 0.0]


# ---------------------------------------------------------------- forward (Eq. 2, Eq. 4)
def test_forward_hand_worked_integers():
    X = np.array([[1, 2], [0, -1], [3, 1]], dtype=np.float64)
    W = np.array([[2, 0, 1], [1, -1, 4]], dtype=np.float64)
    b = np.array([10, 20, 30], dtype=np.float64)
    assert oracle.linear_forward(X, W).tolist() == [[4, -2, 9], [-1, 1, -4], [7, -1, 7]]
    assert oracle.linear_forward(X, W, b).tolist() == [[14, 18, 39], [9, 21, 26], [17, 19, 37]]


def test_forward_equals_library_matmul_and_splits_by_rows():
    rng = np.random.default_rng(3)
    X, W, b = rng.standard_normal((37, 19)), rng.standard_normal((19, 23)), rng.standard_normal(23)
    Y = oracle.linear_forward(X, W, b)
    assert np.allclose(Y, X @ W + b, rtol=1e-13, atol=1e-13)
    assert not np.allclose(Y, X @ W, atol=1e-3) and not np.allclose(Y, (W.T @ X.T).T[:, ::-1] + b, atol=1e-3)
    # Eq. 4: the forward of the kept rows and of the dropped rows, put back in place, is the full forward
    keep = np.sort(rng.choice(37, 18, replace=False))
    drop = np.setdiff1d(np.arange(37), keep)
    Z = np.empty_like(Y)
    Z[keep] = oracle.linear_forward(X[keep], W, b)
    Z[drop] = oracle.linear_forward(X[drop], W, b)
    assert np.array_equal(Z, Y)


def test_forward_and_backward_are_adjoint():
    # <Y(W + E) - Y(W), G> = <E, dW(G)> and <Y(X + D) - Y(X), G> = <D, dX(G)> exactly (bilinearity, Eq. 2 and Eq. 3)
    rng = np.random.default_rng(4)
    X, W = rng.integers(-3, 4, (11, 6)).astype(np.float64), rng.integers(-3, 4, (6, 5)).astype(np.float64)
    G, E, D = (rng.integers(-3, 4, s).astype(np.float64) for s in ((11, 5), (6, 5), (11, 6)))
    full = oracle.full_backward(X, G, W)
    assert np.sum((oracle.linear_forward(X, W + E) - oracle.linear_forward(X, W)) * G) == np.sum(E * full["dW"])
    assert np.sum((oracle.linear_forward(X + D, W) - oracle.linear_forward(X, W)) * G) == np.sum(D * full["dX"])
    b = rng.integers(-3, 4, 5).astype(np.float64)
    assert np.sum((oracle.linear_forward(X, W, b) - oracle.linear_forward(X, W)) * G) == np.sum(b * full["db"])
