"""Pins for the oracle's attention functions (CPU only).

The backward is checked against things that are not itself: central differences of the forward, the full
attention backward written out as matrix products (the supplementary's gradient equations), the paper's
statement that with queries dropped the kept query rows get their exact gradient and the key gradient is
Q_keep^T dM_keep / sqrt(d), attention among the gathered kept tokens, and the memory ratios the paper prints.
"""
import os

import numpy as np
import pytest

import oracle


def _lists(B, n, sets):
    """Per-sample token subsets (local positions) -> global row lists with offsets."""
    rows, offs = [], [0]
    for b in range(B):
        rows += [b * n + t for t in sets[b]]
        offs.append(len(rows))
    return np.array(rows, dtype=np.int32), np.array(offs, dtype=np.int32)


def _all(B, n):
    return _lists(B, n, [list(range(n))] * B)


def _full_backward_numpy(Q, K, V, dA, B, n, heads):
    """Full attention backward per (sample, head) as matrix products: S = softmax(Q K^T / sqrt(d)),
    dV = S^T dA, dS = dA V^T, dM = S * (dS - rowsum(S * dS)), dQ = dM K / sqrt(d), dK = dM^T Q / sqrt(d)."""
    C = Q.shape[1]
    d = C // heads
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(Q), np.zeros_like(Q)
    dM_all = {}
    for b in range(B):
        for h in range(heads):
            sl = (slice(b * n, (b + 1) * n), slice(h * d, (h + 1) * d))
            q, k, v, da = Q[sl], K[sl], V[sl], dA[sl]
            m = q @ k.T / np.sqrt(d)
            s = np.exp(m - m.max(axis=1, keepdims=True))
            s /= s.sum(axis=1, keepdims=True)
            ds = da @ v.T
            dm = s * (ds - (s * ds).sum(axis=1, keepdims=True))
            dQ[sl], dK[sl], dV[sl] = dm @ k / np.sqrt(d), dm.T @ q / np.sqrt(d), s.T @ da
            dM_all[(b, h)] = (dm, s)
    return dQ, dK, dV, dM_all


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_backward_is_the_gradient_of_the_forward_by_central_differences():
    B, n, heads, d = 2, 6, 2, 3
    M, C = B * n, heads * d
    Q, K, V, G = (_rand((M, C), s) for s in range(4))
    qr, qo = _lists(B, n, [[0, 2, 5], [1, 3, 4, 5]])
    kr, ko = _lists(B, n, [[1, 2, 3, 4], [0, 5]])
    loss = lambda q, k, v: float((oracle.attention_forward(q, k, v, qr, qo, kr, ko, heads) * G).sum())
    dQ, dK, dV = oracle.attention_backward(Q, K, V, G, qr, qo, kr, ko, heads)
    eps = 1e-6
    for T, dT, which in ((Q, dQ, 0), (K, dK, 1), (V, dV, 2)):
        num = np.zeros_like(T)
        for idx in np.ndindex(*T.shape):
            args = [Q.copy(), K.copy(), V.copy()]
            args[which][idx] += eps
            up = loss(*args)
            args[which][idx] -= 2 * eps
            num[idx] = (up - loss(*args)) / (2 * eps)
        assert np.allclose(dT, num, rtol=1e-6, atol=1e-8), which
    # gradients are dropped outside the lists
    assert not dQ[[1, 3, 4, 6, 8]].any() and not dK[[0, 5, 7, 8, 9, 10]].any() and not dV[[0, 5, 7, 8, 9, 10]].any()


def test_all_tokens_equal_the_full_backward_written_as_matrix_products():
    B, n, heads, d = 3, 9, 2, 4
    Q, K, V, dA = (_rand((B * n, heads * d), 10 + s) for s in range(4))
    rows, offs = _all(B, n)
    got = oracle.attention_backward(Q, K, V, dA, rows, offs, rows, offs, heads)
    want = _full_backward_numpy(Q, K, V, dA, B, n, heads)[:3]
    for g, w in zip(got, want):
        assert np.allclose(g, w, rtol=1e-12, atol=1e-13)
    # the forward too: A = S V
    A = oracle.attention_forward(Q, K, V, rows, offs, rows, offs, heads)
    d_ = d
    for b in range(B):
        for h in range(heads):
            sl = (slice(b * n, (b + 1) * n), slice(h * d_, (h + 1) * d_))
            m = Q[sl] @ K[sl].T / np.sqrt(d_)
            s = np.exp(m - m.max(axis=1, keepdims=True)); s /= s.sum(axis=1, keepdims=True)
            assert np.allclose(A[sl], s @ V[sl], rtol=1e-12, atol=1e-13)


def test_drop_query_only_kept_query_rows_are_exact_and_the_key_gradient_uses_kept_rows():
    # the supplementary's worked case: dM of dropped queries is zero; dQ_keep is the exact gradient, dQ_drop = 0,
    # dK = Q_keep^T dM_keep / sqrt(d); with dA non-zero only on kept rows (the chain rule inside a block), dV = S_keep^T dA_keep
    B, n, heads, d = 2, 8, 2, 4
    Q, K, V, dA = (_rand((B * n, heads * d), 20 + s) for s in range(4))
    keep = [[0, 3, 4, 7], [1, 2, 6]]
    qr, qo = _lists(B, n, keep)
    kr, ko = _all(B, n)
    dQ, dK, dV = oracle.attention_backward(Q, K, V, dA, qr, qo, kr, ko, heads)
    fQ, fK, fV, dM = _full_backward_numpy(Q, K, V, dA, B, n, heads)
    assert np.allclose(dQ[qr], fQ[qr], rtol=1e-12, atol=1e-13)
    dropped = np.setdiff1d(np.arange(B * n), qr)
    assert not dQ[dropped].any()
    for b in range(B):
        for h in range(heads):
            dm, s = dM[(b, h)]
            kk = keep[b]
            sl = (slice(b * n, (b + 1) * n), slice(h * d, (h + 1) * d))
            assert np.allclose(dK[sl], dm[kk].T @ Q[sl][kk] / np.sqrt(d), rtol=1e-12, atol=1e-13)
            assert np.allclose(dV[sl], s[kk].T @ dA[sl][kk], rtol=1e-12, atol=1e-13)
    assert not np.allclose(dK, fK)          # an estimate, not the exact key gradient


def test_drop_qkv_is_attention_among_the_gathered_kept_tokens():
    B, n, heads, d = 2, 10, 3, 4
    Q, K, V, dA = (_rand((B * n, heads * d), 30 + s) for s in range(4))
    keep = [[0, 2, 3, 8, 9], [1, 4, 5, 6, 7]]
    rows, offs = _lists(B, n, keep)
    dQ, dK, dV = oracle.attention_backward(Q, K, V, dA, rows, offs, rows, offs, heads)
    g = lambda T: T[rows]
    sub = _full_backward_numpy(g(Q), g(K), g(V), g(dA), B, 5, heads)[:3]       # both samples keep 5 tokens
    for got, want in zip((dQ, dK, dV), sub):
        assert np.allclose(got[rows], want, rtol=1e-12, atol=1e-13)
        assert not got[np.setdiff1d(np.arange(B * n), rows)].any()
    A = oracle.attention_forward(Q, K, V, rows, offs, rows, offs, heads)
    assert not A[np.setdiff1d(np.arange(B * n), rows)].any()


def test_softmax_rows_are_shift_invariant_and_value_gradients_sum_to_da():
    # adding a constant to every key along q's direction shifts each row of M uniformly: S and all gradients but dK's
    # q-component are unchanged; and since every row of S sums to one, sum_j dV_j = sum_i dA_i
    B, n, heads, d = 1, 7, 1, 5
    Q, K, V, dA = (_rand((n, d), 40 + s) for s in range(4))
    rows, offs = _all(B, n)
    dQ, dK, dV = oracle.attention_backward(Q, K, V, dA, rows, offs, rows, offs, heads)
    assert np.allclose(dV.sum(axis=0), dA.sum(axis=0), rtol=1e-12)
    assert np.allclose((dK).sum(axis=0), 0.0, atol=1e-12)      # rows of dM sum to zero


def test_memory_ratios_the_paper_prints(golden_dir):
    printed = {}
    with open(os.path.join(golden_dir, "attention_memory_ratios.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                m, r, v = line.split()
                printed[(m, float(r))] = float(v)
    d, n = 64.0, 196.0
    # Drop Query only: the term count reproduces the printed numbers (0.610, 0.414 against 0.61, 0.42)
    for r in (0.5, 0.25):
        assert abs(oracle.attention_memory_ratio(oracle.ATTN_DROP_QUERY, d, n, r) - printed[("drop_query", r)]) < 0.01
    # Drop QKV: the printed 0.46 / 0.22 are what the equation's right-hand side gives as printed, r (3 + 2 r x) / (3 + 2 x)
    # with x = d / n; the term count on its left-hand side, (3 r h d n + 2 r^2 h n n) / (3 h d n + 2 h n n), needs x = n / d
    # and gives 0.33 / 0.12.  Both facts are pinned; the count is what the oracle returns.
    x = d / n
    for r in (0.5, 0.25):
        assert abs(r * (3 + 2 * r * x) / (3 + 2 * x) - printed[("drop_qkv", r)]) < 0.006
        count = oracle.attention_memory_ratio(oracle.ATTN_DROP_QKV, d, n, r)
        assert abs(count - r * (3 + 2 * r * (n / d)) / (3 + 2 * (n / d))) < 1e-12
        assert count < printed[("drop_qkv", r)]
    assert abs(oracle.attention_memory_ratio(oracle.ATTN_DROP_QKV, d, n, 1.0) - 1.0) < 1e-12
    assert abs(oracle.attention_memory_ratio(oracle.ATTN_DROP_QUERY, d, n, 1.0) - 1.0) < 1e-12
