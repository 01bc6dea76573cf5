"""`sbp_attention_backward` (attention with the gradient kept on token subsets, Sec. 4) against the fp64 oracle:
relative Frobenius error within the bf16 tolerance for dQ, dK, dV, every element within its own bound, and all-zero
bit patterns in the rows whose gradient is dropped."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, host, run_sample_keep

pytestmark = pytest.mark.gpu

D = 64


def _inputs(M, heads, seed, fused):
    C = heads * D
    Q = synth.gaussian_tensor((M, C), "bf16", seed, 0, 1.0)
    K = synth.gaussian_tensor((M, C), "bf16", seed, 1, 1.0)
    V = synth.gaussian_tensor((M, C), "bf16", seed, 2, 1.0)
    dA = synth.gaussian_tensor((M, C), "bf16", seed, 3, 1e-2)
    return Q, K, V, dA


def _identity(B, N):
    return np.arange(B * N, dtype=np.int32), (np.arange(B + 1) * N).astype(np.int32)


def _run(B, N, heads, Q, K, V, dA, q_list, kv_list, flags, max_kept, fused):
    """q_list / kv_list: (rows, offsets) device tensors or None."""
    M, C = B * N, heads * D
    if fused:     # the three slices of one [M, 3C] projection output, gradients into one [M, 3C] buffer
        qkv = dev(np.concatenate([Q, K, V], axis=1), "bf16")
        Qd, Kd, Vd, ld = qkv[:, :C], qkv[:, C:2 * C], qkv[:, 2 * C:], 3 * C
        out = torch.full((M, 3 * C), float("nan"), dtype=torch.bfloat16, device="cuda")
        dQ, dK, dV = out[:, :C], out[:, C:2 * C], out[:, 2 * C:]
    else:
        Qd, Kd, Vd, ld = dev(Q, "bf16"), dev(K, "bf16"), dev(V, "bf16"), C
        dQ, dK, dV = (torch.full((M, C), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(3))
    dAd = dev(dA, "bf16")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    qr, qo = q_list if q_list is not None else (None, None)
    kr, ko = kv_list if kv_list is not None else (None, None)
    sbp.sbp_attention_backward(sbp.SBP_BF16, Qd, Kd, Vd, ld, dAd, C, qr, qo, kr, ko, B, N, heads, D, max_kept, dQ, dK, dV, ld,
                               flags, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    back = lambda t: host(t.contiguous())
    return back(dQ), back(dK), back(dV)


def _check(got_bits, want, rows_in_set, M, name):
    got = synth.bf16_bits_to_f64(got_bits)
    rel = float(np.linalg.norm(got - want) / np.linalg.norm(want))
    assert rel <= 5e-3, (name, rel)
    inside = want[rows_in_set]
    rms = float(np.sqrt(np.mean(inside * inside)))
    # one rounding of the result to bf16 plus the bf16 rounding of the softmax / dM blocks between the products
    assert (np.abs(got[rows_in_set] - inside) <= 2.0 ** -7 * np.abs(inside) + 2e-2 * rms).all(), name
    outside = np.ones(M, dtype=bool)
    outside[rows_in_set] = False
    assert not got_bits[outside].any(), (name, "rows outside the token set must be +0.0")
    return rel


@pytest.mark.parametrize("B,H,W,heads,r,mode,variant,fused", [
    (3, 14, 14, 2, 0.5, 0, "qkv", False),          # Drop QKV: 98 kept tokens, one tile each way
    (3, 14, 14, 3, 0.25, 0, "qkv", True),          # 49 kept tokens, fused projection layout
    (2, 14, 14, 12, 0.5, 0, "qkv", True),          # ViT-B/16 heads
    (2, 14, 14, 2, 0.75, 0, "qkv", False),         # 147 kept tokens: two query tiles and two key tiles
    (2, 14, 14, 2, 1.0, 0, "full", False),         # keep ratio 1: ordinary attention backward, 196 tokens
    (3, 14, 14, 2, 0.5, 0, "query", False),        # Drop Query only: 98 queries against all 196 keys
    (2, 14, 14, 2, 0.25, 0, "query", True),
    (5, 7, 7, 4, 0.5, 1, "qkv", False),            # grid mask on an odd map: 24 or 25 kept tokens per sample
    (2, 16, 16, 1, 0.5, 1, "qkv", False),          # 256 tokens, 128 kept: exactly one full tile
    (2, 16, 16, 2, 1.0, 0, "full", True),          # 256 tokens on both sides: the largest supported
    (2, 14, 14, 2, 0.5, 0, "mixed", False),        # queries at 0.75, keys / values at 0.5 (their own lists)
])
def test_attention_backward_matches_the_oracle(B, H, W, heads, r, mode, variant, fused):
    N, M = H * W, B * H * W
    Q, K, V, dA = _inputs(M, heads, 300 + heads + int(100 * r), fused)
    f = lambda a: synth.bf16_bits_to_f64(a)
    all_rows, all_offs = _identity(B, N)
    if variant == "full":
        q_np = kv_np = (all_rows, all_offs)
        got = _run(B, N, heads, Q, K, V, dA, None, None, sbp.SBP_FLAG_ATTN_ALL_KEYS, 0, fused)
    else:
        rows_d, offs_d, cap = run_sample_keep(mode, B, H, W, r, seed=4, step=1)
        keep, offs = oracle.sample_keep(mode, B, H, W, r, 4, 1, 0)
        assert np.array_equal(host(offs_d), offs)
        q_np = (keep, offs)
        if variant == "qkv":
            kv_np = q_np
            got = _run(B, N, heads, Q, K, V, dA, (rows_d, offs_d), None, 0, cap, fused)
        elif variant == "query":
            kv_np = (all_rows, all_offs)
            got = _run(B, N, heads, Q, K, V, dA, (rows_d, offs_d), None, sbp.SBP_FLAG_ATTN_ALL_KEYS, cap, fused)
        else:
            q_rows_d, q_offs_d, qcap = run_sample_keep(mode, B, H, W, 0.75, seed=9, step=0)
            q_np = oracle.sample_keep(mode, B, H, W, 0.75, 9, 0, 0)
            kv_np = (keep, offs)
            got = _run(B, N, heads, Q, K, V, dA, (q_rows_d, q_offs_d), (rows_d, offs_d), 0, max(cap, qcap), fused)
    want = oracle.attention_backward(f(Q), f(K), f(V), f(dA), q_np[0], q_np[1], kv_np[0], kv_np[1], heads)
    errs = [_check(got[0], want[0], q_np[0], M, "dQ"), _check(got[1], want[1], kv_np[0], M, "dK"),
            _check(got[2], want[2], kv_np[0], M, "dV")]
    print(variant, r, errs)


def test_kept_rows_only_leaves_the_other_rows_alone():
    B, H, W, heads = 3, 14, 14, 2
    N, M = H * W, B * H * W
    Q, K, V, dA = _inputs(M, heads, 55, False)
    rows_d, offs_d, cap = run_sample_keep(0, B, H, W, 0.5, seed=8)
    keep = host(rows_d)[:int(host(offs_d)[-1])]
    full = _run(B, N, heads, Q, K, V, dA, (rows_d, offs_d), None, 0, cap, False)
    part = _run(B, N, heads, Q, K, V, dA, (rows_d, offs_d), None, sbp.SBP_FLAG_ATTN_KEPT_ROWS_ONLY, cap, False)
    other = np.ones(M, dtype=bool); other[keep] = False
    nan_bits = host(torch.full((1,), float("nan"), dtype=torch.bfloat16, device="cuda"))[0]
    for a, b in zip(full, part):
        assert np.array_equal(a[keep], b[keep])
        assert (b[other] == nan_bits).all()              # untouched: still the fill value of the test's output buffers


def test_attention_backward_is_deterministic_and_checks_its_arguments():
    B, H, W, heads = 2, 14, 14, 2
    N, M, C = H * W, B * H * W, heads * D
    Q, K, V, dA = _inputs(M, heads, 77, False)
    rows_d, offs_d, cap = run_sample_keep(0, B, H, W, 0.5, seed=1)
    a = _run(B, N, heads, Q, K, V, dA, (rows_d, offs_d), None, 0, cap, False)
    b = _run(B, N, heads, Q, K, V, dA, (rows_d, offs_d), None, 0, cap, False)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    t = torch.zeros((M, C), dtype=torch.bfloat16, device="cuda")
    call = lambda **kw: sbp.sbp_attention_backward(kw.get("dt", sbp.SBP_BF16), t, t, t, kw.get("ld", C), t, C, kw.get("qr", rows_d),
                                                   kw.get("qo", offs_d), None, None, B, kw.get("N", N), heads, kw.get("d", D),
                                                   kw.get("cap", cap), t, t, t, C, kw.get("flags", 0), None, check=False)
    assert call(d=32) == sbp.SBP_ERR_UNSUPPORTED
    assert call(dt=sbp.SBP_F32) == sbp.SBP_ERR_UNSUPPORTED
    assert call(ld=C - 8) == sbp.SBP_ERR_INVALID_ARG
    assert call(qo=None) == sbp.SBP_ERR_INVALID_ARG
    assert call(cap=0) == sbp.SBP_ERR_INVALID_ARG
    assert call(cap=N + 1) == sbp.SBP_ERR_INVALID_ARG
    assert call(flags=1) == sbp.SBP_ERR_INVALID_ARG
    assert call(flags=512) == sbp.SBP_ERR_INVALID_ARG
    assert call(N=400, cap=300) == sbp.SBP_ERR_UNSUPPORTED          # more than 256 kept tokens per sample
    assert call(N=400, flags=sbp.SBP_FLAG_ATTN_ALL_KEYS) == sbp.SBP_ERR_UNSUPPORTED
