"""The workspace-free bias gradient, for callers that cannot allocate device memory.

Some users of the library have no allocator to ask for the scratch buffer `sbp_linear_backward`
wants: an operator plugin that only ever sees its tensors, code running under a memory pool that a
host framework owns and has frozen, a service with a fixed device-memory budget.
`sbp_bias_grad_static` keeps its scratch in a fixed array inside the library instead.  This file
checks it against the ordinary entry point and against the fp64 oracle on calls in a row (each with
other sizes and data, so stale scratch contents from the call before would show), with a row count
read from device memory that is below the capacity, on two calls enqueued back to back with a single
synchronisation after both, and that sizes beyond the built-in scratch are refused.  It is collected last so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth

pytestmark = pytest.mark.gpu


def _oracle_db(dtype, dY, keep, start):
    want = oracle.linear_backward(np.zeros((len(keep), 1)), synth.to_f64(dY, dtype), np.zeros((1, dY.shape[1])), keep,
                                  want=("db",))["db"]
    return want + start


def _db_both_ways(dtype, M, C_out, keep, data_seed, accumulate=False):
    code = sbp.SBP_BF16 if dtype == "bf16" else sbp.SBP_F32
    dY = synth.gaussian_tensor((M, C_out), dtype, data_seed, 2, 1.0)
    dY_d = torch.from_numpy(dY).cuda()
    if dtype == "bf16":
        dY_d = dY_d.view(torch.bfloat16)
    rows = torch.from_numpy(keep).cuda()
    M_keep = len(keep)
    flags = sbp.SBP_FLAG_ACCUMULATE if accumulate else 0
    start = 1.5 if accumulate else float("nan")
    # existing entry point: caller-allocated workspace
    nbytes = sbp.sbp_linear_backward_workspace_bytes(code, M, M_keep, 8, C_out)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    want = torch.full((C_out,), start, dtype=torch.float32, device="cuda")
    sbp.sbp_linear_backward(code, None, dY_d, None, rows, None, M, M_keep, 8, C_out, None, want, None, flags, ws, nbytes)
    # new entry point: no workspace, nothing allocated by the call
    got = torch.full((C_out,), start, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    sbp.sbp_bias_grad_static(code, dY_d, rows, None, M, M_keep, C_out, got, flags)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    ref = _oracle_db(dtype, dY, keep, start if accumulate else 0.0)
    return got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64), ref


def test_static_scratch_bias_gradient_matches_the_workspace_version_twice_in_a_row():
    rng = np.random.default_rng(0)
    calls = [("bf16", 3000, 3072, 0.5, False), ("f32", 700, 260, 0.3, False), ("bf16", 1200, 4096, 0.9, True)]
    for i, (dtype, M, C_out, frac, acc) in enumerate(calls):
        keep = np.sort(rng.choice(M, int(M * frac), replace=False)).astype(np.int32)
        got, want, ref = _db_both_ways(dtype, M, C_out, keep, 40 + i, accumulate=acc)
        tol = 5e-3 if dtype == "bf16" else 1e-5
        assert np.isfinite(got).all()
        assert np.linalg.norm(got - want) <= tol * np.linalg.norm(want), (i, dtype)
        assert np.linalg.norm(got - ref) <= tol * np.linalg.norm(ref), (i, dtype)
        # fp32 sums of at most a few thousand terms: every single column is close, not only the norm
        assert np.abs(got - ref).max() <= 1e-4 * np.sqrt(np.mean(ref ** 2)) + 1e-6, (i, dtype)


def test_device_side_count_and_two_calls_without_a_sync_between_them():
    """The kept-row count comes from device memory and is smaller than the capacity; two calls of different
    sizes follow each other on one stream with one synchronisation at the end (the shared scratch is reused
    by the second call as soon as the first has read it: stream order is all that separates them)."""
    rng = np.random.default_rng(5)
    specs = [("bf16", 2500, 1024, 900, 1300), ("f32", 1800, 520, 333, 333)]
    outs, refs = [], []
    keep_alive = []
    for i, (dtype, M, C_out, n_valid, cap) in enumerate(specs):
        code = sbp.SBP_BF16 if dtype == "bf16" else sbp.SBP_F32
        dY = synth.gaussian_tensor((M, C_out), dtype, 60 + i, 2, 1.0)
        dY_d = torch.from_numpy(dY).cuda()
        if dtype == "bf16":
            dY_d = dY_d.view(torch.bfloat16)
        keep = np.sort(rng.choice(M, cap, replace=False)).astype(np.int32)
        rows = torch.from_numpy(keep).cuda()
        cnt = torch.tensor([n_valid], dtype=torch.int32, device="cuda")
        db = torch.full((C_out,), float("nan"), dtype=torch.float32, device="cuda")
        keep_alive.append((dY_d, rows, cnt))
        outs.append((dtype, code, dY_d, rows, cnt, M, cap, C_out, db))
        refs.append(_oracle_db(dtype, dY, keep[:n_valid], 0.0))
    torch.cuda.synchronize()
    for dtype, code, dY_d, rows, cnt, M, cap, C_out, db in outs:
        sbp.sbp_bias_grad_static(code, dY_d, rows, cnt, M, cap, C_out, db, 0)
    torch.cuda.synchronize()
    for (dtype, *_rest, db), ref in zip(outs, refs):
        got = db.cpu().numpy().astype(np.float64)
        tol = 5e-3 if dtype == "bf16" else 1e-5
        assert np.isfinite(got).all()
        assert np.linalg.norm(got - ref) <= tol * np.linalg.norm(ref), dtype


def test_sizes_beyond_the_built_in_scratch_are_refused():
    dY = torch.zeros((16, 4104), dtype=torch.bfloat16, device="cuda")
    rows = torch.arange(8, dtype=torch.int32, device="cuda")
    db = torch.zeros(4104, dtype=torch.float32, device="cuda")
    s = sbp.sbp_bias_grad_static(sbp.SBP_BF16, dY, rows, None, 16, 8, 4104, db, 0, check=False)
    assert s == sbp.SBP_ERR_WORKSPACE
    assert "workspace" in sbp.status_string(s)
    assert sbp.sbp_bias_grad_static(sbp.SBP_BF16, dY, rows, None, 16, 8, 4100, db, 0, check=False) == sbp.SBP_ERR_UNSUPPORTED
    assert sbp.sbp_bias_grad_static(sbp.SBP_BF16, None, rows, None, 16, 8, 4096, db, 0, check=False) == sbp.SBP_ERR_INVALID_ARG
