"""Parity of the CUDA library (through its C ABI) with the fp64 CPU oracle, element by element,
on the same seeded inputs.  Indices and the cached rows must match bit for bit; floating-point
outputs within a relative Frobenius error of 1e-5 (fp32) / 5e-3 (bf16 inputs, fp32 accumulation);
dropped rows of dX must be +0.0 exactly."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth
from gpu_harness import dev, host, run_sample_keep, run_forward_cache, run_backward

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 5e-3}


def relerr(got, want):
    return float(np.linalg.norm(got.astype(np.float64) - want) / max(np.linalg.norm(want), 1e-300))


def elem_ok(got, want, rel, rms_frac):
    """Every element on its own: |got - want| <= rel * |want| + rms_frac * rms(want).  A single wrong entry
    (a clipped tile edge, a row left out of a sum) fails here even where it would drown in the Frobenius norm."""
    rms = float(np.sqrt(np.mean(want * want)))
    return bool((np.abs(got.astype(np.float64) - want) <= rel * np.abs(want) + rms_frac * rms).all())


# dW / db leave fp32 accumulators unrounded; dX is rounded once to the storage type
ELEM = {"f32": dict(acc=(0.0, 1e-4), dx=(1e-5, 1e-4)), "bf16": dict(acc=(0.0, 1e-3), dx=(2.0 ** -8, 1e-3))}


# ------------------------------------------------------------------ sampler
@pytest.mark.parametrize("mode,B,H,W,r,seed,step,off,flags", [
    (0, 2, 16, 1, 0.5, 0, 0, 0, 0),                      # the small fp32 workload's mask
    (0, 64, 14, 14, 0.5, 0, 0, 0, 0),                    # ViT-B/16 token grid
    (0, 5, 14, 14, 0.25, 0xDEADBEEF12345678, 7, 3, 0),
    (0, 3, 14, 14, 0.75, 9, 2 ** 32 - 1, 2 ** 32 - 3, 0),
    (0, 4, 14, 14, 1.0, 1, 1, 0, 0),
    (0, 3, 56, 56, 0.5, 2, 0, 0, 0),                     # several sweeps of the block
    (0, 2, 200, 334, 0.5, 0, 0, 0, 0),                   # detection-resolution map
    (0, 3, 100, 100, 0.5, 4, 1, 0, 0),                   # one sample over a cluster of 2 blocks
    (0, 2, 128, 160, 0.25, 5, 2, 9, 0),                  # ... of 4 blocks
    (0, 1, 181, 181, 0.75, 6, 0, 0, sbp.SBP_FLAG_SHARE_MASK),   # ... of 8 blocks, ragged slices
    (0, 7, 1, 1, 0.5, 3, 0, 0, 0),
    (0, 3, 3, 3, 0.01, 3, 0, 0, 0),
    (0, 6, 9, 11, 0.5, 4, 2, 5, sbp.SBP_FLAG_SHARE_MASK),
    (1, 64, 7, 7, 0.5, 0, 0, 0, 0),                      # ragged counts (24 / 25 per sample)
    (1, 9, 7, 5, 0.25, 5, 1, 2, 0),
    (1, 9, 5, 7, 0.75, 6, 2, 0, 0),
    (1, 4, 14, 14, 1.0, 0, 0, 0, 0),
    (1, 64, 56, 56, 0.5, 0, 3, 0, 0),
    (1, 5, 7, 7, 0.5, 0, 0, 1, sbp.SBP_FLAG_SHARE_MASK),
    (1, 2, 200, 334, 0.5, 1, 0, 0, 0),
    (2, 4, 8, 196, 0.5, 0, 0, 0, 0),                     # whole frames of a video clip: 8 frames of 14x14 tokens
    (2, 3, 16, 49, 0.25, 7, 3, 11, 0),
    (2, 2, 5, 6, 0.75, 1, 9, 0, sbp.SBP_FLAG_SHARE_MASK),
    (2, 1, 1500, 3, 0.5, 2, 1, 4, 0),                    # many frames: several sweeps of the ranking loops
    (2, 5, 32, 1, 1.0, 0, 0, 0, 0),
    (3, 64, 9, 5, 0.5, 4, 2, 0, 0),                      # every second frame, ragged counts (5 or 4 of 9 frames)
    (3, 48, 10, 3, 0.25, 9, 1, 7, 0),
    (3, 600, 7, 2, 0.75, 9, 1, 0, 0),                    # more samples than threads: the offset sum loops
    (3, 5, 6, 49, 0.5, 2, 0, 3, sbp.SBP_FLAG_SHARE_MASK),
    (3, 3, 8, 196, 1.0, 0, 0, 0, 0),
])
def test_keep_indices_bit_exact(mode, B, H, W, r, seed, step, off, flags):
    want_rows, want_offs = oracle.sample_keep(mode, B, H, W, r, seed, step, off, flags)
    rows, offs, cap = run_sample_keep(mode, B, H, W, r, seed, step, off, flags)
    assert np.array_equal(host(offs), want_offs)
    n = int(want_offs[-1])
    assert np.array_equal(host(rows)[:n], want_rows)
    assert np.all(host(rows)[n:] == -7)                   # nothing written past M_keep


def test_equal_philox_words_are_broken_by_position():
    # with 2^17 positions some 32-bit words collide near any threshold with small probability;
    # the large map at several seeds exercises the equal-word path of the selection
    for seed in range(3):
        want_rows, _ = oracle.sample_keep(0, 1, 512, 256, 0.5, seed)
        rows, _, _ = run_sample_keep(0, 1, 512, 256, 0.5, seed)
        assert np.array_equal(host(rows), want_rows)


# ------------------------------------------------------------- forward cache
@pytest.mark.parametrize("dtype,M,C,M_keep", [("f32", 32, 32, 16), ("bf16", 1000, 768, 517), ("bf16", 333, 8, 100),
                                              ("f32", 64, 4, 64), ("bf16", 5000, 3072, 1)])
def test_forward_cache_bitwise(dtype, M, C, M_keep):
    X = synth.gaussian_tensor((M, C), dtype, 77, 0, 1.0)
    keep = np.sort(np.random.default_rng(M).choice(M, M_keep, replace=False)).astype(np.int32)
    got = run_forward_cache(dtype, dev(X, dtype), torch.from_numpy(keep).cuda(), M_keep)
    assert host(got).tobytes() == oracle.forward_cache(X, keep).tobytes()


def test_forward_cache_device_count_and_zeroed_padding():
    M, C, cap, M_keep = 200, 64, 120, 97
    X = synth.gaussian_tensor((M, C), "bf16", 78, 0, 1.0)
    keep = np.sort(np.random.default_rng(1).choice(M, cap, replace=False)).astype(np.int32)
    cnt = torch.tensor([M_keep], dtype=torch.int32, device="cuda")
    got = host(run_forward_cache("bf16", dev(X, "bf16"), torch.from_numpy(keep).cuda(), cap, cnt))
    assert got[:M_keep].tobytes() == oracle.forward_cache(X, keep[:M_keep]).tobytes()
    assert np.all(got[M_keep:] == 0)


# ------------------------------------------------------------ linear backward
def _case(dtype, B, H, W, C_in, C_out, r, mode=0, seed=0, data_seed=5, sig=(1.0, 0.02, 1e-2)):
    M = B * H * W
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, data_seed, *sig)
    keep, offs = oracle.sample_keep(mode, B, H, W, r, seed)
    return M, X, Wt, dY, keep


def _check_backward(dtype, M, X, Wt, dY, keep, flags=0, cap=None, count_on_device=False):
    M_keep = len(keep)
    cap = M_keep if cap is None else cap
    rows = np.zeros(max(cap, 1), dtype=np.int32)
    rows[:M_keep] = keep
    rows_d = torch.from_numpy(rows).cuda()
    cnt = torch.tensor([M_keep], dtype=torch.int32, device="cuda") if count_on_device else None
    Xk_d = run_forward_cache(dtype, dev(X, dtype), rows_d, cap, cnt)
    got = run_backward(dtype, Xk_d, dev(dY, dtype), dev(Wt, dtype), rows_d, cap, cnt, flags=flags)
    assert got["status"] == 0
    Xk = oracle.forward_cache(X, keep)
    assert host(Xk_d)[:M_keep].tobytes() == Xk.tobytes()
    want = oracle.linear_backward(synth.to_f64(Xk, dtype), synth.to_f64(dY, dtype), synth.to_f64(Wt, dtype), keep)
    tol = TOL[dtype]
    assert relerr(host(got["dW"]), want["dW"]) <= tol
    assert relerr(host(got["db"]), want["db"]) <= tol
    assert elem_ok(host(got["dW"]), want["dW"], *ELEM[dtype]["acc"])
    assert elem_ok(host(got["db"]), want["db"], *ELEM[dtype]["acc"])
    dX_bits = host(got["dX"])
    dX = synth.to_f64(dX_bits, dtype)
    assert relerr(dX, want["dX"]) <= tol
    if M_keep:
        assert elem_ok(dX[keep], want["dX"][keep], *ELEM[dtype]["dx"])
    drop = np.setdiff1d(np.arange(M), keep)
    assert not np.any(dX_bits[drop].view(np.uint16 if dtype == "bf16" else np.uint32))   # +0.0 bit pattern
    return got, want


def test_small_fp32_layer():
    # B=2, N=16, 32 -> 64, r=0.5, seed 0
    w = synth.workload("single_fp32")
    M, X, Wt, dY, keep = _case("f32", w["B"], w["H"], w["W"], w["C_in"], w["C_out"], w["keep_ratio"],
                               data_seed=w["data_seed"], sig=(w["sigma_x"], w["sigma_w"], w["sigma_dy"]))
    assert len(keep) == 16
    _check_backward("f32", M, X, Wt, dY, keep)


@pytest.mark.parametrize("B,H,W,C_in,C_out,r", [
    (3, 14, 14, 96, 200, 0.5),        # ragged tiles everywhere
    (2, 9, 7, 4, 4, 0.25),
    (1, 300, 1, 260, 68, 0.75),
    (4, 8, 8, 64, 64, 1.0),
])
def test_fp32_shapes(B, H, W, C_in, C_out, r):
    M, X, Wt, dY, keep = _case("f32", B, H, W, C_in, C_out, r, sig=(1.0, 0.1, 1.0))
    _check_backward("f32", M, X, Wt, dY, keep)


@pytest.mark.parametrize("B,H,W,C_in,C_out,r,mode", [
    (8, 14, 14, 768, 3072, 0.5, 0),      # ViT-B fc1 shape at a batch the oracle finishes quickly
    (8, 14, 14, 3072, 768, 0.5, 0),      # fc2
    (5, 14, 14, 768, 768, 0.25, 0),      # proj, ragged last row tile (245 kept rows)
    (3, 14, 14, 768, 2304, 0.75, 0),     # qkv
    (2, 14, 14, 256, 128, 1.0, 0),       # keep everything
    (2, 56, 56, 128, 512, 0.5, 0),       # ConvNeXt stage-1 pointwise, narrow C_in (BN = 128 path)
    (2, 56, 56, 512, 128, 0.5, 1),       # grid mask
    (64, 7, 7, 1024, 256, 0.5, 1),       # grid mask with ragged per-sample counts
    (1, 40, 10, 136, 200, 0.5, 0),       # channel counts that are multiples of 8 only
    (1, 100, 1, 128, 128, 0.65, 0),      # a single partial row tile
])
def test_bf16_tensor_core_shapes(B, H, W, C_in, C_out, r, mode):
    M, X, Wt, dY, keep = _case("bf16", B, H, W, C_in, C_out, r, mode=mode)
    _check_backward("bf16", M, X, Wt, dY, keep)


@pytest.mark.parametrize("B,H,W,C_in,C_out,r", [(2, 14, 14, 64, 32, 0.5), (1, 20, 1, 768, 256, 0.5), (3, 7, 7, 8, 8, 0.5)])
def test_bf16_small_shapes_use_plain_fma(B, H, W, C_in, C_out, r):
    M, X, Wt, dY, keep = _case("bf16", B, H, W, C_in, C_out, r)
    _check_backward("bf16", M, X, Wt, dY, keep)


def test_bf16_plain_fma_flag_agrees_with_tensor_cores():
    M, X, Wt, dY, keep = _case("bf16", 4, 14, 14, 256, 384, 0.5)
    a, _ = _check_backward("bf16", M, X, Wt, dY, keep)
    b, _ = _check_backward("bf16", M, X, Wt, dY, keep, flags=sbp.SBP_FLAG_PLAIN_FMA)
    assert relerr(host(a["dW"]), host(b["dW"]).astype(np.float64)) < 1e-4
    assert np.array_equal(host(a["dX"]) != 0, host(b["dX"]) != 0)


@pytest.mark.parametrize("dtype,C_in,C_out", [("f32", 32, 64), ("bf16", 256, 256)])
def test_device_side_count_smaller_than_capacity(dtype, C_in, C_out):
    # grid masks on odd maps give a data-dependent M_keep below the buffer capacity
    B, H, W = 16, 7, 7
    M, X, Wt, dY, keep = _case(dtype, B, H, W, C_in, C_out, 0.5, mode=1, sig=(1.0, 0.1, 1.0))
    cap = B * oracle.keep_count(1, H, W, 0.5)
    assert len(keep) < cap
    _check_backward(dtype, M, X, Wt, dY, keep, cap=cap, count_on_device=True)


@pytest.mark.parametrize("dtype,C_in,C_out", [("f32", 32, 64), ("bf16", 256, 256)])
def test_nothing_kept_gives_all_zero_gradients(dtype, C_in, C_out):
    M, cap = 200, 100
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, 3)
    rows_d = torch.zeros(cap, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    Xk_d = run_forward_cache(dtype, dev(X, dtype), rows_d, cap, cnt)
    got = run_backward(dtype, Xk_d, dev(dY, dtype), dev(Wt, dtype), rows_d, cap, cnt)
    assert got["status"] == 0
    for k in ("dW", "db", "dX"):
        assert not np.any(host(got[k]).view(np.uint8)), k


@pytest.mark.parametrize("dtype,C_in,C_out", [("f32", 32, 64), ("bf16", 256, 384), ("bf16", 128, 264)])   # last: bias from the dW tiles
def test_accumulate_flag_adds_into_dw_and_db(dtype, C_in, C_out):
    M, X, Wt, dY, keep = _case(dtype, 4, 14, 14, C_in, C_out, 0.5, sig=(1.0, 0.1, 1.0))
    rows_d = torch.from_numpy(keep).cuda()
    Xk_d = run_forward_cache(dtype, dev(X, dtype), rows_d, len(keep))
    init = {"dW": torch.full((C_in, C_out), 2.0, device="cuda"), "db": torch.full((C_out,), -3.0, device="cuda")}
    got = run_backward(dtype, Xk_d, dev(dY, dtype), dev(Wt, dtype), rows_d, len(keep), flags=sbp.SBP_FLAG_ACCUMULATE,
                       init=init, want=("dW", "db"))
    want = oracle.linear_backward(synth.to_f64(oracle.forward_cache(X, keep), dtype), synth.to_f64(dY, dtype),
                                  synth.to_f64(Wt, dtype), keep, want=("dW", "db"))
    assert relerr(host(got["dW"]), want["dW"] + 2.0) <= TOL[dtype]
    assert relerr(host(got["db"]), want["db"] - 3.0) <= TOL[dtype]


def test_outputs_can_be_skipped():
    M, X, Wt, dY, keep = _case("bf16", 2, 14, 14, 256, 256, 0.5)
    rows_d = torch.from_numpy(keep).cuda()
    Xk_d = run_forward_cache("bf16", dev(X, "bf16"), rows_d, len(keep))
    only_dx = run_backward("bf16", None, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, len(keep), want=("dX",))
    only_dw = run_backward("bf16", Xk_d, dev(dY, "bf16"), None, rows_d, len(keep), want=("dW",))
    full = run_backward("bf16", Xk_d, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, len(keep))
    assert torch.equal(only_dx["dX"], full["dX"]) and torch.equal(only_dw["dW"], full["dW"])


def test_results_are_deterministic():
    M, X, Wt, dY, keep = _case("bf16", 6, 14, 14, 768, 768, 0.5)
    rows_d = torch.from_numpy(keep).cuda()
    Xk_d = run_forward_cache("bf16", dev(X, "bf16"), rows_d, len(keep))
    a = run_backward("bf16", Xk_d, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, len(keep))
    b = run_backward("bf16", Xk_d, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, len(keep))
    for k in ("dW", "db", "dX"):
        assert torch.equal(a[k], b[k])


@pytest.mark.parametrize("dtype,C_in,C_out", [("f32", 32, 64), ("bf16", 256, 256)])
def test_validate_flag_reports_bad_indices_and_leaves_outputs_alone(dtype, C_in, C_out):
    M = 300
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, 4)
    for bad in ([0, 5, 5, 9] + list(range(10, 106)), [0, 5, 300] + list(range(301, 398)), [3, 2] + list(range(4, 102))):
        keep = np.array(bad, dtype=np.int32)
        rows_d = torch.from_numpy(keep).cuda()
        Xk_d = torch.zeros((len(keep), C_in), dtype=dev(X, dtype).dtype, device="cuda")
        got = run_backward(dtype, Xk_d, dev(dY, dtype), dev(Wt, dtype), rows_d, len(keep), flags=sbp.SBP_FLAG_VALIDATE)
        assert got["status"] == sbp.SBP_ERR_BAD_INDICES
        assert torch.isnan(got["dW"]).all() and torch.isnan(got["db"]).all() and torch.isnan(got["dX"].float()).all()
    good = np.arange(0, 200, 2, dtype=np.int32)
    rows_d = torch.from_numpy(good).cuda()
    Xk_d = run_forward_cache(dtype, dev(X, dtype), rows_d, len(good))
    got = run_backward(dtype, Xk_d, dev(dY, dtype), dev(Wt, dtype), rows_d, len(good), flags=sbp.SBP_FLAG_VALIDATE)
    assert got["status"] == 0 and not torch.isnan(got["dW"]).any()


def test_full_path_sampler_to_gradients_on_device():
    # sample -> cache -> backward entirely from device-resident indices, grid mask, device count
    B, H, W, C_in, C_out = 32, 7, 7, 512, 256
    M = B * H * W
    X, Wt, dY = synth.layer_inputs("bf16", M, C_in, C_out, 11)
    rows_d, offs_d, cap = run_sample_keep(1, B, H, W, 0.5, seed=3, step=1)
    cnt = offs_d[B:B + 1]
    Xk_d = run_forward_cache("bf16", dev(X, "bf16"), rows_d, B * cap, cnt)
    got = run_backward("bf16", Xk_d, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, B * cap, cnt)
    keep, _ = oracle.sample_keep(1, B, H, W, 0.5, seed=3, step=1)
    want = oracle.linear_backward(synth.to_f64(oracle.forward_cache(X, keep), "bf16"), synth.to_f64(dY, "bf16"),
                                  synth.to_f64(Wt, "bf16"), keep)
    assert got["status"] == 0
    assert relerr(host(got["dW"]), want["dW"]) <= 5e-3
    assert relerr(host(got["db"]), want["db"]) <= 5e-3
    assert relerr(synth.to_f64(host(got["dX"]), "bf16"), want["dX"]) <= 5e-3


def test_bounded_wait_gives_up_reports_and_leaves_the_stream_usable():
    # a device-side wait that nothing will ever satisfy: it must expire after its limit, set the status word,
    # let the kernel return, and the next call on the same stream must work as usual
    import time
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    completed = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    sbp.sbp_selftest_bounded_wait(200.0, status, completed)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert int(status.item()) == sbp.SBP_ERR_TIMEOUT and int(completed.item()) == 0
    assert 0.19 <= waited < 1.5
    rows, offs, _ = run_sample_keep(0, 2, 14, 14, 0.5)
    want_rows, want_offs = oracle.sample_keep(0, 2, 14, 14, 0.5)
    assert np.array_equal(host(offs), want_offs) and np.array_equal(host(rows)[:len(want_rows)], want_rows)
    assert sbp.sbp_selftest_bounded_wait(0.0, status, completed, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_selftest_bounded_wait(5000.0, status, completed, check=False) == sbp.SBP_ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs two GPUs in one process")
def test_one_process_drives_two_devices():
    # the opt-in for large dynamic shared memory belongs to the (kernel, device) pair: a tensor-core backward on
    # device 0 and then on device 1 from the same process must both launch (no peer memory, no collective)
    M, X, Wt, dY, keep = _case("bf16", 4, 14, 14, 256, 384, 0.5)
    want = oracle.linear_backward(synth.to_f64(oracle.forward_cache(X, keep), "bf16"), synth.to_f64(dY, "bf16"),
                                  synth.to_f64(Wt, "bf16"), keep)
    for d in (0, 1):
        with torch.cuda.device(d):
            rows_d = torch.from_numpy(keep).cuda()
            Xk_d = run_forward_cache("bf16", dev(X, "bf16"), rows_d, len(keep))
            got = run_backward("bf16", Xk_d, dev(dY, "bf16"), dev(Wt, "bf16"), rows_d, len(keep))
            assert got["status"] == 0
            assert relerr(host(got["dW"]), want["dW"]) <= 5e-3 and relerr(synth.to_f64(host(got["dX"]), "bf16"), want["dX"]) <= 5e-3
