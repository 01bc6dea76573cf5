"""`sbp_step_host` - the whole step from host tensors, the call the benchmark's end-to-end figure goes
through - against the fp64 oracle: indices and offsets bit-exact, gradients within the path's tolerance and
element by element, dropped rows of dX all-zero bits, status word clear."""
import numpy as np
import pytest
import torch

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import synth

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 5e-3}


def _run_step(dtype, mode, B, H, W, C_in, C_out, r, seed, step, offset, flags=0, sig=(1.0, 0.02, 1e-2), data_seed=21):
    code = sbp.SBP_BF16 if dtype == "bf16" else sbp.SBP_F32
    M = B * H * W
    X, Wt, dY = synth.layer_inputs(dtype, M, C_in, C_out, data_seed, *sig)
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
    Xp, Wp, dYp = pin(X), pin(Wt), pin(dY)
    cap = B * sbp.sbp_keep_count(mode, H, W, r)
    out_dt = torch.int16 if dtype == "bf16" else torch.float32
    dW = torch.full((C_in, C_out), float("nan"), dtype=torch.float32).pin_memory()
    db = torch.full((C_out,), float("nan"), dtype=torch.float32).pin_memory()
    dX = torch.full((M, C_in), -1, dtype=out_dt).pin_memory()
    rows = torch.full((cap,), -7, dtype=torch.int32).pin_memory()
    offs = torch.full((B + 1,), -7, dtype=torch.int32).pin_memory()
    st = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    nbytes = sbp.sbp_step_host_arena_bytes(code, mode, B, H, W, C_in, C_out, r)
    arena = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    sbp.sbp_step_host(code, mode, B, H, W, C_in, C_out, r, seed, step, offset, flags, Xp, dYp, Wp, dW, db, dX, rows, offs,
                      st, arena, nbytes)
    torch.cuda.synchronize()
    return (X, Wt, dY), dict(dW=dW.numpy(), db=db.numpy(), dX=dX.numpy(), rows=rows.numpy(), offs=offs.numpy(),
                             status=int(st.item()))


@pytest.mark.parametrize("dtype,mode,B,H,W,C_in,C_out,r,seed,step,offset,sig", [
    ("f32", 0, 2, 16, 1, 32, 64, 0.5, 0, 0, 0, (1.0, 32 ** -0.5, 1.0)),        # the small fp32 layer
    ("bf16", 0, 8, 14, 14, 768, 3072, 0.5, 0, 4, 16, (1.0, 0.02, 1e-2)),       # ViT-B fc1 shape, a shard starting at sample 16
    ("bf16", 1, 16, 7, 7, 1024, 256, 0.5, 3, 1, 0, (1.0, 0.02, 1e-2)),         # grid mask, ragged counts: device-side M_keep
    ("bf16", 0, 2, 56, 56, 128, 512, 0.25, 9, 2, 5, (1.0, 0.02, 1e-2)),        # narrow layer
])
def test_step_from_host_tensors_matches_the_oracle(dtype, mode, B, H, W, C_in, C_out, r, seed, step, offset, sig):
    (X, Wt, dY), got = _run_step(dtype, mode, B, H, W, C_in, C_out, r, seed, step, offset, flags=sbp.SBP_FLAG_VALIDATE,
                                 sig=sig)
    assert got["status"] == 0
    keep, offs = oracle.sample_keep(mode, B, H, W, r, seed, step, offset)
    n = len(keep)
    assert np.array_equal(got["offs"], offs)
    assert np.array_equal(got["rows"][:n], keep)          # entries past keep_offsets[B] are unspecified
    want = oracle.linear_backward(synth.to_f64(oracle.forward_cache(X, keep), dtype), synth.to_f64(dY, dtype),
                                  synth.to_f64(Wt, dtype), keep)
    rel = lambda g, w: float(np.linalg.norm(g.astype(np.float64) - w) / np.linalg.norm(w))
    rms = lambda a: float(np.sqrt(np.mean(a * a)))
    acc_frac = 1e-3 if dtype == "bf16" else 1e-4
    for k in ("dW", "db"):
        assert rel(got[k], want[k]) <= TOL[dtype], k
        assert np.abs(got[k] - want[k]).max() <= acc_frac * rms(want[k]), k
    dX_bits = got["dX"].view(np.uint16) if dtype == "bf16" else got["dX"]
    dXf = synth.to_f64(dX_bits, dtype)
    assert rel(dXf, want["dX"]) <= TOL[dtype]
    dropped = np.ones(B * H * W, dtype=bool)
    dropped[keep] = False
    assert not dX_bits[dropped].view(np.uint16 if dtype == "bf16" else np.uint32).any()


def test_step_host_argument_errors():
    code = sbp.SBP_BF16
    fake = 0x1000
    call = lambda **kw: sbp.sbp_step_host(code, kw.get("mode", 0), 2, 4, 4, 128, 128, kw.get("r", 0.5), 0, 0, 0, kw.get("flags", 0),
                                          kw.get("X", fake), fake, fake, fake, fake, fake, None, None, None, kw.get("arena", None),
                                          kw.get("bytes", 0), stream=0, check=False)
    assert call(X=None) == sbp.SBP_ERR_INVALID_ARG
    assert call(flags=sbp.SBP_FLAG_ACCUMULATE) == sbp.SBP_ERR_UNSUPPORTED
    assert call(mode=1, r=0.6) == sbp.SBP_ERR_UNSUPPORTED
    assert call() == sbp.SBP_ERR_WORKSPACE                    # no arena
