"""Helpers for the GPU parity tests: move seeded numpy inputs to the device, run the CUDA
library through its C-ABI binding, bring results back as numpy.  No arithmetic of the method
lives here."""
import numpy as np
import torch

import paper_2210_00129_b200 as sbp


def dev(a: np.ndarray, dtype: str):
    """numpy (float32, or uint16 bf16 bit patterns) -> CUDA tensor of the path's storage type."""
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if dtype == "bf16":
        assert a.dtype == np.uint16
        return t.view(torch.bfloat16)
    return t


def host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def dt_code(dtype: str) -> int:
    return sbp.SBP_BF16 if dtype == "bf16" else sbp.SBP_F32


def run_sample_keep(mode, B, H, W, r, seed=0, step=0, offset=0, flags=0):
    cap = sbp.sbp_keep_count(mode, H, W, r)
    rows = torch.full((max(B * cap, 1),), -7, dtype=torch.int32, device="cuda")
    offs = torch.full((B + 1,), -7, dtype=torch.int32, device="cuda")
    sbp.sbp_sample_keep(mode, B, H, W, r, seed, step, offset, flags, rows, offs)
    torch.cuda.synchronize()
    return rows, offs, cap


def run_forward_cache(dtype, X_dev, keep_rows_dev, M_keep_cap, M_keep_dev=None):
    M, C = X_dev.shape
    out = torch.full((max(M_keep_cap, 1), C), 7.0, dtype=X_dev.dtype, device="cuda")
    sbp.sbp_forward_cache(dt_code(dtype), X_dev, M, C, keep_rows_dev, M_keep_dev, M_keep_cap, out)
    torch.cuda.synchronize()
    return out


def run_backward(dtype, X_keep_dev, dY_dev, W_dev, keep_rows_dev, M_keep_cap, M_keep_dev=None, flags=0,
                 want=("dW", "db", "dX"), init=None, with_status=True, M=None, dX_rows=None):
    """M: rows of the layer (default: rows of dY, which a packed dY does not have); dX_rows: rows of the dX buffer."""
    C_out = dY_dev.shape[1]
    M = dY_dev.shape[0] if M is None else M
    C_in = W_dev.shape[0] if W_dev is not None else X_keep_dev.shape[1]
    code = dt_code(dtype)
    nbytes = sbp.sbp_linear_backward_workspace_bytes(code, M, M_keep_cap, C_in, C_out)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda") if with_status else None
    fill = float("nan")
    dW = torch.full((C_in, C_out), fill, dtype=torch.float32, device="cuda") if "dW" in want else None
    db = torch.full((C_out,), fill, dtype=torch.float32, device="cuda") if "db" in want else None
    dX = torch.full((M if dX_rows is None else max(dX_rows, 1), C_in), fill, dtype=dY_dev.dtype,
                    device="cuda") if "dX" in want else None
    if init is not None:
        if dW is not None: dW.copy_(init["dW"])
        if db is not None: db.copy_(init["db"])
    sbp.sbp_linear_backward(code, X_keep_dev, dY_dev, W_dev, keep_rows_dev, M_keep_dev, M, M_keep_cap, C_in, C_out,
                            dW, db, dX, flags, ws, nbytes, status)
    torch.cuda.synchronize()
    out = {}
    if dW is not None: out["dW"] = dW
    if db is not None: out["db"] = db
    if dX is not None: out["dX"] = dX
    out["status"] = int(status.item()) if status is not None else 0
    return out
