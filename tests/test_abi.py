"""Host-side checks of the C-ABI library that need no GPU: it builds, loads, exports every
symbol the header declares, its pure host functions agree with the oracle's rule, and argument
errors are returned before anything is launched."""
import ctypes
import os
import re

import pytest

import oracle
import paper_2210_00129_b200 as sbp
from paper_2210_00129_b200 import build as sbp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sbp_build.build()
    return sbp.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sbp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sbp_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert set(names) == set(sbp.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n
        assert callable(getattr(sbp, n, None)) or n == "sbp_status_string"


def test_status_strings(lib):
    seen = {sbp.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert sbp.status_string(99) == "unknown status"


@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_keep_count_matches_the_rule(lib, mode):
    ratios = (0.25, 0.5, 0.75, 1.0) if mode in (1, 3) else (0.01, 0.25, 0.3, 0.5, 0.75, 0.999, 1.0)
    for H, W in [(1, 1), (14, 14), (7, 7), (3, 5), (56, 56), (200, 334), (16, 1)]:
        for r in ratios:
            assert sbp.sbp_keep_count(mode, H, W, r) == oracle.keep_count(mode, H, W, r)
    assert sbp.sbp_keep_count(mode, 0, 4, 0.5) == -1
    assert sbp.sbp_keep_count(mode, 4, 4, 0.0) == -1
    assert sbp.sbp_keep_count(mode, 4, 4, 1.5) == -1
    assert sbp.sbp_keep_count(mode, 4, 4, float("nan")) == -1
    assert sbp.sbp_keep_count(1, 4, 4, 0.3) == -1


def test_host_detected_errors_return_before_any_launch(lib):
    fake = 0x1000  # never dereferenced: every call below must fail its host checks first
    assert sbp.sbp_sample_keep(0, 2, 4, 4, 0.5, 0, 0, 0, 0, None, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(0, 0, 4, 4, 0.5, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(0, 2, 4, 4, 1.5, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(0, 2, 4, 4, 0.5, 0, 2 ** 32, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(0, 2, 4, 4, 0.5, 0, 0, 2 ** 32 - 1, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(0, 2 ** 20, 2 ** 6, 2 ** 6, 0.5, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(1, 2, 4, 4, 0.6, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_UNSUPPORTED
    assert sbp.sbp_sample_keep(2, 2, 4096, 4, 0.5, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_UNSUPPORTED   # too many frames
    assert sbp.sbp_sample_keep(4, 2, 4, 4, 0.5, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_sample_keep(3, 2, 4, 4, 0.6, 0, 0, 0, 0, fake, fake, stream=0, check=False) == sbp.SBP_ERR_UNSUPPORTED
    # forward cache: misaligned pointer, row bytes not a multiple of 16
    assert sbp.sbp_forward_cache(1, fake + 2, 8, 8, fake, None, 4, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    assert sbp.sbp_forward_cache(1, fake, 8, 4, fake, None, 4, fake, stream=0, check=False) == sbp.SBP_ERR_UNSUPPORTED
    assert sbp.sbp_forward_cache(0, fake, 8, 4, fake, None, 9, fake, stream=0, check=False) == sbp.SBP_ERR_INVALID_ARG
    # backward: channel multiples, workspace, null inputs
    args = dict(M=32, M_keep_cap=16, C_in=32, C_out=64)
    need = sbp.sbp_linear_backward_workspace_bytes(0, 32, 16, 32, 64)
    assert need >= 256
    call = lambda **kw: sbp.sbp_linear_backward(
        kw.get("dt", 0), fake, kw.get("dY", fake), fake, fake, None, args["M"], args["M_keep_cap"],
        kw.get("C_in", 32), args["C_out"], fake, fake, fake, kw.get("flags", 0), kw.get("ws", fake - 0x1000 + 0x1000),
        kw.get("ws_bytes", need), None, stream=0, check=False)
    assert call(dY=None) == sbp.SBP_ERR_INVALID_ARG
    assert call(C_in=30) == sbp.SBP_ERR_UNSUPPORTED
    assert call(dt=1, C_in=36) == sbp.SBP_ERR_UNSUPPORTED
    assert call(ws_bytes=need - 1) == sbp.SBP_ERR_WORKSPACE
    assert call(ws=None) == sbp.SBP_ERR_WORKSPACE
    assert call(ws=fake + 16) == sbp.SBP_ERR_WORKSPACE
    assert call(flags=sbp.SBP_FLAG_VALIDATE) == sbp.SBP_ERR_INVALID_ARG     # validate needs a status word


def test_workspace_query_grows_with_the_problem(lib):
    small = sbp.sbp_linear_backward_workspace_bytes(1, 12544, 6272, 768, 3072)
    assert small % 256 == 0 and small >= 64 * 3072 * 4
    assert sbp.sbp_linear_backward_workspace_bytes(1, 0, 0, 0, 0) == 256


def test_split_plans_are_searched_once_per_shape(lib):
    # more layer shapes than any small cache would hold (ConvNeXt-B alone has eight point-wise shapes):
    # the second round of queries must not search again
    shapes = [(64 * hw * hw, d_in, d_out) for d, hw in ((128, 56), (256, 28), (512, 14), (1024, 7), (192, 28))
              for d_in, d_out in ((d, 4 * d), (4 * d, d))]
    assert len(shapes) == 10
    for M, ci, co in shapes:
        sbp.sbp_linear_backward_workspace_bytes(1, M, M // 2, ci, co)
    seen = sbp.sbp_plan_search_count()
    assert seen >= len(shapes)
    for _ in range(3):
        for M, ci, co in shapes:
            sbp.sbp_linear_backward_workspace_bytes(1, M, M // 2, ci, co)
            sbp.sbp_linear_backward_kernel_count(1, M, M // 2, ci, co)
    assert sbp.sbp_plan_search_count() == seen


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(sbp, "_lib", None)
    monkeypatch.setattr(sbp, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="missing"):
        sbp.sbp_keep_count(0, 4, 4, 0.5)
