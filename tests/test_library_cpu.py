"""CPU-side checks of the CUDA library: it loads without a GPU, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import re
from pathlib import Path

import pytest

from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import build as libbuild

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.lib()


def test_every_declared_symbol_is_exported(lib):
    header = (ROOT / "include" / "fp8mlp.h").read_text()
    declared = set(re.findall(r"\b(fp8mlp_[a-z0-9_]+)\s*\(", header))
    declared -= {"fp8mlp_ctx"}
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/fp8mlp.h but not exported"
    assert declared == set(B.EXPORTS)


def test_strerror_and_launch_count(lib):
    assert lib.fp8mlp_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert lib.fp8mlp_strerror(code) not in (b"", b"unknown error code")
    assert lib.fp8mlp_launch_count() >= 0


def test_argument_errors_are_caught_before_any_launch(lib):
    n0 = lib.fp8mlp_launch_count()
    h = C.c_void_p()
    assert lib.fp8mlp_create(None, 16, 16, 16, 0) == B.ERR_ARG
    assert lib.fp8mlp_create(C.byref(h), 16, 24, 16, 0) == B.ERR_SHAPE      # d not a multiple of 16
    assert lib.fp8mlp_create(C.byref(h), 16, 16, 40, 0) == B.ERR_SHAPE      # f not a multiple of 16
    assert lib.fp8mlp_create(C.byref(h), -1, 16, 16, 0) == B.ERR_SHAPE
    assert lib.fp8mlp_create(C.byref(h), 16, 16, 16, 64) == B.ERR_ARG       # unknown flag
    assert h.value is None
    assert lib.fp8mlp_destroy(None) == B.OK
    # quantize: null pointers, bad enums, bad shapes, misalignment
    q = lib.fp8mlp_quantize
    assert q(None, B.BF16, 1, 16, B.E4M3, B.SCALE_GIVEN, 256, None, None, 256, 16, None) == B.ERR_ARG
    assert q(256, 7, 1, 16, B.E4M3, B.SCALE_GIVEN, 256, None, None, 256, 16, None) == B.ERR_ARG
    assert q(256, B.BF16, 1, 16, 5, B.SCALE_GIVEN, 256, None, None, 256, 16, None) == B.ERR_ARG
    assert q(256, B.BF16, 1, 16, B.E4M3, B.SCALE_FROM_CURRENT_AMAX, 256, None, None, 256, 16, None) == B.ERR_ARG
    assert q(256, B.BF16, 1, 24, B.E4M3, B.SCALE_GIVEN, 256, None, None, 256, 32, None) == B.ERR_SHAPE
    assert q(256, B.BF16, 1, 32, B.E4M3, B.SCALE_GIVEN, 256, None, None, 256, 16, None) == B.ERR_SHAPE
    assert q(264, B.BF16, 1, 16, B.E4M3, B.SCALE_GIVEN, 256, None, None, 256, 16, None) == B.ERR_ALIGN
    g = lib.fp8mlp_gemm_fp8
    assert g(16, 16, 16, None, 1, 0, 256, 1, 0, None, None, 256, None) == B.ERR_ARG
    assert g(16, 24, 16, 256, 1, 0, 256, 1, 0, None, None, 256, None) == B.ERR_SHAPE
    assert g(16, 16, 16, 256, 1, 3, 256, 1, 0, None, None, 256, None) == B.ERR_ARG
    assert g(16, 16, 16, 264, 1, 0, 256, 1, 0, None, None, 256, None) == B.ERR_ALIGN
    assert lib.fp8mlp_forward(None, 1, None, None, None, None, 0, None, None, None, None) == B.ERR_ARG
    assert lib.fp8mlp_backward(None, 1, None, 0, None, None, None, None, None, None, None) == B.ERR_ARG
    assert lib.fp8mlp_update_scales(None, None, None, None) == B.ERR_ARG
    assert lib.fp8mlp_launch_count() == n0


def test_binding_refuses_to_run_without_the_library(tmp_path, monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", tmp_path / "libfp8mlp.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()


def test_binding_constants_match_the_header():
    """The Python binding repeats the header's enumerators by value; a drift between the two would pass
    wrong flags silently."""
    import ctypes as C
    header = (ROOT / "include" / "fp8mlp.h").read_text()
    enums = {name: int(val) for name, val in re.findall(r"\bFP8MLP_([A-Z0-9_]+)\s*=\s*(-?\d+)", header)}
    for name in ("OK", "ERR_ARG", "ERR_SHAPE", "ERR_ALIGN", "ERR_CUDA", "ERR_TIMEOUT", "ERR_STATE", "E4M3", "E5M2", "BF16", "F32",
                 "SMOOTH", "SAVE_FOR_BWD", "H_BF16", "GU_FP8", "SCALE_GIVEN", "SCALE_FROM_CURRENT_AMAX",
                 "WS_XQ", "WS_W12Q", "WS_W3Q", "WS_HQ", "WS_GU", "WS_DYQ", "WS_DZQ", "WS_HB", "WS_W3B"):
        assert name in enums, name
        assert getattr(B, name) == enums[name], name
    phases = [n for n, _ in sorted(((n[3:], v) for n, v in enums.items() if n.startswith("PH_") and n != "PH_COUNT"),
                                   key=lambda t: t[1])]
    assert len(B.PHASES) == enums["PH_COUNT"] == len(phases)
    # the scale / amax structs: one device pointer per member, in the header's order
    members = lambda typ: re.search(r"typedef struct \{ float ([^}]*); \} " + typ, header).group(1).replace("*", "").replace(" ", "").split(",")
    assert [n for n, _ in B._Scales._fields_] == members("fp8mlp_scales")
    assert [n for n, _ in B._Amax._fields_] == members("fp8mlp_amax")
    assert C.sizeof(B._Scales) == 8 * len(B._Scales._fields_)
