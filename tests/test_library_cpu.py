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


def test_gemm_plans_at_the_benchmark_shapes():
    """Host logic of the GEMM launcher (tiling, rasterisation, split contraction, staged stores), asked through the
    C ABI without a device, at the 7B shape for the token counts of the benchmark's sweep."""
    from paper_2409_12517_b200 import binding as B
    d, f, sms = 4096, 11008, 148
    plan = lambda kind, M, N, K, **kw: B.fp8mlp_gemm_plan(kind, M, N, K, sms, **kw)
    # T = 16384: CTA pairs everywhere; the bf16-output GEMMs on 256 x 512 tiles (their output staged for bulk stores: the
    # epilogue of a wide tile is not hidden); nothing split; the fp32 outputs stored directly
    T = 16384
    g1, g2 = plan(B.GEMM_SWIGLU_FWD, T, f, d), plan(B.GEMM_BF16_OUT, T, d, f)
    assert (g1["cta_pairs"], g1["tile_rows"], g1["tile_cols"], g1["m_tiles"], g1["n_tiles"], g1["k_stages"]) == (1, 256, 128, 64, 86, 32)
    assert (g2["tile_cols"], g2["n_tiles"], g2["k_stages"], g2["split_k"], g2["staged_stores"]) == (512, 8, 86, 1, 1)
    # rasterisation: bands along the smaller operand, the whole of it while it is under 96 MiB
    assert (g2["band_along_n"], g2["band_tiles"]) == (1, 8)                                     # all of W3' (45 MB)
    w3, d1, w12 = plan(B.GEMM_F32_OUT, f, d, T), plan(B.GEMM_BF16_OUT, T, d, 2 * f), plan(B.GEMM_F32_OUT, d, 2 * f, T)
    assert (w3["band_along_n"], w3["band_tiles"]) == (1, 16) and (d1["band_along_n"], d1["band_tiles"]) == (1, 8)
    assert (w12["band_along_n"], w12["band_tiles"]) == (0, 16) and w12["work_items"] == 16 * 86 and w12["staged_stores"] == 0
    big = plan(B.GEMM_BF16_OUT, 8192, 8192, 2 * 28672)                                           # 70B input gradient: W12 is 470 MB
    assert big["band_along_n"] == 0 or big["band_tiles"] < big["n_tiles"]
    assert (g1["band_along_n"], g1["band_tiles"]) == (0, 16)                                     # fused epilogues: 16 row tiles
    # T = 512: 32 tiles for 74 CTA pairs -> the long contractions are split in two; the weight gradients (4 stages of
    # work per tile) stage their output; without a context's workspace nothing is split
    T = 512
    g2, d1 = plan(B.GEMM_BF16_OUT, T, d, f), plan(B.GEMM_BF16_OUT, T, d, 2 * f)
    assert (g2["tile_cols"], g2["m_tiles"] * g2["n_tiles"], g2["split_k"], g2["stages_per_share"], g2["work_items"]) == (256, 32, 2, 43, 64)
    assert (d1["split_k"], d1["stages_per_share"]) == (2, 86)
    assert plan(B.GEMM_BF16_OUT, T, d, f, with_workspace=False)["split_k"] == 1
    w3, w12 = plan(B.GEMM_F32_OUT, f, d, T), plan(B.GEMM_F32_OUT, d, 2 * f, T)
    assert w3["k_stages"] == 4 and w3["staged_stores"] == 1 and w12["staged_stores"] == 1 and w3["split_k"] == 1
    assert plan(B.GEMM_F32_OUT, f, d, 2048)["staged_stores"] == 0                                # 16 stages: direct stores
    assert plan(B.GEMM_SWIGLU_BWD, T, f, d)["split_k"] == 1                                       # fused epilogues never split
    # every share of a split contraction is non-empty and the shares cover it
    for K in (1024, 1152, 2304, 4608, 11008, 22016, 100000):
        p = plan(B.GEMM_BF16_OUT, 256, 256, K)
        assert (p["split_k"] - 1) * p["stages_per_share"] < p["k_stages"] <= p["split_k"] * p["stages_per_share"]
        assert p["split_k"] == 1 or p["stages_per_share"] >= 8
    # at most 128 rows: single CTAs with 128-row tiles
    s = plan(B.GEMM_BF16_OUT, 128, 4096, 4096)
    assert (s["cta_pairs"], s["tile_rows"]) == (0, 128)
    assert B.lib().fp8mlp_gemm_plan(7, 16, 16, 16, 148, 0, None) == B.ERR_ARG
