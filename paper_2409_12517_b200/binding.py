"""Python binding of libfp8mlp.so: same names as the C ABI, argument marshalling only.

Every function takes torch CUDA tensors (PyTorch is used for device memory and streams),
passes their device pointers and the current CUDA stream to the C entry point of the same
name, and raises Fp8MlpError on a non-zero status.  No step of the method runs in Python,
and there is no fallback: if the CUDA library is missing, loading fails loudly.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libfp8mlp.so"

OK, ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_CUDA, ERR_TIMEOUT, ERR_STATE, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5, -6, -7
STATIC_SCRATCH_BYTES = 4 * 1024 * 1024
E4M3, E5M2 = 0, 1
BF16, F32 = 0, 1
SMOOTH, SAVE_FOR_BWD, H_BF16, GU_FP8 = 1, 2, 4, 8
SCALE_GIVEN, SCALE_FROM_CURRENT_AMAX, SCALE_GIVEN_WEIGHTS_CAST = 0, 1, 2
WS_XQ, WS_W12Q, WS_W3Q, WS_HQ, WS_GU, WS_DYQ, WS_DZQ, WS_HB, WS_W3B = range(9)

EXPORTS = [
    "fp8mlp_create", "fp8mlp_destroy", "fp8mlp_strerror", "fp8mlp_last_cuda_error", "fp8mlp_status",
    "fp8mlp_workspace", "fp8mlp_launch_count", "fp8mlp_quantize", "fp8mlp_update_scales",
    "fp8mlp_forward", "fp8mlp_backward", "fp8mlp_gemm_fp8", "fp8mlp_profile_enable", "fp8mlp_profile_read",
    "fp8mlp_forward_static", "fp8mlp_adam_step", "fp8mlp_scale_from_amax",
    "fp8mlp_merge_weights", "fp8mlp_forward_merged", "fp8mlp_gemm_bf16",
    "fp8mlp_selftest_wait_timeout", "fp8mlp_adam_step_cast", "fp8mlp_gemm_plan", "fp8mlp_code_stats",
]
PHASES = ["quant_x", "quant_w12", "quant_w3", "gemm1_swiglu", "gemm2_down", "quant_dy", "dgrad2_swiglu_bwd",
          "wgrad3", "dgrad1", "wgrad12", "misc"]


class Fp8MlpError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().fp8mlp_strerror(code).decode()
        detail = lib().fp8mlp_last_cuda_error().decode() if code == ERR_CUDA else ""
        super().__init__(f"{where}: {msg} ({code}){' — ' + detail if detail else ''}")


class _Scales(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("x", "w12", "w3", "dy", "dz", "h", "gu")]


class _Amax(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("x", "w1", "w2", "w3", "dy", "dz", "h", "gu")]


class _AdamTensor(C.Structure):
    _fields_ = [("w", C.c_void_p), ("g", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p), ("n", C.c_int64),
                ("scale_m_in", C.c_void_p), ("scale_v_in", C.c_void_p), ("scale_m_out", C.c_void_p),
                ("scale_v_out", C.c_void_p), ("amax_m", C.c_void_p), ("amax_v", C.c_void_p)]


class _GemmPlan(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("cta_pairs", "tile_rows", "tile_cols", "m_tiles", "n_tiles", "k_stages", "split_k",
                                       "stages_per_share", "band_along_n", "band_tiles", "staged_stores")] + [("work_items", C.c_int64)]


class _AdamCast(C.Structure):
    _fields_ = [("dst", C.c_void_p), ("cols", C.c_int64), ("ld_dst", C.c_int64), ("scale", C.c_void_p),
                ("row_div", C.c_void_p), ("amax", C.c_void_p)]


_lib = None


def lib():
    """The loaded shared library (built by build.py); raises if it is not there."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2409_12517_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(str(LIB_PATH))
        L.fp8mlp_strerror.restype = C.c_char_p
        L.fp8mlp_strerror.argtypes = [C.c_int]
        L.fp8mlp_last_cuda_error.restype = C.c_char_p
        L.fp8mlp_launch_count.restype = C.c_int64
        L.fp8mlp_create.argtypes = [C.POINTER(C.c_void_p), C.c_int64, C.c_int64, C.c_int64, C.c_uint32]
        L.fp8mlp_destroy.argtypes = [C.c_void_p]
        L.fp8mlp_status.argtypes = [C.c_void_p, C.c_void_p]
        L.fp8mlp_workspace.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_int64)]
        L.fp8mlp_quantize.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.fp8mlp_update_scales.argtypes = [C.c_void_p, C.POINTER(_Amax), C.POINTER(_Scales), C.c_void_p]
        L.fp8mlp_forward.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                     C.POINTER(_Scales), C.POINTER(_Amax), C.c_void_p, C.c_void_p]
        L.fp8mlp_backward.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int, C.POINTER(_Scales), C.POINTER(_Amax),
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.fp8mlp_gemm_fp8.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int,
                                      C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.fp8mlp_forward_static.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_uint32, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_int, C.POINTER(_Scales), C.POINTER(_Amax),
                                            C.c_void_p, C.c_void_p]
        L.fp8mlp_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.fp8mlp_gemm_bf16.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                       C.c_void_p, C.c_void_p]
        L.fp8mlp_merge_weights.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                           C.POINTER(_Scales), C.POINTER(_Amax), C.c_void_p]
        L.fp8mlp_forward_merged.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int, C.POINTER(_Scales),
                                            C.POINTER(_Amax), C.c_void_p, C.c_void_p]
        L.fp8mlp_adam_step.argtypes = [C.POINTER(_AdamTensor), C.c_int, C.c_float, C.c_float, C.c_float, C.c_float,
                                       C.c_float, C.c_int64, C.c_void_p]
        L.fp8mlp_adam_step_cast.argtypes = [C.POINTER(_AdamTensor), C.POINTER(_AdamCast), C.c_int, C.c_float, C.c_float,
                                            C.c_float, C.c_float, C.c_float, C.c_int64, C.c_void_p]
        L.fp8mlp_code_stats.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.fp8mlp_gemm_plan.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.POINTER(_GemmPlan)]
        L.fp8mlp_scale_from_amax.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.fp8mlp_profile_enable.argtypes = [C.c_void_p, C.c_int]
        L.fp8mlp_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        missing = [name for name in EXPORTS if not hasattr(L, name)]
        if missing:
            raise RuntimeError(f"{LIB_PATH} does not export {missing}")
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != OK:
        raise Fp8MlpError(code, where)


def _scales(s: dict) -> _Scales:
    return _Scales(*[(s[n].data_ptr() if s.get(n) is not None else None) for n in ("x", "w12", "w3", "dy", "dz", "h", "gu")])


def _amax(a: dict | None):
    if a is None:
        return None
    return _Amax(*[(a[n].data_ptr() if a.get(n) is not None else None) for n in ("x", "w1", "w2", "w3", "dy", "dz", "h", "gu")])


def fp8mlp_launch_count() -> int:
    return int(lib().fp8mlp_launch_count())


def fp8mlp_create(T_max: int, d_model: int, d_ff: int, flags: int) -> int:
    """Returns the context handle (an integer address)."""
    h = C.c_void_p()
    _check(lib().fp8mlp_create(C.byref(h), T_max, d_model, d_ff, flags), "fp8mlp_create")
    return h.value


def fp8mlp_destroy(ctx: int) -> None:
    _check(lib().fp8mlp_destroy(C.c_void_p(ctx)), "fp8mlp_destroy")


def fp8mlp_status(ctx: int) -> int:
    """Synchronises the current stream and returns OK or ERR_TIMEOUT (does not raise)."""
    return int(lib().fp8mlp_status(C.c_void_p(ctx), _stream()))


def fp8mlp_selftest_wait_timeout(ctx: int, timeout_us: int) -> None:
    """Runs a kernel whose bounded wait must time out; afterwards fp8mlp_status reports ERR_TIMEOUT once."""
    _check(lib().fp8mlp_selftest_wait_timeout(C.c_void_p(ctx), timeout_us, _stream()), "fp8mlp_selftest_wait_timeout")


def fp8mlp_workspace(ctx: int, which: int):
    """(device pointer, bytes) of one of the WS_* buffers."""
    p, n = C.c_void_p(), C.c_int64()
    _check(lib().fp8mlp_workspace(C.c_void_p(ctx), which, C.byref(p), C.byref(n)), "fp8mlp_workspace")
    return p.value, n.value


def fp8mlp_profile_enable(ctx: int, on: bool) -> None:
    _check(lib().fp8mlp_profile_enable(C.c_void_p(ctx), int(on)), "fp8mlp_profile_enable")


def fp8mlp_profile_read(ctx: int) -> dict:
    """{phase name: (milliseconds, brackets)} accumulated since the last read."""
    n = len(PHASES)
    ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
    _check(lib().fp8mlp_profile_read(C.c_void_p(ctx), ms, cnt), "fp8mlp_profile_read")
    return {PHASES[i]: (float(ms[i]), int(cnt[i])) for i in range(n)}


def fp8mlp_quantize(src, fp8_fmt: int, scale_mode: int, scale, amax, row_mul, dst, ld_dst: int | None = None) -> None:
    """src: 2-D bf16 or fp32 tensor; dst: uint8 tensor; scale/amax: 1-element fp32 tensors."""
    rows, cols = src.shape
    dtype = {torch.bfloat16: BF16, torch.float32: F32}[src.dtype]
    ld = cols if ld_dst is None else ld_dst
    _check(lib().fp8mlp_quantize(_ptr(src), dtype, rows, cols, fp8_fmt, scale_mode, _ptr(scale), _ptr(amax),
                                 _ptr(row_mul), _ptr(dst), ld, _stream()), "fp8mlp_quantize")


def fp8mlp_update_scales(ctx: int, amax: dict, scales: dict) -> None:
    a, s = _amax(amax), _scales(scales)
    _check(lib().fp8mlp_update_scales(C.c_void_p(ctx), C.byref(a), C.byref(s), _stream()), "fp8mlp_update_scales")


def fp8mlp_forward(ctx: int, T: int, x, W1, W2, W3, scale_mode: int, scales: dict, amax: dict | None, y) -> None:
    s, a = _scales(scales), _amax(amax)
    _check(lib().fp8mlp_forward(C.c_void_p(ctx), T, _ptr(x), _ptr(W1), _ptr(W2), _ptr(W3), scale_mode, C.byref(s),
                                C.byref(a) if a is not None else None, _ptr(y), _stream()), "fp8mlp_forward")


def fp8mlp_forward_static(T: int, d_model: int, d_ff: int, flags: int, x, W1, W2, W3, scale_mode: int,
                          scales: dict, amax: dict | None, y) -> None:
    """Forward for callers that cannot allocate device memory: no context, the library's built-in
    4 MiB scratch instead (shapes beyond it raise ERR_TOO_LARGE).  Calls that overlap on the GPU race."""
    s, a = _scales(scales), _amax(amax)
    _check(lib().fp8mlp_forward_static(T, d_model, d_ff, flags, _ptr(x), _ptr(W1), _ptr(W2), _ptr(W3), scale_mode,
                                       C.byref(s), C.byref(a) if a is not None else None, _ptr(y), _stream()),
           "fp8mlp_forward_static")


def fp8mlp_backward(ctx: int, T: int, dy, scale_mode: int, scales: dict, amax: dict | None, dx, dW1, dW2, dW3) -> None:
    s, a = _scales(scales), _amax(amax)
    _check(lib().fp8mlp_backward(C.c_void_p(ctx), T, _ptr(dy), scale_mode, C.byref(s),
                                 C.byref(a) if a is not None else None, _ptr(dx), _ptr(dW1), _ptr(dW2), _ptr(dW3),
                                 _stream()), "fp8mlp_backward")


def fp8mlp_gemm_fp8(M: int, N: int, K: int, A, a_kmajor: bool, a_fmt: int, B, b_kmajor: bool, b_fmt: int,
                    scale_a, scale_b, out) -> None:
    _check(lib().fp8mlp_gemm_fp8(M, N, K, _ptr(A), int(a_kmajor), a_fmt, _ptr(B), int(b_kmajor), b_fmt,
                                 _ptr(scale_a), _ptr(scale_b), _ptr(out), _stream()), "fp8mlp_gemm_fp8")


def fp8mlp_merge_weights(ctx: int, W1, W2, W3, s, scale_mode: int, scales: dict, amax: dict | None) -> None:
    sc, a = _scales(scales), _amax(amax)
    _check(lib().fp8mlp_merge_weights(C.c_void_p(ctx), _ptr(W1), _ptr(W2), _ptr(W3), _ptr(s), scale_mode, C.byref(sc),
                                      C.byref(a) if a is not None else None, _stream()), "fp8mlp_merge_weights")


def fp8mlp_forward_merged(ctx: int, T: int, x, scale_mode: int, scales: dict, amax: dict | None, y) -> None:
    sc, a = _scales(scales), _amax(amax)
    _check(lib().fp8mlp_forward_merged(C.c_void_p(ctx), T, _ptr(x), scale_mode, C.byref(sc),
                                       C.byref(a) if a is not None else None, _ptr(y), _stream()), "fp8mlp_forward_merged")


def fp8mlp_adam_step(tensors: list, lr: float, beta1: float, beta2: float, eps: float, weight_decay: float,
                     step: int) -> None:
    """tensors: dicts with torch tensors w, g (fp32), m, v (uint8 codes) and 1-element fp32 tensors
    scale_m_in, scale_v_in, scale_m_out, scale_v_out, amax_m, amax_v.  Everything is updated in place."""
    arr = (_AdamTensor * len(tensors))()
    for a, t in zip(arr, tensors):
        a.w, a.g, a.m, a.v, a.n = t["w"].data_ptr(), t["g"].data_ptr(), t["m"].data_ptr(), t["v"].data_ptr(), t["w"].numel()
        for k in ("scale_m_in", "scale_v_in", "scale_m_out", "scale_v_out", "amax_m", "amax_v"):
            setattr(a, k, t[k].data_ptr())
    _check(lib().fp8mlp_adam_step(arr, len(tensors), lr, beta1, beta2, eps, weight_decay, step, _stream()),
           "fp8mlp_adam_step")


def fp8mlp_adam_step_cast(tensors: list, casts: list, lr: float, beta1: float, beta2: float, eps: float,
                          weight_decay: float, step: int) -> None:
    """fp8mlp_adam_step that also writes the E4M3 codes of the updated weights.  casts: one entry per tensor, None or a
    dict with dst (device pointer as int, or a uint8 tensor), cols, ld_dst, scale (1-element fp32 tensor), and
    optionally row_div (fp32 tensor, one per row) and amax (1-element fp32 tensor)."""
    arr = (_AdamTensor * len(tensors))()
    for a, t in zip(arr, tensors):
        a.w, a.g, a.m, a.v, a.n = t["w"].data_ptr(), t["g"].data_ptr(), t["m"].data_ptr(), t["v"].data_ptr(), t["w"].numel()
        for k in ("scale_m_in", "scale_v_in", "scale_m_out", "scale_v_out", "amax_m", "amax_v"):
            setattr(a, k, t[k].data_ptr())
    carr = (_AdamCast * len(tensors))()
    for c, d in zip(carr, casts):
        if d is None:
            continue
        c.dst = d["dst"] if isinstance(d["dst"], int) else d["dst"].data_ptr()
        c.cols, c.ld_dst, c.scale = d["cols"], d["ld_dst"], d["scale"].data_ptr()
        c.row_div = d["row_div"].data_ptr() if d.get("row_div") is not None else None
        c.amax = d["amax"].data_ptr() if d.get("amax") is not None else None
    _check(lib().fp8mlp_adam_step_cast(arr, carr, len(tensors), lr, beta1, beta2, eps, weight_decay, step, _stream()),
           "fp8mlp_adam_step_cast")


def fp8mlp_code_stats(codes, fp8_fmt: int, counts, ld: int | None = None) -> None:
    """codes: 2-D uint8 CUDA tensor (row stride ld, default cols); counts: int64 CUDA tensor of 2 elements, receives
    (zero codes, codes at the largest finite magnitude)."""
    rows, cols = codes.shape
    _check(lib().fp8mlp_code_stats(_ptr(codes), rows, cols, cols if ld is None else ld, fp8_fmt, C.c_void_p(counts.data_ptr()),
                                   C.c_void_p(counts.data_ptr() + 8), _stream()), "fp8mlp_code_stats")


GEMM_F32_OUT, GEMM_BF16_OUT, GEMM_SWIGLU_FWD, GEMM_SWIGLU_BWD = 0, 1, 2, 3


def fp8mlp_gemm_plan(kind: int, M: int, N: int, K: int, sm_count: int = 148, with_workspace: bool = True) -> dict:
    """How the library would tile and schedule one GEMM (host arithmetic only; works without a GPU)."""
    p = _GemmPlan()
    _check(lib().fp8mlp_gemm_plan(kind, M, N, K, sm_count, int(with_workspace), C.byref(p)), "fp8mlp_gemm_plan")
    return {n: getattr(p, n) for n, _ in _GemmPlan._fields_}


def fp8mlp_scale_from_amax(amax, fp8_fmt: int, scale) -> None:
    _check(lib().fp8mlp_scale_from_amax(_ptr(amax), fp8_fmt, _ptr(scale), _stream()), "fp8mlp_scale_from_amax")


def fp8mlp_gemm_bf16(M: int, N: int, K: int, A, a_kmajor: bool, B, b_kmajor: bool, out) -> None:
    _check(lib().fp8mlp_gemm_bf16(M, N, K, _ptr(A), int(a_kmajor), _ptr(B), int(b_kmajor), _ptr(out), _stream()),
           "fp8mlp_gemm_bf16")


# ---------------------------------------------------------------- conveniences (allocation only)

def new_scales(d_ff: int, device="cuda") -> dict:
    """Caller-owned scale buffers, initialised to 1."""
    s = {n: torch.ones(1, dtype=torch.float32, device=device) for n in ("x", "w12", "w3", "dy", "dz", "gu")}
    s["h"] = torch.ones(d_ff, dtype=torch.float32, device=device)
    return s


def new_amax(d_ff: int, device="cuda") -> dict:
    a = {n: torch.zeros(1, dtype=torch.float32, device=device) for n in ("x", "w1", "w2", "w3", "dy", "dz", "gu")}
    a["h"] = torch.zeros(d_ff, dtype=torch.float32, device=device)
    return a


class _DeviceBytes:
    """Exposes a raw device pointer through the CUDA array interface (zero-copy view for torch)."""

    def __init__(self, ptr: int, nbytes: int):
        self.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (ptr, False), "version": 2}


def workspace_tensor(ctx: int, which: int, shape, dtype):
    """A copy of the first prod(shape) elements of a workspace buffer, as a torch tensor (for tests)."""
    ptr, nbytes = fp8mlp_workspace(ctx, which)
    n = 1
    for s in shape:
        n *= s
    need = n * torch.empty(0, dtype=dtype).element_size()
    assert need <= nbytes
    if need == 0:
        return torch.empty(shape, dtype=dtype, device="cuda")
    raw = torch.as_tensor(_DeviceBytes(ptr, nbytes), device="cuda")
    return raw[:need].view(dtype).view(shape).clone()


def workspace_fill(ctx: int, which: int, byte: int) -> None:
    """Sets every byte of a workspace buffer (for tests: a poison pattern shows what a call failed to write)."""
    ptr, nbytes = fp8mlp_workspace(ctx, which)
    if nbytes:
        torch.as_tensor(_DeviceBytes(ptr, nbytes), device="cuda").fill_(byte)
