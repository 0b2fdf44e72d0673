"""ctypes front end of the CPU oracle (oracle/fp8mlp_oracle.c).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg
may import this; the CUDA library and its Python binding never do.  This wrapper only
marshals numpy arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "fp8mlp_oracle.c"
_LIB = _HERE / "liboracle.so"
_ADAM_SRC = _HERE / "fp8adam_oracle.c"
_ADAM_LIB = _HERE / "liboracle_adam.so"

E4M3, E5M2 = 0, 1
FLAG_SMOOTH, FLAG_Q_IDENTITY, FLAG_NO_BF16, FLAG_H_BF16, FLAG_GU_FP8 = 1, 2, 4, 8, 16
SCALE_GIVEN, SCALE_CURRENT = 0, 1

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no contraction, no fast-math, OpenMP on the outer GEMM loop)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                               "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    if force or not _ADAM_LIB.exists() or _ADAM_LIB.stat().st_mtime < _ADAM_SRC.stat().st_mtime:
        tmp = _ADAM_LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
                               "-o", str(tmp), str(_ADAM_SRC), "-lm"])
        os.replace(tmp, _ADAM_LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(str(_LIB))
        _lib.orc_decode.restype = C.c_float
        _lib.orc_decode.argtypes = [C.c_int, C.c_uint8]
        _lib.orc_encode.restype = C.c_uint8
        _lib.orc_encode.argtypes = [C.c_int, C.c_float]
        _lib.orc_fmt_max.restype = C.c_float
        _lib.orc_fmt_max.argtypes = [C.c_int]
        _lib.orc_amax.restype = C.c_float
        _lib.orc_amax.argtypes = [C.c_void_p, C.c_int64]
        _lib.orc_amax_rows.restype = C.c_float
        _lib.orc_amax_rows.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p]
        _lib.orc_scale_from_amax.restype = C.c_float
        _lib.orc_scale_from_amax.argtypes = [C.c_int, C.c_float]
        _lib.orc_pow2_scale.restype = C.c_float
        _lib.orc_pow2_scale.argtypes = [C.c_int, C.c_float]
        _lib.orc_swiglu.restype = C.c_float
        _lib.orc_swiglu.argtypes = [C.c_float, C.c_float]
        _lib.orc_swiglu_grad.restype = None
        _lib.orc_swiglu_grad.argtypes = [C.c_float, C.c_float, C.c_float, C.c_void_p, C.c_void_p]
        _lib.orc_f32_to_bf16.restype = C.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [C.c_float]
        _lib.orc_num_threads.restype = C.c_int
        _lib.orc_forward.restype = C.c_int
        _lib.orc_backward.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def fmt_max(fmt: int) -> float:
    return float(lib().orc_fmt_max(fmt))


def encode(fmt: int, v) -> np.ndarray:
    v = _f32(v)
    out = np.empty(v.shape, dtype=np.uint8)
    lib().orc_encode_array(C.c_int(fmt), _p(v), C.c_int64(v.size), _p(out))
    return out


def decode(fmt: int, codes) -> np.ndarray:
    c = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(c.shape, dtype=np.float32)
    lib().orc_decode_array(C.c_int(fmt), _p(c), C.c_int64(c.size), _p(out))
    return out


def bf16_bits(v) -> np.ndarray:
    v = _f32(v)
    out = np.empty(v.shape, dtype=np.uint16)
    lib().orc_f32_to_bf16_array(_p(v), C.c_int64(v.size), _p(out))
    return out


def bf16_to_f32(h) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.shape, dtype=np.float32)
    lib().orc_bf16_to_f32_array(_p(h), C.c_int64(h.size), _p(out))
    return out


def amax(v, row_mul=None) -> float:
    v = _f32(v)
    if row_mul is None:
        return float(lib().orc_amax(_p(v), C.c_int64(v.size)))
    rm = _f32(row_mul)
    return float(lib().orc_amax_rows(_p(v), C.c_int64(v.shape[0]), C.c_int64(v.shape[1]), _p(rm)))


def scale_from_amax(fmt: int, a: float) -> float:
    return float(lib().orc_scale_from_amax(fmt, np.float32(a)))


def pow2_scale(fmt: int, a: float) -> float:
    return float(lib().orc_pow2_scale(fmt, np.float32(a)))


def quantize(src, fmt: int, scale: float, row_mul=None, flags: int = 0):
    """Returns (codes uint8 [rows, cols], decoded float32, amax of src*row_mul)."""
    src = _f32(src)
    rows, cols = src.shape
    rm = None if row_mul is None else _f32(row_mul)
    codes = np.empty((rows, cols), dtype=np.uint8)
    deq = np.empty((rows, cols), dtype=np.float32)
    a = C.c_float(0)
    lib().orc_quantize(_p(src), C.c_int64(rows), C.c_int64(cols), _p(rm), C.c_int(fmt), C.c_float(scale),
                       C.c_uint(flags), _p(codes), C.c_int64(cols), _p(deq), C.byref(a))
    return codes, deq, float(a.value)


def code_stats(fmt: int, codes) -> tuple:
    """(number of zero codes, number of codes at the largest finite magnitude) of a 2-D uint8 array of FP8 codes."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows, cols = codes.shape
    z, t = C.c_int64(0), C.c_int64(0)
    lib().orc_code_stats(C.c_int(fmt), _p(codes), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols), C.byref(z), C.byref(t))
    return int(z.value), int(t.value)


def gemm(A, B) -> np.ndarray:
    """C = A @ B in fp32 with sequential accumulation over the contraction index.

    A [M, K] and B [K, N] may be arbitrary strided 2-D float32 views (e.g. transposes).
    """
    assert A.dtype == np.float32 and B.dtype == np.float32 and A.shape[1] == B.shape[0]
    M, K = A.shape
    N = B.shape[1]
    out = np.empty((M, N), dtype=np.float32)
    lib().orc_gemm(C.c_int64(M), C.c_int64(N), C.c_int64(K),
                   C.c_void_p(A.ctypes.data), C.c_int64(A.strides[0] // 4), C.c_int64(A.strides[1] // 4),
                   C.c_void_p(B.ctypes.data), C.c_int64(B.strides[0] // 4), C.c_int64(B.strides[1] // 4),
                   _p(out))
    return out


def swiglu(u: float, g: float) -> float:
    return float(lib().orc_swiglu(np.float32(u), np.float32(g)))


def swiglu_grad(u: float, g: float, dh: float):
    du, dg = C.c_float(0), C.c_float(0)
    lib().orc_swiglu_grad(np.float32(u), np.float32(g), np.float32(dh), C.byref(du), C.byref(dg))
    return float(du.value), float(dg.value)


def forward(x_bf16, W1, W2, W3, *, flags: int = FLAG_SMOOTH, scale_mode: int = SCALE_CURRENT,
            sx=None, sw12=None, s_h=None, sw3=None, sgu=None, want_float_operands: bool = False) -> dict:
    """Forward of the block.  x_bf16: uint16 [T,d]; W1,W2 [d,f]; W3 [f,d] float32.

    In SCALE_GIVEN mode sx, sw12, s_h[f], sw3 (and sgu with FLAG_GU_FP8) must be supplied.  Returns
    every intermediate the CUDA path can be compared on.
    """
    x_bf16 = np.ascontiguousarray(x_bf16, dtype=np.uint16)
    W1, W2, W3 = _f32(W1), _f32(W2), _f32(W3)
    T, d = x_bf16.shape
    f = W1.shape[1]
    assert W1.shape == (d, f) and W2.shape == (d, f) and W3.shape == (f, d)
    c_sx, c_sw12, c_sw3 = C.c_float(sx or 0), C.c_float(sw12 or 0), C.c_float(sw3 or 0)
    sh = np.zeros(f, dtype=np.float32) if s_h is None else _f32(s_h).copy()
    if scale_mode == SCALE_GIVEN:
        assert None not in (sx, sw12, sw3) and s_h is not None and sh.shape == (f,)
    am = [C.c_float(0) for _ in range(4)]
    gu_fp8 = bool(flags & FLAG_GU_FP8)
    if gu_fp8 and scale_mode == SCALE_GIVEN:
        assert sgu is not None
    c_sgu, a_gu = C.c_float(sgu or 0), C.c_float(0)
    GUq = np.empty((T, 2 * f), np.uint8) if gu_fp8 else None
    r = dict(
        amax_h=np.empty(f, np.float32), Xq=np.empty((T, d), np.uint8), W12q=np.empty((d, 2 * f), np.uint8),
        W3q=np.empty((f, d), np.uint8), Hq=np.empty((T, f), np.uint8), G=np.empty((T, f), np.uint16),
        U=np.empty((T, f), np.uint16), H=np.empty((T, f), np.float32), Y_bits=np.empty((T, d), np.uint16),
        Y=np.empty((T, d), np.float32))
    fl = {}
    if want_float_operands:
        fl = dict(xq_f=np.empty((T, d), np.float32), w12q_f=np.empty((d, 2 * f), np.float32),
                  w3q_f=np.empty((f, d), np.float32), hq_f=np.empty((T, f), np.float32),
                  G_f32=np.empty((T, f), np.float32), U_f32=np.empty((T, f), np.float32))
    rc = lib().orc_forward(
        C.c_int64(T), C.c_int64(d), C.c_int64(f), C.c_uint(flags), C.c_int(scale_mode),
        _p(x_bf16), _p(W1), _p(W2), _p(W3),
        C.byref(c_sx), C.byref(c_sw12), _p(sh), C.byref(c_sw3),
        C.byref(am[0]), C.byref(am[1]), C.byref(am[2]), C.byref(am[3]), _p(r["amax_h"]),
        _p(r["Xq"]), _p(r["W12q"]), _p(r["W3q"]), _p(r["Hq"]), _p(r["G"]), _p(r["U"]), _p(r["H"]),
        _p(r["Y_bits"]), _p(r["Y"]),
        _p(fl.get("xq_f")), _p(fl.get("w12q_f")), _p(fl.get("w3q_f")), _p(fl.get("hq_f")),
        _p(fl.get("G_f32")), _p(fl.get("U_f32")),
        C.byref(c_sgu), C.byref(a_gu), _p(GUq))
    assert rc == 0
    r.update(fl)
    if gu_fp8:
        r.update(GUq=GUq, sgu=float(c_sgu.value), amax_gu=float(a_gu.value))
    r.update(sx=float(c_sx.value), sw12=float(c_sw12.value), sw3=float(c_sw3.value), s_h=sh,
             amax_x=float(am[0].value), amax_w1=float(am[1].value), amax_w2=float(am[2].value),
             amax_w3=float(am[3].value), flags=flags, T=T, d=d, f=f)
    return r


def backward(fwd: dict, dy_bf16, *, scale_mode: int = SCALE_CURRENT, sdy=None, sdz=None,
             want_intermediates: bool = False) -> dict:
    """Backward of the block from the dict forward() returned (same flags).  want_intermediates adds the fp32
    dH [T,f] and dZ = [dG | dU] [T,2f] as they stand before the E5M2 cast."""
    dy_bf16 = np.ascontiguousarray(dy_bf16, dtype=np.uint16)
    T, d, f, flags = fwd["T"], fwd["d"], fwd["f"], fwd["flags"]
    assert dy_bf16.shape == (T, d)
    if scale_mode == SCALE_GIVEN:
        assert sdy is not None and sdz is not None
    c_sdy, c_sdz = C.c_float(sdy or 0), C.c_float(sdz or 0)
    a_dy, a_dz = C.c_float(0), C.c_float(0)
    r = dict(dYq=np.empty((T, d), np.uint8), dZq=np.empty((T, 2 * f), np.uint8),
             dX_bits=np.empty((T, d), np.uint16), dX=np.empty((T, d), np.float32),
             dW1=np.empty((d, f), np.float32), dW2=np.empty((d, f), np.float32), dW3=np.empty((f, d), np.float32))
    if want_intermediates:
        r.update(dH=np.empty((T, f), np.float32), dZ=np.empty((T, 2 * f), np.float32))
    rc = lib().orc_backward(
        C.c_int64(T), C.c_int64(d), C.c_int64(f), C.c_uint(flags), C.c_int(scale_mode), _p(dy_bf16),
        _p(fwd["Xq"]), _p(fwd["W12q"]), _p(fwd["W3q"]), _p(fwd["Hq"]),
        _p(fwd.get("xq_f")), _p(fwd.get("w12q_f")), _p(fwd.get("w3q_f")), _p(fwd.get("hq_f")),
        _p(fwd["G"]), _p(fwd["U"]), _p(fwd.get("G_f32")), _p(fwd.get("U_f32")),
        C.c_float(fwd["sx"]), C.c_float(fwd["sw12"]), _p(fwd["s_h"]), C.c_float(fwd["sw3"]),
        C.byref(c_sdy), C.byref(c_sdz), C.byref(a_dy), C.byref(a_dz),
        _p(r["dYq"]), _p(r["dZq"]), _p(r["dX_bits"]), _p(r["dX"]), _p(r["dW1"]), _p(r["dW2"]), _p(r["dW3"]),
        _p(fwd.get("GUq")), C.c_float(fwd.get("sgu", 1.0)), _p(r.get("dH")), _p(r.get("dZ")))
    assert rc == 0
    r.update(sdy=float(c_sdy.value), sdz=float(c_sdz.value), amax_dy=float(a_dy.value), amax_dz=float(a_dz.value))
    return r


def mlp_f64(x, W1, W2, W3, s=None):
    """The unquantised block in fp64 (definition).  Returns (H, Y)."""
    x, W1, W2, W3 = (np.ascontiguousarray(a, dtype=np.float64) for a in (x, W1, W2, W3))
    T, d = x.shape
    f = W1.shape[1]
    sv = None if s is None else np.ascontiguousarray(s, dtype=np.float64)
    H, Y = np.empty((T, f)), np.empty((T, d))
    lib().orc_mlp_f64(C.c_int64(T), C.c_int64(d), C.c_int64(f), _p(x), _p(W1), _p(W2), _p(W3), _p(sv), _p(H), _p(Y))
    return H, Y


def mlp_f64_backward(x, W1, W2, W3, dY):
    x, W1, W2, W3, dY = (np.ascontiguousarray(a, dtype=np.float64) for a in (x, W1, W2, W3, dY))
    T, d = x.shape
    f = W1.shape[1]
    dX, dW1, dW2, dW3 = np.empty((T, d)), np.empty((d, f)), np.empty((d, f)), np.empty((f, d))
    lib().orc_mlp_f64_backward(C.c_int64(T), C.c_int64(d), C.c_int64(f), _p(x), _p(W1), _p(W2), _p(W3), _p(dY),
                               _p(dX), _p(dW1), _p(dW2), _p(dW3))
    return dX, dW1, dW2, dW3


# ---------------------------------------------------------------- Adam with FP8 moments (fp8adam_oracle.c)
ADAM_Q_IDENTITY, ADAM_M_AS_E5M2, ADAM_V_AS_E4M3 = 1, 2, 4
_adam = None


def _adam_lib():
    global _adam
    if _adam is None:
        build()
        _adam = C.CDLL(str(_ADAM_LIB))
        _adam.adam_decode.restype = C.c_float
        _adam.adam_decode.argtypes = [C.c_int, C.c_uint8]
        _adam.adam_encode.restype = C.c_uint8
        _adam.adam_encode.argtypes = [C.c_int, C.c_float]
        _adam.adam_bias_correction.restype = C.c_float
        _adam.adam_bias_correction.argtypes = [C.c_float, C.c_int64]
        _adam.adam_step.restype = None
    return _adam


def adam_encode(second_moment: bool, v: float) -> int:
    return int(_adam_lib().adam_encode(int(second_moment), np.float32(v)))


def adam_decode(second_moment: bool, code: int) -> float:
    return float(_adam_lib().adam_decode(int(second_moment), code))


def adam_bias_correction(beta: float, step: int) -> float:
    return float(_adam_lib().adam_bias_correction(np.float32(beta), step))


def adam_step(w, g, mq, vq, *, lr, beta1, beta2, eps, weight_decay, step, sm_in=1.0, sv_in=1.0, sm_out=1.0,
              sv_out=1.0, m32=None, v32=None, flags=0):
    """One Adam step in place (w fp32; mq, vq uint8 codes, or m32, v32 fp32 with the quantisation off).
    Returns (amax_m, amax_v) of the new fp32 moments."""
    assert w.dtype == np.float32 and g.dtype == np.float32 and w.flags.c_contiguous and g.flags.c_contiguous
    if m32 is not None:
        flags |= ADAM_Q_IDENTITY
        assert m32.dtype == np.float32 and v32.dtype == np.float32
    else:
        assert mq.dtype == np.uint8 and vq.dtype == np.uint8
    am, av = C.c_float(0), C.c_float(0)
    _adam_lib().adam_step(C.c_int64(w.size), C.c_uint(flags), _p(w), _p(g), _p(mq), _p(vq), _p(m32), _p(v32),
                          C.c_float(lr), C.c_float(beta1), C.c_float(beta2), C.c_float(eps), C.c_float(weight_decay),
                          C.c_int64(step), C.c_float(sm_in), C.c_float(sv_in), C.c_float(sm_out), C.c_float(sv_out),
                          C.byref(am), C.byref(av))
    return float(am.value), float(av.value)


def adam_step_and_cast(w, g, mq, vq, *, cols: int, scale: float, row_div=None, **adam):
    """The optimizer step followed by the E4M3 cast of the updated master weights for the next forward (Section 6.2
    of the paper keeps high-precision master weights and quantises them to E4M3 for the forward phase): the
    composition adam_step -> quantize of this module, nothing else.  w is updated in place; returns
    (amax_m, amax_v, codes [n / cols, cols], amax of the cast values)."""
    am, av = adam_step(w, g, mq, vq, **adam)
    inv = None if row_div is None else (np.float32(1.0) / np.asarray(row_div, np.float32)).astype(np.float32)
    codes, _, amax_w = quantize(w.reshape(-1, cols), E4M3, scale, row_mul=inv)
    return am, av, codes, amax_w
