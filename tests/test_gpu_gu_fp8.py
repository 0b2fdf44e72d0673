"""FP8MLP_GU_FP8 through the C ABI: the SwiGLU inputs G, U are kept for backward as E4M3 codes with one
per-tensor scale instead of bf16 (an option; the paper does not say how these activations are stored).
Forward + backward against the oracle's ORC_FLAG_GU_FP8 path, just-in-time and delayed scales, shapes with
ragged channel tiles (f % 256 != 0), a 16-channel tail (f % 32 == 16) and several token tiles."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from helpers import (bf16_bits_to_f32, bf16_dev_to_bits, check_amax_dz, code_mismatch, e4m3_step, nmax_err, nmax_err_bf16,
                     to_dev, to_dev_bf16)
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu

CODE_FRAC = 1e-3
OUT_TOL = 2e-3


def _run(w, flags, mode, given=None):
    T, d, f = w.T, w.d, w.f
    ctx = B.fp8mlp_create(T, d, f, flags | B.SAVE_FOR_BWD | B.GU_FP8)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        if given is not None:
            for k, v in given.items():
                sc[k].copy_(to_dev(np.atleast_1d(np.asarray(v, np.float32))))
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros_like(y)
        dW1 = torch.full((d, f), float("nan"), device="cuda")
        dW2 = torch.full((d, f), float("nan"), device="cuda")
        dW3 = torch.full((f, d), float("nan"), device="cuda")
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3), mode, sc, am, y)
        ws = lambda which, shape: B.workspace_tensor(ctx, which, shape, torch.uint8).cpu().numpy()
        out = dict(GUq=ws(B.WS_GU, (T, 2 * f)), Hq=ws(B.WS_HQ, (T, f)), Xq=ws(B.WS_XQ, (T, d)))
        B.fp8mlp_backward(ctx, T, to_dev_bf16(w.dY), mode, sc, am, dx, dW1, dW2, dW3)
        assert B.fp8mlp_status(ctx) == B.OK
        out.update(dZq=ws(B.WS_DZQ, (T, 2 * f)), Y=bf16_dev_to_bits(y), dX=bf16_dev_to_bits(dx),
                   dW1=dW1.cpu().numpy(), dW2=dW2.cpu().numpy(), dW3=dW3.cpu().numpy(),
                   sc={k: v.cpu().numpy() for k, v in sc.items()}, am={k: v.cpu().numpy() for k, v in am.items()})
        return out
    finally:
        B.fp8mlp_destroy(ctx)


def _check(r, fw, bw, given_scales):
    assert np.array_equal(r["Xq"], fw["Xq"])
    assert np.isclose(r["am"]["gu"][0], fw["amax_gu"], rtol=1e-5, atol=0), "max of |G|, |U|"
    if given_scales:
        assert r["sc"]["gu"][0] == np.float32(fw["sgu"]), "the given scale is left alone"
    else:
        assert np.isclose(r["sc"]["gu"][0], fw["sgu"], rtol=1e-5, atol=0), "scale of the saved activations"
    frac, worst = code_mismatch(r["GUq"], fw["GUq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"saved G, U codes: {frac:.2e} differ, worst {worst} steps"
    frac, worst = code_mismatch(r["Hq"], fw["Hq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"Hq codes: {frac:.2e} differ, worst {worst} steps"
    assert nmax_err_bf16(r["Y"], fw["Y"]) <= OUT_TOL, "Y"
    # the saved activations are E4M3 codes here: where a stored code differs from the oracle's (by one step: checked
    # above) the maximum of dZ is held to the envelope that step opens, elsewhere to the accumulation-order bar
    gu = oracle.decode(oracle.E4M3, fw["GUq"]).astype(np.float64)
    f = gu.shape[1] // 2
    inv = 1.0 / float(fw["sgu"])
    differs = r["GUq"] != fw["GUq"]                      # the step is granted only where the stored code differs
    check_amax_dz("amax of dZ", r["am"]["dz"][0], bw, gu[:, :f] * inv, gu[:, f:] * inv,
                  np.where(differs[:, :f], e4m3_step(gu[:, :f]), 0.0) * inv, np.where(differs[:, f:], e4m3_step(gu[:, f:]), 0.0) * inv)
    assert r["sc"]["dz"][0] == np.float32(bw["sdz"]), "scale of dZ"
    frac, worst = code_mismatch(r["dZq"], bw["dZq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"dZq codes: {frac:.2e} differ, worst {worst} steps"
    assert nmax_err_bf16(r["dX"], bw["dX"]) <= OUT_TOL, "dX"
    for name in ("dW1", "dW2", "dW3"):
        assert np.all(np.isfinite(r[name])), name
        e = nmax_err(r[name], bw[name])
        assert e <= OUT_TOL, f"{name}: {e}"


@pytest.mark.parametrize("smooth", [True, False])
@pytest.mark.parametrize("cfg", ["tiny", (333, 512, 1040), (700, 256, 1536), (1, 16, 16)])
def test_gu_fp8_current_amax(cfg, smooth):
    w = wl.make_config("tiny") if cfg == "tiny" else wl.make("gu8", 41, *cfg, w_std=0.05, channel_outlier_frac=0.01)
    ofl = (oracle.FLAG_SMOOTH if smooth else 0) | oracle.FLAG_GU_FP8
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=ofl)
    bw = oracle.backward(fw, w.dY, want_intermediates=True)
    r = _run(w, B.SMOOTH if smooth else 0, B.SCALE_FROM_CURRENT_AMAX)
    _check(r, fw, bw, given_scales=False)


@pytest.mark.parametrize("shape", [(200, 320, 272), (130, 144, 528), (515, 256, 400)])
def test_gu_fp8_given_scales(shape):
    """Delayed scaling: every scale, the one of the saved activations included, comes from a previous batch
    (through the oracle), so values may saturate; the codes still agree."""
    T, d, f = shape
    prev = wl.make("prev", 7, T, d, f, w_std=0.05)
    w = wl.make("cur", 8, T, d, f, w_std=0.05)
    ofl = oracle.FLAG_SMOOTH | oracle.FLAG_GU_FP8
    pf = oracle.forward(prev.x, prev.W1, prev.W2, prev.W3, flags=ofl)
    pb = oracle.backward(pf, prev.dY)
    given = dict(x=pf["sx"], w12=pf["sw12"], w3=pf["sw3"], h=pf["s_h"], dy=pb["sdy"], dz=pb["sdz"], gu=pf["sgu"])
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=ofl, scale_mode=oracle.SCALE_GIVEN, sx=pf["sx"],
                        sw12=pf["sw12"], s_h=pf["s_h"], sw3=pf["sw3"], sgu=pf["sgu"])
    bw = oracle.backward(fw, w.dY, scale_mode=oracle.SCALE_GIVEN, sdy=pb["sdy"], sdz=pb["sdz"], want_intermediates=True)
    r = _run(w, B.SMOOTH, B.SCALE_GIVEN, given=given)
    _check(r, fw, bw, given_scales=True)


def test_gu_fp8_update_scales_and_workspace_size():
    """fp8mlp_update_scales turns amax.gu into 448 / amax; the saved-activation workspace is half as large."""
    f = 64
    a = B.fp8mlp_create(32, 64, f, B.SMOOTH | B.SAVE_FOR_BWD)
    b = B.fp8mlp_create(32, 64, f, B.SMOOTH | B.SAVE_FOR_BWD | B.GU_FP8)
    try:
        assert B.fp8mlp_workspace(a, B.WS_GU)[1] == 2 * B.fp8mlp_workspace(b, B.WS_GU)[1] == 32 * 2 * f * 2
        sc, am = B.new_scales(f), B.new_amax(f)
        am["gu"].fill_(3.5)
        B.fp8mlp_update_scales(b, am, sc)
        torch.cuda.synchronize()
        assert sc["gu"].item() == np.float32(oracle.scale_from_amax(oracle.E4M3, 3.5))
        sc["gu"].fill_(1.0)
        B.fp8mlp_update_scales(a, am, sc)          # a context without the flag leaves it alone
        torch.cuda.synchronize()
        assert sc["gu"].item() == 1.0
    finally:
        B.fp8mlp_destroy(a)
        B.fp8mlp_destroy(b)


def test_gu_fp8_flag_combinations():
    L = B.lib()
    h = C.c_void_p()
    assert L.fp8mlp_create(C.byref(h), 16, 16, 16, B.GU_FP8) == B.ERR_ARG                       # nothing is saved
    assert L.fp8mlp_create(C.byref(h), 16, 16, 16, B.GU_FP8 | B.SAVE_FOR_BWD | B.H_BF16) == B.ERR_ARG


def test_gu_fp8_empty_batch_and_missing_scale():
    f = 64
    w = wl.make("e", 2, 16, 64, f, w_std=0.05)
    ctx = B.fp8mlp_create(16, 64, f, B.SMOOTH | B.SAVE_FOR_BWD | B.GU_FP8)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        am["gu"].fill_(9.0)
        B.fp8mlp_forward(ctx, 0, None, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, None)
        g = [torch.full((64, 64), 7.0, device="cuda") for _ in range(3)]
        B.fp8mlp_backward(ctx, 0, None, B.SCALE_FROM_CURRENT_AMAX, sc, am, None, g[0], g[1], g[2])
        torch.cuda.synchronize()
        assert am["gu"].item() == 0 and sc["gu"].item() == 1.0      # no tokens: maximum 0, scale falls back to 1
        assert all(float(t.abs().max()) == 0 for t in g)
        # a scales struct without the member is refused before anything is launched
        sc_missing = dict(sc, gu=None)
        y = torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(B.Fp8MlpError) as ei:
            B.fp8mlp_forward(ctx, 16, to_dev_bf16(w.x), W1, W2, W3, B.SCALE_GIVEN, sc_missing, am, y)
        assert ei.value.code == B.ERR_ARG
        assert B.fp8mlp_status(ctx) == B.OK
    finally:
        B.fp8mlp_destroy(ctx)
