"""Parity of the inference form of Smooth-SwiGLU (end of Section 4.4: s_i folded into the weights,
w1~_i = Q(s_i w1_i), w3~_i = Q(s_i^-1 w3_i)) with the CPU oracle.  On the oracle's side the merged
block is what the paper says it is: the ordinary quantised SwiGLU MLP (one per-tensor scale for the
SwiGLU output) run on the merged master weights."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_dev_to_bits, bf16_bits_to_f32, code_mismatch, nmax_err, to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _merged_masters(w, s):
    s = s.astype(np.float32)
    W1m = (w.W1 * s[None, :]).astype(np.float32)
    W3m = (w.W3 * (np.float32(1.0) / s)[:, None]).astype(np.float32)
    return W1m, W3m


def _check(w, s, mode, given=None):
    W1m, W3m = _merged_masters(w, s)
    kw = {} if given is None else dict(scale_mode=oracle.SCALE_GIVEN, **given)
    fw = oracle.forward(w.x, W1m, w.W2, W3m, flags=0, **kw)
    T, d, f = w.T, w.d, w.f
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(B.Fp8MlpError) as ei:                       # nothing merged yet
            B.fp8mlp_forward_merged(ctx, T, to_dev_bf16(w.x), mode, sc, am, y)
        assert ei.value.code == B.ERR_STATE
        if given is not None:
            for k, name in (("x", "sx"), ("w12", "sw12"), ("w3", "sw3")):
                sc[k].fill_(float(given[name]))
            sc["h"].copy_(to_dev(given["s_h"]))
        B.fp8mlp_merge_weights(ctx, to_dev(w.W1), to_dev(w.W2), to_dev(w.W3), to_dev(s.astype(np.float32)), mode, sc, am)
        B.fp8mlp_forward_merged(ctx, T, to_dev_bf16(w.x), mode, sc, am, y)
        assert B.fp8mlp_status(ctx) == B.OK
        ws = lambda which, shape: B.workspace_tensor(ctx, which, shape, torch.uint8).cpu().numpy()
        assert np.array_equal(ws(B.WS_XQ, (T, d)), fw["Xq"]), "x codes"
        assert np.array_equal(ws(B.WS_W12Q, (d, 2 * f)), fw["W12q"]), "[W2 | W1 diag(s)] codes"
        assert np.array_equal(ws(B.WS_W3Q, (f, d)), fw["W3q"]), "diag(1/s) W3 codes"
        assert am["w1"].item() == np.float32(fw["amax_w1"]) and am["w3"].item() == np.float32(fw["amax_w3"])
        assert sc["w12"].item() == np.float32(fw["sw12"]) and sc["w3"].item() == np.float32(fw["sw3"])
        assert np.allclose(am["h"].cpu().numpy(), fw["amax_h"], rtol=1e-5, atol=0)
        assert np.allclose(sc["h"].cpu().numpy(), fw["s_h"], rtol=1e-5, atol=0)
        frac, worst = code_mismatch(ws(B.WS_HQ, (T, f)), fw["Hq"])
        assert worst <= 1 and frac <= 1e-3, f"Hq codes: {frac:.2e} differ, worst {worst}"
        e = nmax_err(bf16_bits_to_f32(bf16_dev_to_bits(y)), fw["Y"])
        assert e <= 2e-3, f"Y: {e}"
        # given scales, maxima not asked for: same output
        y2 = torch.zeros_like(y)
        B.fp8mlp_forward_merged(ctx, T, to_dev_bf16(w.x), B.SCALE_GIVEN, sc, None, y2)
        assert torch.equal(y2.view(torch.int16), y.view(torch.int16))
        # a training forward replaces the merged weights
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3), B.SCALE_FROM_CURRENT_AMAX,
                         B.new_scales(f), B.new_amax(f), y2)
        with pytest.raises(B.Fp8MlpError):
            B.fp8mlp_forward_merged(ctx, T, to_dev_bf16(w.x), B.SCALE_GIVEN, sc, None, y2)
    finally:
        B.fp8mlp_destroy(ctx)
    return fw


def test_merged_tiny_config_scales_from_smooth_training_run():
    w = wl.make_config("tiny")
    s = oracle.forward(w.x, w.W1, w.W2, w.W3)["s_h"]                   # the s_i a Smooth-SwiGLU training step derived
    _check(w, s, B.SCALE_FROM_CURRENT_AMAX)


@pytest.mark.parametrize("shape", [(200, 320, 272), (333, 512, 1040)])
def test_merged_ragged_shapes_arbitrary_s_given_scales(shape):
    T, d, f = shape
    w = wl.make("m", 21, T, d, f, w_std=0.05, channel_outlier_frac=0.01)
    s = np.exp(np.random.default_rng(5).normal(0, 1.5, f)).astype(np.float32)      # not powers of two
    W1m, W3m = _merged_masters(w, s)
    prev = wl.make("mp", 22, T, d, f, w_std=0.05)
    pf = oracle.forward(prev.x, W1m, w.W2, W3m, flags=0)               # scales of a previous batch
    _check(w, s, B.SCALE_GIVEN, given=dict(sx=pf["sx"], sw12=pf["sw12"], s_h=pf["s_h"], sw3=pf["sw3"]))
