"""Parity of fp8mlp_forward / fp8mlp_backward with the CPU oracle, element by element.

Bars (from the benchmark definition): quantised inputs and amax bit-exact; SwiGLU codes at most
1 code step apart on at most 0.1 % of elements (fp32 accumulation order and the exponential
differ); Y, dX, dW within 2e-3 of the oracle's max |value|.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import (bf16_dev_to_bits, bf16_bits_to_f32, bf16_ulp, check_amax_dz, check_dz_codes, code_diff, code_mismatch, nmax_err,
                     nmax_err_bf16, record_parity, to_dev, to_dev_bf16)
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu

CODE_FRAC = 1e-3
OUT_TOL = 2e-3
AMAX_RTOL = 1e-5


class Run:
    """One forward(+backward) through the C ABI with everything the oracle can be compared on."""

    def __init__(self, w, flags, mode, given=None, backward=True):
        T, d, f = w.T, w.d, w.f
        self.w = w
        self.smooth = bool(flags & B.SMOOTH)
        self.ctx = B.fp8mlp_create(max(T, 1), d, f, flags)
        self.sc, self.am = B.new_scales(f), B.new_amax(f)
        if given is not None:
            for k, v in given.items():
                self.sc[k].copy_(to_dev(np.atleast_1d(np.asarray(v, np.float32))))
        x = to_dev_bf16(w.x)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        B.fp8mlp_forward(self.ctx, T, x, W1, W2, W3, mode, self.sc, self.am, y)
        self.Y_bits = bf16_dev_to_bits(y)
        ws = lambda which, shape, dt=torch.uint8: B.workspace_tensor(self.ctx, which, shape, dt).cpu().numpy()
        self.Xq, self.W12q = ws(B.WS_XQ, (T, d)), ws(B.WS_W12Q, (d, 2 * f))
        self.W3q, self.Hq = ws(B.WS_W3Q, (f, d)), ws(B.WS_HQ, (T, f))
        if flags & B.SAVE_FOR_BWD:
            self.GU = B.workspace_tensor(self.ctx, B.WS_GU, (T, 2 * f), torch.int16).cpu().numpy().view(np.uint16)
        if backward:
            dy = to_dev_bf16(w.dY)
            dx = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
            self.dW1 = torch.full((d, f), float("nan"), device="cuda")
            self.dW2 = torch.full((d, f), float("nan"), device="cuda")
            self.dW3 = torch.full((f, d), float("nan"), device="cuda")
            B.fp8mlp_backward(self.ctx, T, dy, mode, self.sc, self.am, dx, self.dW1, self.dW2, self.dW3)
            self.dX_bits = bf16_dev_to_bits(dx)
            self.dYq, self.dZq = ws(B.WS_DYQ, (T, d)), ws(B.WS_DZQ, (T, 2 * f))
        assert B.fp8mlp_status(self.ctx) == B.OK
        self.scales = {k: v.cpu().numpy() for k, v in self.sc.items()}
        self.amax = {k: v.cpu().numpy() for k, v in self.am.items()}

    def close(self):
        B.fp8mlp_destroy(self.ctx)


def check_forward(r: Run, fw: dict, save=True):
    f = r.w.f
    assert r.scales["x"][0] == np.float32(fw["sx"]) and r.scales["w12"][0] == np.float32(fw["sw12"])
    assert r.amax["x"][0] == np.float32(fw["amax_x"])
    assert r.amax["w1"][0] == np.float32(fw["amax_w1"]) and r.amax["w2"][0] == np.float32(fw["amax_w2"])
    assert np.array_equal(r.Xq, fw["Xq"]), "x codes differ"
    assert np.array_equal(r.W12q, fw["W12q"]), "[W2|W1] codes differ"
    assert np.allclose(r.amax["h"], fw["amax_h"], rtol=AMAX_RTOL, atol=0), "per-channel amax of H"
    if r.smooth:
        assert np.array_equal(r.scales["h"], fw["s_h"]), "per-channel scales s_i"
    else:   # 448 / max amax_h inherits the last-bit difference of amax_h (accumulation order)
        assert np.allclose(r.scales["h"], fw["s_h"], rtol=AMAX_RTOL, atol=0), "per-tensor scale of H"
    assert r.amax["w3"][0] == np.float32(fw["amax_w3"]) and r.scales["w3"][0] == np.float32(fw["sw3"])
    assert np.array_equal(r.W3q, fw["W3q"]), "W3' codes differ"
    frac, worst = code_mismatch(r.Hq, fw["Hq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"Hq codes: {frac:.2e} differ, worst {worst} steps"
    if save:
        # element by element: the two fp32 values differ in accumulation order only, so their bf16 roundings are
        # equal or, across a rounding boundary, one spacing apart
        for name, got, ref in (("G", r.GU[:, :f], fw["G"]), ("U", r.GU[:, f:], fw["U"])):
            e = nmax_err_bf16(got, bf16_bits_to_f32(ref))
            assert e <= 1e-5, f"saved {name}: {e} beyond one bf16 spacing"
    # Y is contracted from the Hq codes: the few allowed one-step differences (a step is 6-12 % of that element) are
    # carried through the oracle's own W3' codes and set aside; zero when the codes agree, so no excuse for the GEMM
    dh = code_diff(oracle.E4M3, r.Hq, fw["Hq"])
    dq2 = (np.float32(1.0) / np.float32(fw["sw3"])) * (np.float32(1.0) if r.smooth else np.float32(1.0) / fw["s_h"][0])
    y_ref = fw["Y"] + (dh @ oracle.decode(oracle.E4M3, fw["W3q"]).astype(np.float64)) * float(dq2) if np.any(dh) else fw["Y"]
    e = nmax_err(bf16_bits_to_f32(r.Y_bits), y_ref)
    assert e <= OUT_TOL, f"Y: {e}"


def check_backward(r: Run, fw: dict, bw: dict, many_codes: bool = False):
    assert r.amax["dy"][0] == np.float32(bw["amax_dy"]) and r.scales["dy"][0] == np.float32(bw["sdy"])
    assert np.array_equal(r.dYq, bw["dYq"]), "dY codes differ"
    # the accumulation-order bar, opened by one bf16 spacing only at the elements whose saved G or U does differ
    # from the oracle's (those have passed their own bar: at most one spacing)
    f = r.w.f
    g, u = bf16_bits_to_f32(fw["G"]), bf16_bits_to_f32(fw["U"])
    g_step = np.where(r.GU[:, :f] != fw["G"], bf16_ulp(g), 0.0)
    u_step = np.where(r.GU[:, f:] != fw["U"], bf16_ulp(u), 0.0)
    record_parity("amax_dz " + r.w.name, saved_activations_differing=int(np.count_nonzero(g_step) + np.count_nonzero(u_step)),
                  **check_amax_dz("amax of dZ", r.amax["dz"][0], bw, g, u, g_step, u_step, AMAX_RTOL))
    assert r.scales["dz"][0] == np.float32(bw["sdz"]), "scale of dZ"
    if many_codes:      # among hundreds of thousands of codes a few sit at the zero of the gate derivative
        check_dz_codes("dZq", r.dZq, bw["dZq"], CODE_FRAC, OUT_TOL)
    else:
        frac, worst = code_mismatch(r.dZq, bw["dZq"])
        assert worst <= 1 and frac <= CODE_FRAC, f"dZq codes: {frac:.2e} differ, worst {worst} steps"
    # Outputs contracted from codes that may differ by a step on a few elements (dX, dW1, dW2 from dZq; dW3 from Hq):
    # with few tokens one such step is visible in a weight-gradient column.  That part is computed from the code
    # differences and the oracle's other operand and set aside (zero where the codes agree); the rest meets the bar.
    inv = lambda v: np.float64(np.float32(1.0) / np.float32(v))
    dz = code_diff(oracle.E5M2, r.dZq, bw["dZq"])
    dh = code_diff(oracle.E4M3, r.Hq, fw["Hq"])
    shift = dict(dX=0.0, dW1=0.0, dW2=0.0, dW3=0.0)
    if np.any(dz):
        xq = oracle.decode(oracle.E4M3, fw["Xq"]).astype(np.float64)
        shift["dX"] = (dz @ oracle.decode(oracle.E4M3, fw["W12q"]).astype(np.float64).T) * inv(bw["sdz"]) * inv(fw["sw12"])
        shift["dW2"] = (xq.T @ dz[:, :f]) * inv(fw["sx"]) * inv(bw["sdz"])
        shift["dW1"] = (xq.T @ dz[:, f:]) * inv(fw["sx"]) * inv(bw["sdz"])
    if np.any(dh):
        dyq = oracle.decode(oracle.E5M2, bw["dYq"]).astype(np.float64)
        shift["dW3"] = (dh.T @ dyq) * inv(bw["sdy"]) * (1.0 / fw["s_h"].astype(np.float64))[:, None]
    for name, got, ref in (("dX", bf16_bits_to_f32(r.dX_bits), bw["dX"]), ("dW1", r.dW1.cpu().numpy(), bw["dW1"]),
                           ("dW2", r.dW2.cpu().numpy(), bw["dW2"]), ("dW3", r.dW3.cpu().numpy(), bw["dW3"])):
        assert np.all(np.isfinite(got)), f"{name} has unwritten or non-finite entries"
        e = nmax_err(got, ref + shift[name])
        assert e <= OUT_TOL, f"{name}: {e} (literal {nmax_err(got, ref)})"


def _oracle_flags(flags):
    return oracle.FLAG_SMOOTH if flags & B.SMOOTH else 0


@pytest.mark.parametrize("flags", [B.SMOOTH | B.SAVE_FOR_BWD, B.SAVE_FOR_BWD])
def test_tiny_config_current_amax(flags):
    """The tiny benchmark configuration (T=128, d=256, f=704: 5.5 channel tiles), scales from the
    current amax, Smooth-SwiGLU on and off."""
    w = wl.make_config("tiny")
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=_oracle_flags(flags))
    bw = oracle.backward(fw, w.dY, want_intermediates=True)
    r = Run(w, flags, B.SCALE_FROM_CURRENT_AMAX)
    try:
        check_forward(r, fw)
        check_backward(r, fw, bw)
    finally:
        r.close()


@pytest.mark.parametrize("shape", [(200, 320, 272), (1, 16, 16), (130, 144, 528), (333, 512, 1040), (300, 512, 2304),
                                   (2048, 256, 272)])
def test_ragged_shapes_given_scales(shape):
    """Several tiles with ragged tails in every dimension, delayed-scaling mode: scales come from an
    oracle run on other data (a previous step), so values also saturate and underflow.  The last shapes have
    few output tiles and long contractions, so their GEMMs split the contraction over several CTA pairs:
    (333, 512, 1040) the input-gradient GEMM in two; (300, 512, 2304) the down projection in two and the
    input-gradient GEMM in four; (2048, 256, 272) both weight-gradient GEMMs (fp32 outputs, one with a per-row
    divisor, one with its columns split over two outputs at a column that is no multiple of 32)."""
    T, d, f = shape
    w = wl.make("r", 11, T, d, f, w_std=0.05, channel_outlier_frac=0.01, token_outlier_frac=0.02)
    prev = wl.make("p", 12, T, d, f, w_std=0.05)
    pf = oracle.forward(prev.x, w.W1, w.W2, w.W3)
    pb = oracle.backward(pf, prev.dY)
    given = dict(x=pf["sx"], w12=pf["sw12"], w3=pf["sw3"], h=pf["s_h"], dy=pb["sdy"], dz=pb["sdz"])
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, scale_mode=oracle.SCALE_GIVEN, sx=pf["sx"], sw12=pf["sw12"],
                        s_h=pf["s_h"], sw3=pf["sw3"])
    bw = oracle.backward(fw, w.dY, scale_mode=oracle.SCALE_GIVEN, sdy=pb["sdy"], sdz=pb["sdz"], want_intermediates=True)
    r = Run(w, B.SMOOTH | B.SAVE_FOR_BWD, B.SCALE_GIVEN, given=given)
    try:
        for k, v in given.items():                       # given scales are left alone
            assert np.array_equal(r.scales[k], np.atleast_1d(np.asarray(v, np.float32)))
        check_forward(r, fw)
        check_backward(r, fw, bw)
    finally:
        r.close()


def test_ragged_shape_on_wide_tiles():
    """The down projection and the input-gradient GEMM switch to 256 x 512 tiles once those fill the CTA pairs
    (at least half as many tiles as SMs).  T = 2520 and d = 4048 give 10 x 8 such tiles with a ragged last row
    of tiles (216 of 256 tokens) and a ragged last column of tiles (464 of 512 outputs); f stays small so that
    the oracle finishes in seconds."""
    T, d, f = 2520, 4048, 144
    w = wl.make("wide", 21, T, d, f, w_std=0.05, channel_outlier_frac=0.01)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    bw = oracle.backward(fw, w.dY, want_intermediates=True)
    r = Run(w, B.SMOOTH | B.SAVE_FOR_BWD, B.SCALE_FROM_CURRENT_AMAX)
    try:
        check_forward(r, fw)
        check_backward(r, fw, bw, many_codes=True)
    finally:
        r.close()


def test_forward_only_context_and_state_errors():
    w = wl.make("s", 2, 64, 128, 256, w_std=0.05)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    r = Run(w, B.SMOOTH, B.SCALE_FROM_CURRENT_AMAX, backward=False)
    try:
        check_forward(r, fw, save=False)
        dx = torch.zeros((w.T, w.d), dtype=torch.bfloat16, device="cuda")
        g = torch.zeros((w.d, w.f), device="cuda")
        g3 = torch.zeros((w.f, w.d), device="cuda")
        with pytest.raises(B.Fp8MlpError) as ei:
            B.fp8mlp_backward(r.ctx, w.T, to_dev_bf16(w.dY), B.SCALE_GIVEN, r.sc, r.am, dx, g, g, g3)
        assert ei.value.code == B.ERR_STATE
        with pytest.raises(B.Fp8MlpError) as ei:
            B.fp8mlp_forward(r.ctx, w.T + 1, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3),
                             B.SCALE_GIVEN, r.sc, r.am, dx)
        assert ei.value.code == B.ERR_SHAPE
    finally:
        r.close()


def test_empty_batch():
    w = wl.make("e", 2, 16, 64, 64, w_std=0.05)
    ctx = B.fp8mlp_create(16, 64, 64, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(64), B.new_amax(64)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        B.fp8mlp_forward(ctx, 0, None, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, None)
        g1, g2, g3 = (torch.full((64, 64), 7.0, device="cuda") for _ in range(3))
        B.fp8mlp_backward(ctx, 0, None, B.SCALE_FROM_CURRENT_AMAX, sc, am, None, g1, g2, g3)
        torch.cuda.synchronize()
        assert float(g1.abs().max()) == 0 and float(g2.abs().max()) == 0 and float(g3.abs().max()) == 0
        assert am["x"].item() == 0 and float(am["h"].max()) == 0
        assert am["w1"].item() == oracle.amax(w.W1)
    finally:
        B.fp8mlp_destroy(ctx)


def test_step_can_be_captured_in_a_cuda_graph_and_replays_bit_identically():
    """Every call only enqueues kernels on the caller's stream (tensor maps travel as kernel
    parameters, nothing allocates after fp8mlp_create), so once each kernel has run once outside a
    capture the whole delayed-scaling step can be captured and replayed."""
    w = wl.make_config("tiny")
    T, d, f = w.T, w.d, w.f
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        x, dy = to_dev_bf16(w.x), to_dev_bf16(w.dY)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros_like(y)
        dW1, dW2, dW3 = torch.zeros_like(W1), torch.zeros_like(W2), torch.zeros_like(W3)

        def step(mode):
            B.fp8mlp_forward(ctx, T, x, W1, W2, W3, mode, sc, am, y)
            B.fp8mlp_backward(ctx, T, dy, mode, sc, am, dx, dW1, dW2, dW3)

        step(B.SCALE_FROM_CURRENT_AMAX)
        step(B.SCALE_GIVEN)
        torch.cuda.synchronize()
        ref = [t.clone() for t in (y, dx, dW1, dW2, dW3)]
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                step(B.SCALE_GIVEN)
        for t in (y, dx, dW1, dW2, dW3):
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert B.fp8mlp_status(ctx) == B.OK
        for got, want in zip((y, dx, dW1, dW2, dW3), ref):
            assert torch.equal(got.view(torch.int32) if got.dtype == torch.float32 else got.view(torch.int16),
                               want.view(torch.int32) if want.dtype == torch.float32 else want.view(torch.int16))
    finally:
        B.fp8mlp_destroy(ctx)


def test_empty_inputs_of_the_other_entry_points():
    """T = 0 and n = 0 are legal everywhere: nothing is launched on data, maxima read zero."""
    ctx = B.fp8mlp_create(16, 64, 64, B.SMOOTH)
    hb = B.fp8mlp_create(16, 64, 64, B.H_BF16 | B.SAVE_FOR_BWD)
    try:
        w = wl.make("e2", 3, 16, 64, 64, w_std=0.05)
        sc, am = B.new_scales(64), B.new_amax(64)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        s = torch.ones(64, device="cuda")
        B.fp8mlp_merge_weights(ctx, W1, W2, W3, s, B.SCALE_FROM_CURRENT_AMAX, sc, am)
        B.fp8mlp_forward_merged(ctx, 0, None, B.SCALE_GIVEN, sc, None, None)
        B.fp8mlp_forward(hb, 0, None, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, None)
        g = [torch.full((64, 64), 3.0, device="cuda") for _ in range(3)]
        B.fp8mlp_backward(hb, 0, None, B.SCALE_FROM_CURRENT_AMAX, sc, am, None, g[0], g[1], g[2])
        one = lambda: torch.ones(1, device="cuda")
        empty = dict(w=torch.empty(0, device="cuda"), g=torch.empty(0, device="cuda"),
                     m=torch.empty(0, dtype=torch.uint8, device="cuda"), v=torch.empty(0, dtype=torch.uint8, device="cuda"),
                     scale_m_in=one(), scale_v_in=one(), scale_m_out=one(), scale_v_out=one(),
                     amax_m=torch.full((1,), 5.0, device="cuda"), amax_v=torch.full((1,), 5.0, device="cuda"))
        B.fp8mlp_adam_step([empty], lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.0, step=1)
        torch.cuda.synchronize()
        assert all(float(t.abs().max()) == 0 for t in g)
        assert empty["amax_m"].item() == 0 and empty["amax_v"].item() == 0
        assert B.fp8mlp_status(ctx) == B.OK and B.fp8mlp_status(hb) == B.OK
    finally:
        B.fp8mlp_destroy(ctx)
        B.fp8mlp_destroy(hb)


def test_split_contraction_gives_the_same_bits_every_time():
    """GEMMs with few tiles split their contraction over several CTA pairs and the share that finishes last
    adds the partial sums - always in the order of the shares, so which one is last must not show in the result."""
    T, d, f = 300, 512, 2304
    w = wl.make("det", 23, T, d, f, w_std=0.05)
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        x, dy = to_dev_bf16(w.x), to_dev_bf16(w.dY)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros_like(y)
        dW1, dW2, dW3 = torch.zeros_like(W1), torch.zeros_like(W2), torch.zeros_like(W3)
        B.fp8mlp_forward(ctx, T, x, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        B.fp8mlp_backward(ctx, T, dy, B.SCALE_FROM_CURRENT_AMAX, sc, am, dx, dW1, dW2, dW3)
        first = None
        for _ in range(6):
            B.fp8mlp_forward(ctx, T, x, W1, W2, W3, B.SCALE_GIVEN, sc, am, y)
            B.fp8mlp_backward(ctx, T, dy, B.SCALE_GIVEN, sc, am, dx, dW1, dW2, dW3)
            torch.cuda.synchronize()
            got = [t.view(torch.int16).clone() for t in (y, dx)] + [t.view(torch.int32).clone() for t in (dW1, dW2, dW3)]
            if first is None:
                first = got
            else:
                assert all(torch.equal(a, b) for a, b in zip(got, first))
        assert B.fp8mlp_status(ctx) == B.OK
    finally:
        B.fp8mlp_destroy(ctx)
