"""Parity at the benchmark's full sizes, in the launch configuration bench.py times
(Smooth-SwiGLU on, activations saved, delayed scaling: scales given, maxima emitted).

The whole oracle would take hours at these sizes, so the comparison is on sampled outputs the
oracle computes in full, each with its complete contraction:
  - everything that is one pass over a tensor (the quantised x, [W2|W1], W3', dY and their maxima)
    is compared in full, bit for bit;
  - a sample of tokens gives whole rows of Hq, G, U, Y, dZq and dX (a token's outputs depend on no
    other token once the scales are given);
  - a sample of channels - every outlier channel among them - gives whole columns of Hq and dZq,
    the per-channel maxima, rows of dW3 and columns of dW1, dW2 (a channel's outputs depend on no
    other channel once the scales are given).
That a token / channel sub-problem reproduces the rows / columns of the full run is pinned on the
CPU in test_oracle_pins.py.  The given scales come from an oracle run on a small batch drawn with
another seed (the "previous iteration" of delayed scaling), never from the CUDA path.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import (bf16_bits_to_f32, bf16_ulp, check_amax_dz, check_dz_codes as _check_dz_codes, code_mismatch, code_rank,
                     frac_beyond, nmax_err, nmax_err_bf16, record_parity, to_dev, to_dev_bf16)
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu

CODE_FRAC = 1e-3
OUT_TOL = 2e-3
AMAX_RTOL = 1e-5


def _previous_iteration_scales(w, n_tokens, smooth=True):
    """Scales a delayed-scaling run would hold: from the oracle on a small batch of another seed,
    with two binades of headroom for the activations (the maxima of a few tokens underestimate those
    of thousands)."""
    cfg = dict(wl.CONFIGS[w.name])
    cfg.update(seed=cfg["seed"] + 100, T=n_tokens)
    prev = wl.make("prev", **cfg)
    pf = oracle.forward(prev.x, w.W1, w.W2, w.W3, flags=oracle.FLAG_SMOOTH if smooth else 0)
    pb = oracle.backward(pf, prev.dY)
    s_h = (pf["s_h"] * np.float32(0.25)).astype(np.float32)     # Smooth off: one per-tensor scale, repeated
    inv = (np.float32(1.0) / s_h).astype(np.float32)
    sw3 = oracle.scale_from_amax(oracle.E4M3, oracle.amax(w.W3, inv if smooth else None))
    return dict(x=np.float32(pf["sx"] * 0.5), w12=np.float32(pf["sw12"]), w3=np.float32(sw3), h=s_h,
                dy=np.float32(pb["sdy"] * 0.5), dz=np.float32(pb["sdz"] * 0.25))


BF16_ALLOWANCE_FRAC = 1e-3      # how many elements may need the one-spacing allowance (measured: about 1e-4)
LITERAL_CEILING = 2.0 ** -6     # literal max error of a bf16 output: two bf16 spacings at the tensor's maximum


def _check_bf16_rows(name, got_bits, ref, shift=0.0):
    """Y and dX are bf16 roundings of fp32 results.  Where the two fp32 values straddle a rounding
    boundary the bf16 values are one spacing apart, which on an element above a quarter of the
    maximum is already more than 2e-3 of it: the bar is applied net of that one spacing, and the
    elements that need the allowance must be few.  `shift` is the part explained by operand-code
    differences (see _explained).  The literal error, with no allowance at all, is recorded and held
    to a ceiling of its own so that nothing can hide inside the allowances."""
    target = ref + shift
    e = nmax_err_bf16(got_bits, target)
    assert e <= OUT_TOL, f"{name} rows: {e}"
    got = bf16_bits_to_f32(got_bits)
    fr = frac_beyond(got, target, OUT_TOL)
    assert fr <= BF16_ALLOWANCE_FRAC, f"{name} rows: {fr:.2e} of the elements are a bf16 spacing off"
    literal = nmax_err(got, ref)
    shift_rel = float(np.abs(shift).max() / np.abs(ref).max()) if np.ndim(shift) else 0.0
    assert literal <= LITERAL_CEILING + shift_rel, f"{name} rows: literal error {literal}"
    return dict(net_of_allowances=e, frac_needing_bf16_spacing=fr, literal=literal, explained_shift=shift_rel)


def _explained(code_fmt, got_codes, ref_codes, operand_codes, operand_is_kn, dq):
    """What the few operand-code differences that passed their own bar do to the next GEMM's output:
    sum_i (dec(got[t,i]) - dec(ref[t,i])) * dec(B[i,.]) * dq, from the oracle's other operand.  Zero
    wherever the codes agree, so a wrong GEMM is not excused by it.  Returns (shift, figures); the
    figures say how many output rows it touches (never more than there are differing codes) and bound
    its size: one code step is at most a quarter of the element, so a row with n differing codes moves
    by at most n/4 of the largest single product of the contraction."""
    dec_got = oracle.decode(code_fmt, got_codes).astype(np.float64)
    dec_ref = oracle.decode(code_fmt, ref_codes).astype(np.float64)
    diff = dec_got - dec_ref
    n_diff = int(np.count_nonzero(diff))
    rows_touched = int(np.count_nonzero(np.any(diff != 0, axis=1)))
    figures = dict(differing_codes=n_diff, rows_touched=rows_touched, rows=int(diff.shape[0]))
    idx = np.flatnonzero(np.any(diff != 0, axis=0))
    if idx.size == 0:
        return 0.0, figures
    assert rows_touched <= n_diff
    other = operand_codes[idx, :] if operand_is_kn else operand_codes[:, idx].T          # [len(idx), N]
    other = oracle.decode(oracle.E4M3, np.ascontiguousarray(other)).astype(np.float64)
    shift = (diff[:, idx] @ other) * float(dq)
    per_row = np.count_nonzero(diff, axis=1).max()
    bound = 0.25 * per_row * np.abs(dec_ref).max() * np.abs(other).max() * float(dq)
    assert np.abs(shift).max() <= bound, "the explained shift is larger than one code step per differing code allows"
    return shift, figures


def _sample(rng, n, count, always=()):
    picks = set(int(i) for i in always)
    picks.update({0, n - 1, 127, 128, n // 2})
    while len(picks) < count:
        picks.add(int(rng.integers(0, n)))
    return np.array(sorted(picks), dtype=np.int64)


@pytest.mark.parametrize("name,smooth,n_prev,n_tok,n_ch", [
    ("7b", True, 48, 32, 32), ("7b", False, 32, 32, 32), ("70b", True, 16, 32, 32),
    # the token sweep (1 % of the rows of x multiplied by 50; four of those rows are always in the sample); at
    # T = 512 the GEMMs have fewer tiles than the GPU has CTA pairs and take the small-problem path
    ("sweep_512", True, 32, 32, 32), ("sweep_2048", True, 32, 32, 32), ("sweep_8192", True, 32, 32, 32),
    ("sweep_32768", True, 32, 32, 32)])
def test_full_size_sampled_parity(name, smooth, n_prev, n_tok, n_ch):
    w = wl.make_config(name)
    T, d, f = w.T, w.d, w.f
    given = _previous_iteration_scales(w, n_prev, smooth)
    oflags = oracle.FLAG_SMOOTH if smooth else 0
    rng = np.random.default_rng(1234)
    toks = _sample(rng, T, n_tok, w.outlier_tokens[:4])
    chans = _sample(rng, f, n_ch, w.outlier_channels)

    # ---- CUDA path: one delayed-scaling step through the C ABI
    ctx = B.fp8mlp_create(T, d, f, (B.SMOOTH if smooth else 0) | B.SAVE_FOR_BWD)
    try:
        # every buffer the step writes starts as NaN codes (0x7F / 0xFF patterns): an element the kernels skipped shows
        for which in (B.WS_XQ, B.WS_W12Q, B.WS_W3Q, B.WS_HQ, B.WS_GU, B.WS_DYQ, B.WS_DZQ):
            B.workspace_fill(ctx, which, 0x7F)
        sc, am = B.new_scales(f), B.new_amax(f)
        for k, v in given.items():
            sc[k].copy_(to_dev(np.atleast_1d(np.asarray(v, np.float32))))
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dW1 = torch.full((d, f), float("nan"), device="cuda")
        dW2 = torch.full((d, f), float("nan"), device="cuda")
        dW3 = torch.full((f, d), float("nan"), device="cuda")
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), W1, W2, W3, B.SCALE_GIVEN, sc, am, y)
        B.fp8mlp_backward(ctx, T, to_dev_bf16(w.dY), B.SCALE_GIVEN, sc, am, dx, dW1, dW2, dW3)
        assert B.fp8mlp_status(ctx) == B.OK
        del W1, W2, W3
        ws = lambda which, shape, dt=torch.uint8: B.workspace_tensor(ctx, which, shape, dt)
        ti, ci = torch.from_numpy(toks).cuda(), torch.from_numpy(chans).cuda()
        ci2 = torch.cat([ci, ci + f])
        got = dict(Xq=ws(B.WS_XQ, (T, d)).cpu().numpy(), W12q=ws(B.WS_W12Q, (d, 2 * f)).cpu().numpy(),
                   W3q=ws(B.WS_W3Q, (f, d)).cpu().numpy(), dYq=ws(B.WS_DYQ, (T, d)).cpu().numpy())
        hq, dzq = ws(B.WS_HQ, (T, f)), ws(B.WS_DZQ, (T, 2 * f))
        gu = ws(B.WS_GU, (T, 2 * f), torch.int16)
        got["dZq_top"] = float((dzq & 0x7F).max().view(torch.float8_e5m2).float())      # largest |value| among the codes
        got.update(Hq_rows=hq[ti].cpu().numpy(), Hq_cols=hq[:, ci].cpu().numpy(),
                   dZq_rows=dzq[ti].cpu().numpy(), dZq_cols=dzq[:, ci2].cpu().numpy(),
                   GU_rows=gu[ti].cpu().numpy().view(np.uint16),
                   Y_rows=y[ti].view(torch.int16).cpu().numpy().view(np.uint16),
                   dX_rows=dx[ti].view(torch.int16).cpu().numpy().view(np.uint16),
                   dW1_cols=dW1[:, ci].cpu().numpy(), dW2_cols=dW2[:, ci].cpu().numpy(), dW3_rows=dW3[ci].cpu().numpy())
        assert bool(torch.isfinite(dW1).all()) and bool(torch.isfinite(dW2).all()) and bool(torch.isfinite(dW3).all())
        del hq, dzq, gu
        amax = {k: v.cpu().numpy() for k, v in am.items()}
        scales = {k: v.cpu().numpy() for k, v in sc.items()}
    finally:
        B.fp8mlp_destroy(ctx)
    for k, v in given.items():                               # given scales are left alone
        assert np.array_equal(scales[k], np.atleast_1d(np.asarray(v, np.float32)))

    # ---- one-pass tensors, in full, bit for bit
    x_f = wl.bf16_bits_to_f32(w.x)
    assert amax["x"][0] == np.float32(oracle.amax(x_f))
    assert np.array_equal(got["Xq"], oracle.quantize(x_f, oracle.E4M3, given["x"])[0]), "x codes"
    del x_f
    assert amax["w1"][0] == np.float32(oracle.amax(w.W1)) and amax["w2"][0] == np.float32(oracle.amax(w.W2))
    assert np.array_equal(got["W12q"][:, :f], oracle.quantize(w.W2, oracle.E4M3, given["w12"])[0]), "W2 codes"
    assert np.array_equal(got["W12q"][:, f:], oracle.quantize(w.W1, oracle.E4M3, given["w12"])[0]), "W1 codes"
    inv_s = (np.float32(1.0) / given["h"]).astype(np.float32)
    w3q, _, a_w3 = oracle.quantize(w.W3, oracle.E4M3, given["w3"], row_mul=inv_s if smooth else None)
    assert amax["w3"][0] == np.float32(a_w3) and np.array_equal(got["W3q"], w3q), "W3' codes"
    dy_f = wl.bf16_bits_to_f32(w.dY)
    assert amax["dy"][0] == np.float32(oracle.amax(dy_f))
    assert np.array_equal(got["dYq"], oracle.quantize(dy_f, oracle.E5M2, given["dy"])[0]), "dY codes"
    del dy_f

    # ---- sampled tokens: whole rows
    og = dict(scale_mode=oracle.SCALE_GIVEN, sx=float(given["x"]), sw12=float(given["w12"]), s_h=given["h"],
              sw3=float(given["w3"]))
    fw = oracle.forward(w.x[toks], w.W1, w.W2, w.W3, flags=oflags, **og)
    bw = oracle.backward(fw, w.dY[toks], scale_mode=oracle.SCALE_GIVEN, sdy=float(given["dy"]), sdz=float(given["dz"]),
                         want_intermediates=True)
    frac, worst = code_mismatch(got["Hq_rows"], fw["Hq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"Hq rows: {frac:.2e} differ, worst {worst}"
    for nm, g_bits, ref in (("G", got["GU_rows"][:, :f], fw["G"]), ("U", got["GU_rows"][:, f:], fw["U"])):
        assert nmax_err_bf16(g_bits, bf16_bits_to_f32(ref)) <= 1e-5, f"saved {nm}"
    # Y and dX inherit the (already checked, rare, one-step) differences of the Hq / dZq codes they are
    # contracted from; one step of an E4M3 / E5M2 code is 6-25 % of that element, which on a large element
    # moves the whole output row by more than the bar.  That part is computed from the code differences and
    # the oracle's other operand and set aside; the rest is held to the bar.
    inv = lambda v: np.float32(1.0) / np.float32(v)
    dq2 = inv(given["w3"]) if smooth else inv(given["w3"]) * inv(given["h"][0])
    y_shift, y_expl = _explained(oracle.E4M3, got["Hq_rows"], fw["Hq"], fw["W3q"], True, dq2)
    fig = dict(Hq_rows_frac=frac, Y=_check_bf16_rows("Y", got["Y_rows"], fw["Y"], y_shift), Y_explained=y_expl)
    _check_dz_codes("dZq rows", got["dZq_rows"], bw["dZq"])
    dz_rank = np.abs(code_rank(got["dZq_rows"]) - code_rank(bw["dZq"]))
    fig.update(dZq_rows_frac=float(np.mean(dz_rank > 0)), dZq_rows_frac_beyond_one_step=float(np.mean(dz_rank > 1)))
    dx_shift, dx_expl = _explained(oracle.E5M2, got["dZq_rows"], bw["dZq"], fw["W12q"], False, inv(given["dz"]) * inv(given["w12"]))
    fig.update(dX=_check_bf16_rows("dX", got["dX_rows"], bw["dX"], dx_shift), dX_explained=dx_expl)
    # The maximum of dZ is taken over all T tokens, the oracle's over the sample: it must reach the sample's
    # (within the envelope one bf16 spacing of the saved G, U opens, see helpers.amax_dz_bounds), and it must be
    # the value the largest stored code rounds from (an E5M2 step is a quarter of the value at most).
    g_ref, u_ref = bf16_bits_to_f32(fw["G"]), bf16_bits_to_f32(fw["U"])
    g_step = np.where(got["GU_rows"][:, :f] != fw["G"], bf16_ulp(g_ref), 0.0)       # only where the saved value differs
    u_step = np.where(got["GU_rows"][:, f:] != fw["U"], bf16_ulp(u_ref), 0.0)
    fig.update(saved_GU_differing_frac=float((np.count_nonzero(g_step) + np.count_nonzero(u_step)) / (2.0 * g_step.size)),
               amax_dz=check_amax_dz("amax of dZ", amax["dz"][0], bw, g_ref, u_ref, g_step, u_step, AMAX_RTOL, lower_only=True))
    scaled_top = min(float(amax["dz"][0]) * float(given["dz"]), 57344.0)         # the cast saturates there
    assert abs(got["dZq_top"] - scaled_top) <= 0.125 * scaled_top, "largest dZ code does not match the reported maximum"
    del fw, bw

    # ---- sampled channels: whole columns, per-channel maxima, weight-gradient slices
    ogc = dict(og, s_h=given["h"][chans])
    fwc = oracle.forward(w.x, w.W1[:, chans], w.W2[:, chans], w.W3[chans, :], flags=oflags, **ogc)
    bwc = oracle.backward(fwc, w.dY, scale_mode=oracle.SCALE_GIVEN, sdy=float(given["dy"]), sdz=float(given["dz"]))
    assert np.allclose(amax["h"][chans], fwc["amax_h"], rtol=AMAX_RTOL, atol=0), "per-channel maxima of H"
    frac, worst = code_mismatch(got["Hq_cols"], fwc["Hq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"Hq columns: {frac:.2e} differ, worst {worst}"
    _check_dz_codes("dZq columns", got["dZq_cols"], bwc["dZq"])
    fig.update(Hq_cols_frac=frac)
    for nm, g, ref in (("dW1", got["dW1_cols"], bwc["dW1"]), ("dW2", got["dW2_cols"], bwc["dW2"]),
                       ("dW3", got["dW3_rows"], bwc["dW3"])):
        e = nmax_err(g, ref)
        assert e <= OUT_TOL, f"{nm} slices: {e}"
        fig[nm] = e
    record_parity(f"full size {name} smooth={'on' if smooth else 'off'}", tokens=int(toks.size), channels=int(chans.size), **fig)


def test_7b_forward_smooth_on_versus_off_code_statistics():
    """The forward-only 7B configuration (T=4096, 0.1 % aligned outlier channels), scales from the
    current maxima, Smooth-SwiGLU on and off: properties of the SwiGLU codes that hold at any size.
    On: every channel's largest code sits in the top binade of E4M3 (the (224, 448] invariant of the
    power-of-two s_i), so no channel is crushed by the outliers.  Off: the one per-tensor scale is set
    by the outlier channels (about 100x typical), ordinary channels peak binades lower and several
    times more of their values flush to the zero code."""
    w = wl.make_config("7b_fwd")
    T, d, f = w.T, w.d, w.f
    x, W1, W2, W3 = to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
    toks = _sample(np.random.default_rng(5), T, 32)
    ti = torch.from_numpy(toks).cuda()
    stats = {}
    for smooth in (True, False):
        ctx = B.fp8mlp_create(T, d, f, B.SMOOTH if smooth else 0)
        try:
            sc, am = B.new_scales(f), B.new_amax(f)
            y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
            B.fp8mlp_forward(ctx, T, x, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
            assert B.fp8mlp_status(ctx) == B.OK
            hq = B.workspace_tensor(ctx, B.WS_HQ, (T, f), torch.uint8)
            mag = hq & 0x7F
            stats[smooth] = dict(chan_top=mag.max(dim=0).values.cpu().numpy(), zero_frac=float((mag == 0).float().mean()),
                                 top_frac=float((mag == 0x7E).float().mean()),
                                 amax_h=am["h"].cpu().numpy(), s_h=sc["h"].cpu().numpy(), y_finite=bool(torch.isfinite(y).all()),
                                 y_rows=bf16_bits_to_f32(y[ti].view(torch.int16).cpu().numpy().view(np.uint16)))
        finally:
            B.fp8mlp_destroy(ctx)
    on, off = stats[True], stats[False]
    assert on["y_finite"] and off["y_finite"]
    assert np.allclose(on["amax_h"], off["amax_h"], rtol=1e-5)            # same unscaled SwiGLU output both ways
    # on: s_i * amax_h[i] in (224, 448]  ->  top code between 0x76 (224) and 0x7E (448)
    prod = on["s_h"].astype(np.float64) * on["amax_h"]
    assert np.all((prod > 224.0) & (prod <= 448.0))
    assert on["chan_top"].min() >= 0x76 and on["chan_top"].max() <= 0x7E
    # off: the outlier channels own the range
    out_ch = w.outlier_channels
    assert off["chan_top"].max() == 0x7E and int(np.argmax(off["amax_h"])) in set(out_ch.tolist())
    typical = np.delete(off["chan_top"], out_ch)
    assert np.median(typical) <= 0x76 - 3 * 8                            # three binades or more below the top
    assert off["zero_frac"] > 3 * on["zero_frac"]
    # output error of 32 sampled tokens against the unquantised block in fp64 (the definition, no FP8 anywhere):
    # what the quantisation as a whole costs, with per-channel and with per-tensor scaling of the SwiGLU output
    _, y64 = oracle.mlp_f64(wl.bf16_bits_to_f32(w.x[toks]), w.W1, w.W2, w.W3)
    err = {}
    for key, st in (("on", on), ("off", off)):
        diff = st["y_rows"].astype(np.float64) - y64
        err[key] = dict(max_over_max=float(np.abs(diff).max() / np.abs(y64).max()),
                        rms_over_rms=float(np.sqrt(np.mean(diff ** 2) / np.mean(y64 ** 2))))
    # FP8 with 3 mantissa bits: a few percent either way.  (On one forward pass the two scalings are about equally
    # accurate in this sense - floating-point codes have the same relative spacing at any scale; what per-channel
    # scaling changes is which values underflow, asserted above.  Both figures are recorded.)
    assert err["on"]["rms_over_rms"] < 0.1 and err["off"]["rms_over_rms"] < 0.1
    record_parity("7b forward T=4096, Smooth-SwiGLU on versus off", tokens=int(toks.size),
                  on=dict(zero_code_frac=on["zero_frac"], largest_code_frac=on["top_frac"], Y_vs_fp64=err["on"]),
                  off=dict(zero_code_frac=off["zero_frac"], largest_code_frac=off["top_frac"], Y_vs_fp64=err["off"]))


def test_7b_forward_just_in_time_scales_sampled_channels():
    """The forward-only 7B configuration in the mode it is stated in (every scale from the current
    data, Smooth-SwiGLU on), at full size: the per-tensor scales of x and [W2|W1] against the
    oracle's maxima of the whole tensors, and for a sample of channels (all outlier channels among
    them) the per-channel maxima over all 4096 tokens, the s_i derived from them and the resulting
    code columns - a channel's maximum, scale and codes depend on no other channel."""
    w = wl.make_config("7b_fwd")
    T, d, f = w.T, w.d, w.f
    rng = np.random.default_rng(77)
    chans = _sample(rng, f, 40, w.outlier_channels)
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3), B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        assert B.fp8mlp_status(ctx) == B.OK
        ci = torch.from_numpy(chans).cuda()
        hq_cols = B.workspace_tensor(ctx, B.WS_HQ, (T, f), torch.uint8)[:, ci].cpu().numpy()
        scales = {k: v.cpu().numpy() for k, v in sc.items()}
        amax = {k: v.cpu().numpy() for k, v in am.items()}
    finally:
        B.fp8mlp_destroy(ctx)
    a_x = oracle.amax(wl.bf16_bits_to_f32(w.x))
    a_w = max(oracle.amax(w.W1), oracle.amax(w.W2))
    sx, sw12 = oracle.scale_from_amax(oracle.E4M3, a_x), oracle.scale_from_amax(oracle.E4M3, a_w)
    assert amax["x"][0] == np.float32(a_x) and scales["x"][0] == np.float32(sx) and scales["w12"][0] == np.float32(sw12)
    # the channel sub-problem with those two scales given: its per-channel maxima are the full run's
    probe = oracle.forward(w.x, w.W1[:, chans], w.W2[:, chans], w.W3[chans, :], scale_mode=oracle.SCALE_GIVEN,
                           sx=sx, sw12=sw12, s_h=np.ones(chans.size, np.float32), sw3=1.0)
    assert np.allclose(amax["h"][chans], probe["amax_h"], rtol=AMAX_RTOL, atol=0)
    s_ref = np.array([oracle.pow2_scale(oracle.E4M3, a) for a in probe["amax_h"]], np.float32)
    assert np.array_equal(scales["h"][chans], s_ref), "s_i of the sampled channels"
    fwc = oracle.forward(w.x, w.W1[:, chans], w.W2[:, chans], w.W3[chans, :], scale_mode=oracle.SCALE_GIVEN,
                         sx=sx, sw12=sw12, s_h=s_ref, sw3=1.0)
    frac, worst = code_mismatch(hq_cols, fwc["Hq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"Hq columns: {frac:.2e} differ, worst {worst}"


def test_7b_saved_activations_in_fp8_sampled_tokens():
    """FP8MLP_GU_FP8 at the benchmark's 7B size (delayed scaling): whole rows of the saved E4M3 codes of G, U and of
    what backward makes of them (dZq, dX), and the maximum of |G|, |U| against the sample's."""
    w = wl.make_config("7b")
    T, d, f = w.T, w.d, w.f
    given = _previous_iteration_scales(w, 32, True)
    cfg = dict(wl.CONFIGS[w.name]); cfg.update(seed=cfg["seed"] + 100, T=32)
    prev = wl.make("prev", **cfg)
    pf = oracle.forward(prev.x, w.W1, w.W2, w.W3, flags=oracle.FLAG_SMOOTH | oracle.FLAG_GU_FP8)
    given["gu"] = np.float32(pf["sgu"] * 0.25)
    rng = np.random.default_rng(4321)
    toks = _sample(rng, T, 32, w.outlier_tokens[:4])
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH | B.SAVE_FOR_BWD | B.GU_FP8)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        for k, v in given.items():
            sc[k].copy_(to_dev(np.atleast_1d(np.asarray(v, np.float32))))
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dW1, dW2, dW3 = torch.empty((d, f), device="cuda"), torch.empty((d, f), device="cuda"), torch.empty((f, d), device="cuda")
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), W1, W2, W3, B.SCALE_GIVEN, sc, am, y)
        B.fp8mlp_backward(ctx, T, to_dev_bf16(w.dY), B.SCALE_GIVEN, sc, am, dx, dW1, dW2, dW3)
        assert B.fp8mlp_status(ctx) == B.OK
        ti = torch.from_numpy(toks).cuda()
        gu_rows = B.workspace_tensor(ctx, B.WS_GU, (T, 2 * f), torch.uint8)[ti].cpu().numpy()
        dz_rows = B.workspace_tensor(ctx, B.WS_DZQ, (T, 2 * f), torch.uint8)[ti].cpu().numpy()
        dx_rows = dx[ti].view(torch.int16).cpu().numpy().view(np.uint16)
        a_gu, s_gu = am["gu"].item(), sc["gu"].item()
    finally:
        B.fp8mlp_destroy(ctx)
    assert s_gu == given["gu"]
    fw = oracle.forward(w.x[toks], w.W1, w.W2, w.W3, flags=oracle.FLAG_SMOOTH | oracle.FLAG_GU_FP8,
                        scale_mode=oracle.SCALE_GIVEN, sx=float(given["x"]), sw12=float(given["w12"]), s_h=given["h"],
                        sw3=float(given["w3"]), sgu=float(given["gu"]))
    bw = oracle.backward(fw, w.dY[toks], scale_mode=oracle.SCALE_GIVEN, sdy=float(given["dy"]), sdz=float(given["dz"]))
    assert a_gu >= 0.99999 * fw["amax_gu"]                   # the global maximum covers the sample's
    frac, worst = code_mismatch(gu_rows, fw["GUq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"saved G, U codes: {frac:.2e} differ, worst {worst}"
    _check_dz_codes("dZq rows", dz_rows, bw["dZq"])
    inv = lambda v: np.float32(1.0) / np.float32(v)
    dx_shift, _ = _explained(oracle.E5M2, dz_rows, bw["dZq"], fw["W12q"], False, inv(given["dz"]) * inv(given["w12"]))
    _check_bf16_rows("dX", dx_rows, bw["dX"], dx_shift)


def test_7b_just_in_time_forward_and_backward_sampled_tokens():
    """The benchmark's 7B step with every scale derived from the current data (the mode the paper calls
    just-in-time scaling, Section 2), forward and backward, at full size.

    The per-channel scales need the whole gate/up GEMM (hours on the CPU), so the check is a chain in which
    every scale the CUDA path derived is first tied to the oracle and only then handed to the oracle's
    sampled-token run as a given scale:
      - maxima of one-pass tensors (x, W1, W2, dY): the oracle's, bit for bit, and their scales the oracle's;
      - per-channel maxima of H and the s_i made from them: the oracle's on a sample of channels (all outlier
        channels among them), each over all T tokens; every s_i a power of two that puts its channel's maximum
        in (224, 448];
      - scale of W3': the oracle's scale routine on the oracle's maximum of diag(1/s) W3 for that s;
      - scale of dZ: the oracle's power-of-two routine on the reported maximum, which itself must reach the
        sampled tokens' maximum and match the largest stored code.
    Then whole rows of Hq, Y, dZq and dX for the sampled tokens against the oracle with those scales given."""
    w = wl.make_config("7b")
    T, d, f = w.T, w.d, w.f
    rng = np.random.default_rng(99)
    toks = _sample(rng, T, 32)
    chans = _sample(rng, f, 32, w.outlier_channels)
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        W1, W2, W3 = to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dW1, dW2, dW3 = torch.empty((d, f), device="cuda"), torch.empty((d, f), device="cuda"), torch.empty((f, d), device="cuda")
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        B.fp8mlp_backward(ctx, T, to_dev_bf16(w.dY), B.SCALE_FROM_CURRENT_AMAX, sc, am, dx, dW1, dW2, dW3)
        assert B.fp8mlp_status(ctx) == B.OK
        del W1, W2, W3, dW1, dW2, dW3
        ti = torch.from_numpy(toks).cuda()
        ws = lambda which, shape: B.workspace_tensor(ctx, which, shape, torch.uint8)
        hq_rows = ws(B.WS_HQ, (T, f))[ti].cpu().numpy()
        gu_rows = B.workspace_tensor(ctx, B.WS_GU, (T, 2 * f), torch.int16)[ti].cpu().numpy().view(np.uint16)
        dzq = ws(B.WS_DZQ, (T, 2 * f))
        dz_rows = dzq[ti].cpu().numpy()
        dz_top = float((dzq & 0x7F).max().view(torch.float8_e5m2).float())
        del dzq
        y_rows = y[ti].view(torch.int16).cpu().numpy().view(np.uint16)
        dx_rows = dx[ti].view(torch.int16).cpu().numpy().view(np.uint16)
        scales = {k: v.cpu().numpy() for k, v in sc.items()}
        amax = {k: v.cpu().numpy() for k, v in am.items()}
    finally:
        B.fp8mlp_destroy(ctx)

    E4, E5 = oracle.E4M3, oracle.E5M2
    # one-pass tensors
    a_x, a_dy = oracle.amax(wl.bf16_bits_to_f32(w.x)), oracle.amax(wl.bf16_bits_to_f32(w.dY))
    a_w1, a_w2 = oracle.amax(w.W1), oracle.amax(w.W2)
    sx, sw12 = oracle.scale_from_amax(E4, a_x), oracle.scale_from_amax(E4, max(a_w1, a_w2))
    sdy = oracle.scale_from_amax(E5, a_dy)
    assert amax["x"][0] == np.float32(a_x) and amax["dy"][0] == np.float32(a_dy)
    assert amax["w1"][0] == np.float32(a_w1) and amax["w2"][0] == np.float32(a_w2)
    assert scales["x"][0] == np.float32(sx) and scales["w12"][0] == np.float32(sw12) and scales["dy"][0] == np.float32(sdy)
    # per-channel maxima and s_i on the sampled channels; the invariant on all of them
    probe = oracle.forward(w.x, w.W1[:, chans], w.W2[:, chans], w.W3[chans, :], scale_mode=oracle.SCALE_GIVEN,
                           sx=sx, sw12=sw12, s_h=np.ones(chans.size, np.float32), sw3=1.0)
    assert np.allclose(amax["h"][chans], probe["amax_h"], rtol=AMAX_RTOL, atol=0)
    s_ref = np.array([oracle.pow2_scale(E4, a) for a in probe["amax_h"]], np.float32)
    assert np.array_equal(scales["h"][chans], s_ref), "s_i of the sampled channels"
    s_h = scales["h"]
    prod = s_h.astype(np.float64) * amax["h"]
    assert np.all((prod > 224.0) & (prod <= 448.0)) and np.all(np.frexp(s_h)[0] == 0.5), "s_i: powers of two, (224, 448]"
    # W3' and its scale for that s
    inv_s = (np.float32(1.0) / s_h).astype(np.float32)
    a_w3 = oracle.amax(w.W3, inv_s)
    sw3 = oracle.scale_from_amax(E4, a_w3)
    assert amax["w3"][0] == np.float32(a_w3) and scales["w3"][0] == np.float32(sw3)
    # dZ: its scale from its maximum; the maximum against the largest stored code
    sdz = float(scales["dz"][0])
    assert sdz == oracle.pow2_scale(E5, float(amax["dz"][0])), "scale of dZ from the reported maximum"
    scaled_top = float(amax["dz"][0]) * sdz
    assert 28672.0 < scaled_top <= 57344.0 and abs(dz_top - scaled_top) <= 0.125 * scaled_top

    # sampled tokens with those scales given
    fw = oracle.forward(w.x[toks], w.W1, w.W2, w.W3, scale_mode=oracle.SCALE_GIVEN, sx=sx, sw12=sw12, s_h=s_h, sw3=sw3)
    bw = oracle.backward(fw, w.dY[toks], scale_mode=oracle.SCALE_GIVEN, sdy=sdy, sdz=sdz, want_intermediates=True)
    frac, worst = code_mismatch(hq_rows, fw["Hq"])
    assert worst <= 1 and frac <= CODE_FRAC, f"Hq rows: {frac:.2e} differ, worst {worst}"
    inv = lambda v: np.float32(1.0) / np.float32(v)
    y_shift, y_expl = _explained(E4, hq_rows, fw["Hq"], fw["W3q"], True, inv(sw3))
    fig = dict(Hq_rows_frac=frac, Y=_check_bf16_rows("Y", y_rows, fw["Y"], y_shift), Y_explained=y_expl)
    _check_dz_codes("dZq rows", dz_rows, bw["dZq"])
    dx_shift, dx_expl = _explained(E5, dz_rows, bw["dZq"], fw["W12q"], False, inv(sdz) * inv(sw12))
    fig.update(dX=_check_bf16_rows("dX", dx_rows, bw["dX"], dx_shift), dX_explained=dx_expl)
    g_ref, u_ref = bf16_bits_to_f32(fw["G"]), bf16_bits_to_f32(fw["U"])
    for nm, g_bits, ref in (("G", gu_rows[:, :f], g_ref), ("U", gu_rows[:, f:], u_ref)):
        assert nmax_err_bf16(g_bits, ref) <= 1e-5, f"saved {nm}"
    g_step = np.where(gu_rows[:, :f] != fw["G"], bf16_ulp(g_ref), 0.0)
    u_step = np.where(gu_rows[:, f:] != fw["U"], bf16_ulp(u_ref), 0.0)
    fig.update(amax_dz=check_amax_dz("amax of dZ", amax["dz"][0], bw, g_ref, u_ref, g_step, u_step, AMAX_RTOL, lower_only=True))
    record_parity("full size 7b just-in-time fwd+bwd", tokens=int(toks.size), channels=int(chans.size), **fig)
