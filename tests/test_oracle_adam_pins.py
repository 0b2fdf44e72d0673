"""Pins of the Adam-with-FP8-moments oracle (oracle/fp8adam_oracle.c), all on the CPU.

The paper (Section 5) fixes the storage formats - first moment E4M3, second moment E5M2 - and why:
the update divides by the square root of the second moment, so its smallest values matter and it
needs the wider exponent range.  Everything else is textbook Adam, so the oracle is pinned against
a library Adam / AdamW with the quantisation switched off, its FP8 encoder against two others that
were written independently (the MLP oracle's integer-bit encoder and torch's casts), and the
paper's format claim against a toy problem."""
import numpy as np
import pytest
import torch

import oracle

HP = dict(lr=1e-2, beta1=0.9, beta2=0.95, eps=1e-8)


def test_codes_agree_with_two_independent_encoders():
    rng = np.random.default_rng(0)
    for second, fmt, tdt, top in ((False, oracle.E4M3, torch.float8_e4m3fn, 0x7E), (True, oracle.E5M2, torch.float8_e5m2, 0x7B)):
        for code in range(256):
            if (code & 0x7F) > top:
                continue                                    # NaN / inf codes are never produced
            assert oracle.adam_decode(second, code) == oracle.decode(fmt, np.array([code], np.uint8))[0]
        lim = oracle.fmt_max(fmt)
        vals = np.concatenate([rng.normal(0, lim / 4, 20000), rng.normal(0, 1e-2, 20000), rng.uniform(-2 * lim, 2 * lim, 5000),
                               [0.0, -0.0, lim, -lim, lim * 1.03, 1e30, -1e30]]).astype(np.float32)
        mine = np.array([oracle.adam_encode(second, v) for v in vals], np.uint8)
        assert np.array_equal(mine, oracle.encode(fmt, vals))
        inside = np.abs(vals) <= lim
        lib = torch.from_numpy(vals[inside]).to(tdt).view(torch.uint8).numpy()
        assert np.array_equal(mine[inside], lib)


@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_unquantised_steps_equal_a_library_adamw_in_fp64(wd):
    rng = np.random.default_rng(1)
    n, steps = 4096, 25
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    grads = [(rng.normal(0, 1e-3, n) * (1 + 10 * (rng.random(n) < 0.01))).astype(np.float32) for _ in range(steps)]
    p = torch.tensor(w0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([p], lr=HP["lr"], betas=(float(np.float32(HP["beta1"])), float(np.float32(HP["beta2"]))),
                            eps=float(np.float32(HP["eps"])), weight_decay=float(np.float32(wd)))
    w = w0.copy()
    m32, v32 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t, g in enumerate(grads, start=1):
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        am, av = oracle.adam_step(w, g, None, None, weight_decay=wd, step=t, m32=m32, v32=v32, **HP)
        assert am == np.abs(m32).max() and av == v32.max()
    ref = p.detach().numpy()
    assert np.abs(w - ref).max() <= 2e-6 * np.abs(ref).max()            # fp32 rounding of 25 steps
    # a dropped bias correction, a swapped beta or a misplaced epsilon moves w by far more than that
    assert np.abs(w - w0).max() > 1e-2


def test_first_step_and_stored_codes():
    """From a zero state the first step does not depend on the stored moments: quantised and
    unquantised runs give the same weights and maxima, and the stored codes are the nearest codes
    of the fp32 moments times the scale (encoder of the MLP oracle)."""
    rng = np.random.default_rng(2)
    n = 10000
    w0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    wa, wb = w0.copy(), w0.copy()
    m32, v32 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    mq, vq = np.zeros(n, np.uint8), np.zeros(n, np.uint8)
    oracle.adam_step(wa, g, None, None, weight_decay=0.01, step=1, m32=m32, v32=v32, **HP)
    sm, sv = np.float32(448.0 / np.abs(m32).max()), np.float32(57344.0 / v32.max())
    am, av = oracle.adam_step(wb, g, mq, vq, weight_decay=0.01, step=1, sm_out=sm, sv_out=sv, **HP)
    assert np.array_equal(wa, wb) and am == np.abs(m32).max() and av == v32.max()
    assert np.array_equal(mq, oracle.encode(oracle.E4M3, m32 * sm))
    assert np.array_equal(vq, oracle.encode(oracle.E5M2, v32 * sv))
    assert mq.max() >= 0x7E - 1 and vq.max() == 0x7B              # the maxima land on the top codes
    # second step decodes with the scales the codes were written with
    wc = wb.copy()
    m2 = (oracle.decode(oracle.E4M3, mq) * np.float32(np.float32(1.0) / sm)).astype(np.float32)
    v2 = (oracle.decode(oracle.E5M2, vq) * np.float32(np.float32(1.0) / sv)).astype(np.float32)
    oracle.adam_step(wb, g, mq, vq, weight_decay=0.01, step=2, sm_in=sm, sv_in=sv, sm_out=sm, sv_out=sv, **HP)
    oracle.adam_step(wc, g, None, None, weight_decay=0.01, step=2, m32=m2, v32=v2, **HP)
    assert np.array_equal(wb, wc)                                 # quantised step == fp32 step on the decoded state


def _toy_run(flags, steps=300):
    """Least squares in 64 coordinates whose gradient scales span four decades, per-tensor scaled moments."""
    rng = np.random.default_rng(3)
    n = 64
    curv = np.logspace(-2, 2, n).astype(np.float32)
    target = rng.normal(0, 1, n).astype(np.float32)
    w = np.zeros(n, np.float32)
    mq, vq = np.zeros(n, np.uint8), np.zeros(n, np.uint8)
    m32, v32 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    sm = sv = np.float32(1.0)
    worst_step = 0.0
    for t in range(1, steps + 1):
        g = (curv * (w - target)).astype(np.float32)
        before = w.copy()
        if flags & oracle.ADAM_Q_IDENTITY:
            oracle.adam_step(w, g, None, None, lr=0.05, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.0, step=t, m32=m32, v32=v32)
        else:
            am, av = oracle.adam_step(w, g, mq, vq, lr=0.05, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.0, step=t,
                                      sm_in=sm, sv_in=sv, sm_out=sm, sv_out=sv, flags=flags)
            if t == 1:                                # delayed scaling: fix the scales from the first maxima
                top_m = 57344.0 if flags & oracle.ADAM_M_AS_E5M2 else 448.0
                top_v = 448.0 if flags & oracle.ADAM_V_AS_E4M3 else 57344.0
                sm, sv = np.float32(top_m / (2 * am)), np.float32(top_v / (2 * av))
                mq[:], vq[:] = 0, 0
                w[:] = 0
                continue
        worst_step = max(worst_step, float(np.abs(w - before).max()))
    return float(np.abs(w - target).max()), worst_step


def test_second_moment_needs_the_range_of_e5m2():
    """Section 5: the second moment's small values decide the update (inverse square root), so it
    needs E5M2's range; E4M3 is enough for the first moment.  With per-tensor scaling, E4M3 flushes
    the second moment of the low-curvature coordinates to zero and the step m / (0 + eps) explodes."""
    err_fp32, step_fp32 = _toy_run(oracle.ADAM_Q_IDENTITY)
    err_ok, step_ok = _toy_run(0)                                   # m E4M3, v E5M2: the paper's choice
    err_bad, step_bad = _toy_run(oracle.ADAM_V_AS_E4M3)             # v in E4M3
    assert err_fp32 < 0.2 and err_ok < 0.3
    assert step_ok < 4 * step_fp32 + 0.1
    assert step_bad > 1e3 * step_ok                                 # exploding steps


def test_step_and_cast_is_the_step_followed_by_the_forward_quantisation():
    """The optimizer step that also emits the next forward's E4M3 weight codes is, on the oracle side, the step
    followed by the quantise routine: with lr = 0 the codes are those of the untouched weights; otherwise a
    library's E4M3 cast of (w_new / row_div) * scale, and the reported maximum numpy's."""
    import torch
    rng = np.random.default_rng(3)
    rows, cols = 24, 32
    w = rng.normal(0, 0.02, rows * cols).astype(np.float32)
    g = rng.normal(0, 1e-3, rows * cols).astype(np.float32)
    s = (2.0 ** rng.integers(-2, 6, rows)).astype(np.float32) * np.float32(1.5)
    scale = np.float32(300.0)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.01, step=1)
    w0 = w.copy()
    _, _, codes0, a0 = oracle.adam_step_and_cast(w0, g, np.zeros(w.size, np.uint8), np.zeros(w.size, np.uint8), cols=cols,
                                                 scale=scale, row_div=s, **dict(hp, lr=0.0, weight_decay=0.0))
    ref0, _, ra0 = oracle.quantize(w.reshape(rows, cols), oracle.E4M3, scale, row_mul=(np.float32(1) / s).astype(np.float32))
    assert np.array_equal(w0, w) and np.array_equal(codes0, ref0) and a0 == ra0
    w1, w2 = w.copy(), w.copy()
    m1, v1 = np.zeros(w.size, np.uint8), np.zeros(w.size, np.uint8)
    m2, v2 = np.zeros(w.size, np.uint8), np.zeros(w.size, np.uint8)
    am, av, codes, amax_w = oracle.adam_step_and_cast(w1, g, m1, v1, cols=cols, scale=scale, row_div=s, **hp)
    am2, av2 = oracle.adam_step(w2, g, m2, v2, **hp)
    assert np.array_equal(w1, w2) and np.array_equal(m1, m2) and np.array_equal(v1, v2) and (am, av) == (am2, av2)
    scaled = (w2.reshape(rows, cols) * (np.float32(1) / s).astype(np.float32)[:, None]).astype(np.float32)
    lib_codes = torch.from_numpy((scaled * scale).astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes, lib_codes) and np.float32(amax_w) == np.abs(scaled).max()
