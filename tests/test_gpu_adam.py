"""Parity of fp8mlp_adam_step (Adam with E4M3 first moment and E5M2 second moment, Section 5 of the
paper) with the CPU oracle, through the C ABI.  The kernel performs the oracle's fp32 operations in
the oracle's order, so both code arrays and the reported maxima are compared bit for bit over
several steps with the scales re-derived from the previous step's maxima (delayed scaling).  The
weights see the kernel's approximate square root and division (special-function unit, a few 2^-23
relative each): each step may move a weight by 1e-6 of that step's update plus one rounding of the
weight itself, and since the moments never depend on the weights the differences do not feed back."""
import numpy as np
import pytest
import torch

import oracle
from helpers import nmax_err, to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu

HP = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8)


def _dev_state(w0):
    n = w0.size
    one = lambda: torch.ones(1, device="cuda")
    return dict(w=to_dev(w0.ravel()), g=None, m=torch.zeros(n, dtype=torch.uint8, device="cuda"),
                v=torch.zeros(n, dtype=torch.uint8, device="cuda"), scale_m_in=one(), scale_v_in=one(),
                scale_m_out=one(), scale_v_out=one(), amax_m=torch.zeros(1, device="cuda"), amax_v=torch.zeros(1, device="cuda"))


class _OracleState:
    def __init__(self, w0):
        self.w = w0.ravel().copy()
        self.m = np.zeros(self.w.size, np.uint8)
        self.v = np.zeros(self.w.size, np.uint8)
        self.sm_in = self.sv_in = self.sm_out = self.sv_out = np.float32(1.0)

    def step(self, g, t, wd):
        am, av = oracle.adam_step(self.w, g.ravel(), self.m, self.v, weight_decay=wd, step=t, sm_in=self.sm_in,
                                  sv_in=self.sv_in, sm_out=self.sm_out, sv_out=self.sv_out, **HP)
        # the codes are now written with the "out" scales; the next step stores with scales from these maxima
        self.sm_in, self.sv_in = self.sm_out, self.sv_out
        self.sm_out = np.float32(oracle.scale_from_amax(oracle.E4M3, am))
        self.sv_out = np.float32(oracle.scale_from_amax(oracle.E5M2, av))
        return am, av


def _advance_scales(st):
    st["scale_m_in"].copy_(st["scale_m_out"])
    st["scale_v_in"].copy_(st["scale_v_out"])
    B.fp8mlp_scale_from_amax(st["amax_m"], B.E4M3, st["scale_m_out"])
    B.fp8mlp_scale_from_amax(st["amax_v"], B.E5M2, st["scale_v_out"])


@pytest.mark.parametrize("sizes,wd", [((16,), 0.0), ((256 * 704, 256 * 704, 704 * 256), 0.1), ((48 * 1024 + 16, 999 * 16), 0.01),
                                      ((3 * 1024 * 1024 + 32,), 0.0)])
def test_adam_steps_bit_exact(sizes, wd):
    rng = np.random.default_rng(len(sizes) * 7 + sizes[0])
    w0s = [rng.normal(0, 0.02, n).astype(np.float32) for n in sizes]
    dev = [_dev_state(w0) for w0 in w0s]
    ora = [_OracleState(w0) for w0 in w0s]
    w_prev = {id(st): w0.astype(np.float64).copy() for st, w0 in zip(dev, w0s)}
    drift = {id(st): 0.0 for st in dev}
    for t in range(1, 5):
        # gradients spanning several decades, a few exact zeros, a few outliers
        grads = []
        for n in sizes:
            g = (rng.normal(0, 1e-3, n) * np.exp(rng.normal(0, 2, n))).astype(np.float32)
            g[rng.random(n) < 0.01] = 0.0
            grads.append(g)
        for st, g in zip(dev, grads):
            st["g"] = to_dev(g)
        B.fp8mlp_adam_step(dev, weight_decay=wd, step=t, **HP)
        torch.cuda.synchronize()
        for st, o, g in zip(dev, ora, grads):
            am, av = o.step(g, t, wd)
            assert st["amax_m"].item() == np.float32(am) and st["amax_v"].item() == np.float32(av)
            assert np.array_equal(st["m"].cpu().numpy(), o.m), f"first-moment codes, step {t}"
            assert np.array_equal(st["v"].cpu().numpy(), o.v), f"second-moment codes, step {t}"
            w_before = w_prev[id(st)]
            got_w = st["w"].cpu().numpy()
            slack = 1e-6 * np.abs(o.w.astype(np.float64) - w_before) + np.spacing(np.abs(o.w)) + drift[id(st)]
            assert np.all(np.abs(got_w.astype(np.float64) - o.w) <= slack), f"weights, step {t}"
            drift[id(st)] = np.abs(got_w.astype(np.float64) - o.w)          # carried into the next step's bound
            w_prev[id(st)] = o.w.astype(np.float64).copy()
            _advance_scales(st)
            assert st["scale_m_out"].item() == o.sm_out and st["scale_v_out"].item() == o.sv_out


def test_adam_consumes_the_gradients_of_backward():
    """The block's backward feeds the optimizer: dW1, dW2, dW3 from fp8mlp_backward go straight into
    fp8mlp_adam_step.  The oracle chain (its own backward, its own Adam) must land on the same weights
    up to what the 2e-3-level differences of the gradients can move one Adam step."""
    w = wl.make_config("tiny")
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    bw = oracle.backward(fw, w.dY)
    ctx = B.fp8mlp_create(w.T, w.d, w.f, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(w.f), B.new_amax(w.f)
        Ws = [to_dev(a) for a in (w.W1, w.W2, w.W3)]
        y = torch.zeros((w.T, w.d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros_like(y)
        dWs = [torch.zeros_like(a) for a in Ws]
        B.fp8mlp_forward(ctx, w.T, to_dev_bf16(w.x), Ws[0], Ws[1], Ws[2], B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        B.fp8mlp_backward(ctx, w.T, to_dev_bf16(w.dY), B.SCALE_FROM_CURRENT_AMAX, sc, am, dx, dWs[0], dWs[1], dWs[2])
        states = []
        for W, dW in zip(Ws, dWs):
            st = _dev_state(np.zeros(W.numel(), np.float32))
            st["w"], st["g"] = W.view(-1), dW.view(-1)
            states.append(st)
        B.fp8mlp_adam_step(states, weight_decay=0.0, step=1, **HP)
        assert B.fp8mlp_status(ctx) == B.OK
        for W, w0, g in zip(Ws, (w.W1, w.W2, w.W3), (bw["dW1"], bw["dW2"], bw["dW3"])):
            o = _OracleState(w0)
            o.step(g, 1, 0.0)
            got = W.cpu().numpy().ravel()
            assert np.abs(got - w0.ravel()).max() > 0.5 * HP["lr"]          # the step was taken
            # first step: |update| = lr * |g| / (|g| + eps'), insensitive to small relative changes of g
            assert np.abs(got - o.w).max() <= 1e-2 * HP["lr"]
    finally:
        B.fp8mlp_destroy(ctx)


def test_adam_argument_errors():
    L = B.lib()
    n0 = L.fp8mlp_launch_count()
    assert L.fp8mlp_adam_step(None, 1, 1e-3, 0.9, 0.95, 1e-8, 0.0, 1, None) == B.ERR_ARG
    arr = (B._AdamTensor * 1)()
    arr[0].n = 24
    assert L.fp8mlp_adam_step(arr, 1, 1e-3, 0.9, 0.95, 1e-8, 0.0, 1, None) == B.ERR_SHAPE
    arr[0].n = 32
    assert L.fp8mlp_adam_step(arr, 1, 1e-3, 0.9, 0.95, 1e-8, 0.0, 1, None) == B.ERR_ARG      # null scales
    assert L.fp8mlp_adam_step(arr, 1, 1e-3, 0.9, 0.95, 1e-8, 0.0, 0, None) == B.ERR_ARG      # step 0
    assert L.fp8mlp_adam_step(arr, 9, 1e-3, 0.9, 0.95, 1e-8, 0.0, 1, None) == B.ERR_ARG
    assert L.fp8mlp_launch_count() == n0


def test_adam_step_that_also_casts_the_weights_for_the_next_forward():
    """fp8mlp_adam_step_cast on the three weight matrices of a block, the codes going straight into a context's FP8
    weight buffers ([W2 | W1] with one scale, W3' = diag(1/s) W3 with its own), then a forward that takes them as
    they are.  Against the oracle (step, then its quantise routine): moments and their maxima bit for bit as in
    the plain step; the weight codes equal except where the kernel's approximate square root and division moved a
    weight across a rounding boundary (at most one step on at most 1e-4 of the codes), their maxima to 1e-6.
    Against the CUDA path itself: the codes equal, bit for bit, what the forward's own weight pass makes of the
    updated master weights, and the two forwards give the same output bit for bit."""
    from helpers import bf16_dev_to_bits, code_mismatch
    w = wl.make("ac", 17, 96, 128, 208, w_std=0.05, channel_outlier_frac=0.02)
    T, d, f = w.T, w.d, w.f
    rng = np.random.default_rng(5)
    grads = [rng.normal(0, 1e-3, a.shape).astype(np.float32) for a in (w.W1, w.W2, w.W3)]
    s_h = (2.0 ** rng.integers(-3, 5, f)).astype(np.float32)
    sw12, sw3 = np.float32(2000.0), np.float32(700.0)
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.01)
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        sc["h"].copy_(to_dev(s_h)); sc["w12"].fill_(float(sw12)); sc["w3"].fill_(float(sw3)); sc["x"].fill_(64.0)
        dev = [_dev_state(a) for a in (w.W1, w.W2, w.W3)]
        for st, g in zip(dev, grads):
            st["g"] = to_dev(g.ravel())
        p12, _ = B.fp8mlp_workspace(ctx, B.WS_W12Q)
        p3, _ = B.fp8mlp_workspace(ctx, B.WS_W3Q)
        amax_q = [torch.zeros(1, device="cuda") for _ in range(3)]
        casts = [dict(dst=p12 + f, cols=f, ld_dst=2 * f, scale=sc["w12"], amax=amax_q[0]),            # W1: linear half
                 dict(dst=p12, cols=f, ld_dst=2 * f, scale=sc["w12"], amax=amax_q[1]),                # W2: gate half
                 dict(dst=p3, cols=d, ld_dst=d, scale=sc["w3"], row_div=sc["h"], amax=amax_q[2])]      # W3' = diag(1/s) W3
        B.fp8mlp_adam_step_cast(dev, casts, step=1, **hp)
        torch.cuda.synchronize()
        w12q = B.workspace_tensor(ctx, B.WS_W12Q, (d, 2 * f), torch.uint8).cpu().numpy()
        w3q = B.workspace_tensor(ctx, B.WS_W3Q, (f, d), torch.uint8).cpu().numpy()
        # forward on the codes as they are ...
        x = to_dev_bf16(w.x)
        y_cast = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        B.fp8mlp_forward(ctx, T, x, None, None, None, B.SCALE_GIVEN_WEIGHTS_CAST, sc, am, y_cast)
        # ... and the ordinary forward from the updated masters, which redoes the cast
        W1n, W2n, W3n = (st["w"].view(a.shape) for st, a in zip(dev, (w.W1, w.W2, w.W3)))
        y_plain = torch.zeros_like(y_cast)
        B.fp8mlp_forward(ctx, T, x, W1n, W2n, W3n, B.SCALE_GIVEN, sc, am, y_plain)
        assert B.fp8mlp_status(ctx) == B.OK
        w12q_plain = B.workspace_tensor(ctx, B.WS_W12Q, (d, 2 * f), torch.uint8).cpu().numpy()
        w3q_plain = B.workspace_tensor(ctx, B.WS_W3Q, (f, d), torch.uint8).cpu().numpy()
        amax_plain = [am[k].item() for k in ("w1", "w2", "w3")]
    finally:
        B.fp8mlp_destroy(ctx)
    assert np.array_equal(w12q, w12q_plain) and np.array_equal(w3q, w3q_plain), "codes differ from the forward's own weight pass"
    assert [a.item() for a in amax_q] == amax_plain
    assert np.array_equal(bf16_dev_to_bits(y_cast), bf16_dev_to_bits(y_plain))
    # the oracle: step, then quantise
    for (st, a, g, got_codes, scale, div, aq) in ((dev[0], w.W1, grads[0], w12q[:, f:], sw12, None, amax_q[0]),
                                                 (dev[1], w.W2, grads[1], w12q[:, :f], sw12, None, amax_q[1]),
                                                 (dev[2], w.W3, grads[2], w3q, sw3, s_h, amax_q[2])):
        wo = a.ravel().copy()
        mo, vo = np.zeros(wo.size, np.uint8), np.zeros(wo.size, np.uint8)
        o_am, o_av, o_codes, o_amax = oracle.adam_step_and_cast(wo, g.ravel(), mo, vo, cols=a.shape[1], scale=float(scale),
                                                               row_div=div, step=1, **hp)
        assert np.array_equal(st["m"].cpu().numpy(), mo) and np.array_equal(st["v"].cpu().numpy(), vo)
        assert st["amax_m"].item() == np.float32(o_am) and st["amax_v"].item() == np.float32(o_av)
        frac, worst = code_mismatch(got_codes, o_codes)
        assert worst <= 1 and frac <= 1e-4, f"weight codes: {frac:.2e} differ, worst {worst}"
        assert np.isclose(aq.item(), o_amax, rtol=1e-6, atol=0)
