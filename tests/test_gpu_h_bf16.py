"""The paper's "SwiGLU output in BF16" variant (Section 4.3: everything FP8 except the last linear
layer of the block, whose input is not quantised) through the C ABI: the bf16 tcgen05 GEMM in all
operand layouts, and forward + backward of an FP8MLP_H_BF16 context against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import (bf16_bits_to_f32, bf16_dev_to_bits, bf16_ulp, check_amax_dz, code_mismatch, nmax_err, nmax_err_bf16, to_dev, to_dev_bf16)
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("a_k,b_k", [(True, True), (True, False), (False, False), (False, True)])
@pytest.mark.parametrize("shape", [(128, 256, 64), (16, 16, 16), (144, 272, 400), (640, 768, 1024)])
def test_bf16_gemm_layouts(a_k, b_k, shape):
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    Abits = wl.f32_to_bf16_bits(rng.normal(0, 1, (M, K) if a_k else (K, M)).astype(np.float32))
    Bbits = wl.f32_to_bf16_bits(rng.normal(0, 1, (N, K) if b_k else (K, N)).astype(np.float32))
    Af, Bf = bf16_bits_to_f32(Abits), bf16_bits_to_f32(Bbits)
    ref = oracle.gemm(Af if a_k else Af.T, Bf.T if b_k else Bf)
    out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.fp8mlp_gemm_bf16(M, N, K, to_dev_bf16(Abits), a_k, to_dev_bf16(Bbits), b_k, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.all(np.isfinite(got))
    # bf16 x bf16 products are exact in fp32; only the accumulation order differs
    assert nmax_err(got, ref) <= 2e-5


@pytest.mark.parametrize("cfg", ["tiny", (333, 512, 1040)])
@pytest.mark.parametrize("mode", [B.SCALE_FROM_CURRENT_AMAX])
def test_h_bf16_forward_backward(cfg, mode):
    w = wl.make_config("tiny") if cfg == "tiny" else wl.make("hb", 31, *cfg, w_std=0.05, channel_outlier_frac=0.01)
    T, d, f = w.T, w.d, w.f
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=oracle.FLAG_H_BF16, want_float_operands=True)
    bw = oracle.backward(fw, w.dY, want_intermediates=True)
    ctx = B.fp8mlp_create(T, d, f, B.H_BF16 | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        y = torch.zeros((T, d), dtype=torch.bfloat16, device="cuda")
        dx = torch.zeros_like(y)
        dW1 = torch.full((d, f), float("nan"), device="cuda")
        dW2 = torch.full((d, f), float("nan"), device="cuda")
        dW3 = torch.full((f, d), float("nan"), device="cuda")
        B.fp8mlp_forward(ctx, T, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3), mode, sc, am, y)
        B.fp8mlp_backward(ctx, T, to_dev_bf16(w.dY), mode, sc, am, dx, dW1, dW2, dW3)
        assert B.fp8mlp_status(ctx) == B.OK
        ws = lambda which, shape, dt=torch.uint8: B.workspace_tensor(ctx, which, shape, dt).cpu().numpy()
        assert np.array_equal(ws(B.WS_XQ, (T, d)), fw["Xq"]) and np.array_equal(ws(B.WS_W12Q, (d, 2 * f)), fw["W12q"])
        w3b = ws(B.WS_W3B, (f, d), torch.int16).view(np.uint16)
        assert np.array_equal(bf16_bits_to_f32(w3b), fw["w3q_f"]), "W3 in bf16"
        assert am["w3"].item() == np.float32(fw["amax_w3"])
        assert np.allclose(am["h"].cpu().numpy(), fw["amax_h"], rtol=1e-5, atol=0)
        hb = ws(B.WS_HB, (T, f), torch.int16).view(np.uint16)
        assert nmax_err_bf16(hb, fw["hq_f"]) <= 1e-5, "H in bf16"
        assert nmax_err_bf16(bf16_dev_to_bits(y), fw["Y"]) <= 2e-3, "Y"
        g, u = bf16_bits_to_f32(fw["G"]), bf16_bits_to_f32(fw["U"])
        gu = ws(B.WS_GU, (T, 2 * f), torch.int16).view(np.uint16)
        check_amax_dz("amax of dZ", am["dz"].item(), bw, g, u, np.where(gu[:, :f] != fw["G"], bf16_ulp(g), 0.0),
                      np.where(gu[:, f:] != fw["U"], bf16_ulp(u), 0.0))      # one spacing where the saved value differs
        assert sc["dz"].item() == np.float32(bw["sdz"])
        frac, worst = code_mismatch(ws(B.WS_DZQ, (T, 2 * f)), bw["dZq"])
        assert worst <= 1 and frac <= 1e-3, f"dZq codes: {frac:.2e} differ, worst {worst}"
        assert nmax_err_bf16(bf16_dev_to_bits(dx), bw["dX"]) <= 2e-3, "dX"
        for name, got, ref in (("dW1", dW1, bw["dW1"]), ("dW2", dW2, bw["dW2"]), ("dW3", dW3, bw["dW3"])):
            g = got.cpu().numpy()
            assert np.all(np.isfinite(g)), name
            assert nmax_err(g, ref) <= 2e-3, f"{name}: {nmax_err(g, ref)}"
    finally:
        B.fp8mlp_destroy(ctx)


def test_h_bf16_excludes_smooth():
    L = B.lib()
    import ctypes as C
    h = C.c_void_p()
    assert L.fp8mlp_create(C.byref(h), 16, 16, 16, B.SMOOTH | B.H_BF16) == B.ERR_ARG
