"""Parity of the amax / FP8 cast / scale kernels with the CPU oracle: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f32, to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _one(dev):
    return torch.ones(1, dtype=torch.float32, device=dev), torch.zeros(1, dtype=torch.float32, device=dev)


@pytest.mark.parametrize("fmt", [B.E4M3, B.E5M2])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape", [(1, 16), (37, 48), (128, 256), (1000, 1008), (3, 4096)])
def test_current_amax_quantize_is_bit_exact(fmt, dtype, shape):
    rows, cols = shape
    v = wl.normals(17, 99, rows * cols, std=3.0).reshape(rows, cols)
    v[0, 0] = 0.0
    v.flat[-1] *= 1e-6                                   # lands in the subnormal range after scaling
    if dtype == "bf16":
        bits = wl.f32_to_bf16_bits(v).reshape(rows, cols)
        src, ref_in = to_dev_bf16(bits), bf16_bits_to_f32(bits)
    else:
        src, ref_in = to_dev(v), v
    scale, amax = _one("cuda")
    dst = torch.zeros((rows, cols), dtype=torch.uint8, device="cuda")
    B.fp8mlp_quantize(src, fmt, B.SCALE_FROM_CURRENT_AMAX, scale, amax, None, dst)
    a = oracle.amax(ref_in)
    s = oracle.scale_from_amax(fmt, a)
    codes, _, _ = oracle.quantize(ref_in, fmt, s)
    assert amax.item() == a and scale.item() == s
    assert np.array_equal(dst.cpu().numpy(), codes)


@pytest.mark.parametrize("fmt", [B.E4M3, B.E5M2])
def test_given_scale_saturates_and_reports_amax(fmt):
    rows, cols = 64, 128
    v = wl.normals(3, 5, rows * cols, std=1.0).reshape(rows, cols)
    v[5, 7], v[9, 100] = 1e6, -1e6                       # far beyond the scaled range: must saturate
    src = to_dev(v)
    scale = torch.full((1,), 100.0 if fmt == B.E4M3 else 20000.0, dtype=torch.float32, device="cuda")
    amax = torch.full((1,), 123.0, dtype=torch.float32, device="cuda")     # stale value must be overwritten
    dst = torch.zeros((rows, cols), dtype=torch.uint8, device="cuda")
    B.fp8mlp_quantize(src, fmt, B.SCALE_GIVEN, scale, amax, None, dst)
    codes, _, a = oracle.quantize(v, fmt, scale.item())
    got = dst.cpu().numpy()
    assert np.array_equal(got, codes)
    top = 0x7E if fmt == B.E4M3 else 0x7B
    assert got[5, 7] == top and got[9, 100] == (top | 0x80)
    assert amax.item() == a == 1e6
    # amax is optional with a given scale
    dst2 = torch.zeros_like(dst)
    B.fp8mlp_quantize(src, fmt, B.SCALE_GIVEN, scale, None, None, dst2)
    assert torch.equal(dst, dst2)


def test_row_multiplier_and_strided_destination():
    """W3' = diag(s^-1) W3 written into a wider buffer (the [W2|W1] layout uses the same path)."""
    rows, cols, ld = 96, 64, 160
    v = wl.normals(8, 2, rows * cols, std=0.02).reshape(rows, cols)
    rm = (2.0 ** np.random.default_rng(0).integers(-12, 3, rows)).astype(np.float32)
    rm[3] = 0.3                                          # not a power of two: product is rounded once
    scale, amax = _one("cuda")
    dst = torch.full((rows, ld), 0xAA, dtype=torch.uint8, device="cuda")
    # destination = columns [32, 32+cols) of the wider buffer: base pointer offset by 32 bytes, ld_dst = ld
    import ctypes as C
    src_d, rm_d = to_dev(v), to_dev(rm)
    rc = B.lib().fp8mlp_quantize(C.c_void_p(src_d.data_ptr()), B.F32, rows, cols, B.E4M3, B.SCALE_FROM_CURRENT_AMAX,
                                 C.c_void_p(scale.data_ptr()), C.c_void_p(amax.data_ptr()), C.c_void_p(rm_d.data_ptr()),
                                 C.c_void_p(dst.data_ptr() + 32), ld, C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0
    torch.cuda.synchronize()
    a = oracle.amax(v, row_mul=rm)
    s = oracle.scale_from_amax(B.E4M3, a)
    codes, _, _ = oracle.quantize(v, B.E4M3, s, row_mul=rm)
    got = dst.cpu().numpy()
    assert amax.item() == a and scale.item() == s
    assert np.array_equal(got[:, 32:32 + cols], codes)
    assert np.all(got[:, :32] == 0xAA) and np.all(got[:, 32 + cols:] == 0xAA)      # canaries untouched


def test_empty_tensor():
    scale, amax = _one("cuda")
    amax.fill_(5.0)
    # zero rows: pointers of empty tensors may be null, so pass a real one
    keep = torch.zeros(64, dtype=torch.float32, device="cuda")
    import ctypes as C
    rc = B.lib().fp8mlp_quantize(C.c_void_p(keep.data_ptr()), B.F32, 0, 64, B.E4M3, B.SCALE_FROM_CURRENT_AMAX,
                                 C.c_void_p(scale.data_ptr()), C.c_void_p(amax.data_ptr()), None,
                                 C.c_void_p(keep.data_ptr()), 64, None)
    assert rc == 0
    torch.cuda.synchronize()
    assert amax.item() == 0.0 and scale.item() == 1.0


@pytest.mark.parametrize("smooth", [True, False])
def test_update_scales_matches_oracle(smooth):
    f = 1024 + 16
    rng = np.random.default_rng(4)
    ah = np.exp(rng.uniform(-20, 12, f)).astype(np.float32)
    ah[0], ah[1], ah[2] = 0.0, 448.0, np.float32(0.875 * 2.0 ** -3)
    ctx = B.fp8mlp_create(16, 64, f, B.SMOOTH if smooth else 0)
    try:
        am, sc = B.new_amax(f), B.new_scales(f)
        vals = dict(x=3.7, w1=0.11, w2=0.09, w3=1e-4, dy=4.4e-3, dz=2.3e-5)
        for k, v in vals.items():
            am[k].fill_(v)
        am["h"].copy_(to_dev(ah))
        B.fp8mlp_update_scales(ctx, am, sc)
        torch.cuda.synchronize()
        f32 = lambda v: float(np.float32(v))
        assert sc["x"].item() == oracle.scale_from_amax(B.E4M3, f32(vals["x"]))
        assert sc["w12"].item() == oracle.scale_from_amax(B.E4M3, f32(max(vals["w1"], vals["w2"])))
        assert sc["w3"].item() == oracle.scale_from_amax(B.E4M3, f32(vals["w3"]))
        assert sc["dy"].item() == oracle.scale_from_amax(B.E5M2, f32(vals["dy"]))
        assert sc["dz"].item() == oracle.pow2_scale(B.E5M2, f32(vals["dz"]))
        got = sc["h"].cpu().numpy()
        if smooth:
            ref = np.array([oracle.pow2_scale(B.E4M3, float(a)) for a in ah], np.float32)
        else:
            ref = np.full(f, oracle.scale_from_amax(B.E4M3, float(ah.max())), np.float32)
        assert np.array_equal(got, ref)
    finally:
        B.fp8mlp_destroy(ctx)


@pytest.mark.parametrize("fmt", [B.E4M3, B.E5M2])
@pytest.mark.parametrize("shape,ld", [((1, 16), 16), ((333, 1040), 1040), ((700, 272), 544), ((4096, 11008), 11008)])
def test_code_stats_match_the_oracle(fmt, shape, ld):
    """fp8mlp_code_stats (zero codes, codes at the largest finite magnitude) against the oracle's counts, exactly; rows
    may be strided (a column block of a wider buffer)."""
    rng = np.random.default_rng(shape[0] + fmt)
    full = rng.integers(0, 256, (shape[0], ld), dtype=np.uint8)
    full[rng.random(full.shape) < 0.05] = 0x80                           # plenty of -0
    full[rng.random(full.shape) < 0.01] = 0x7E if fmt == B.E4M3 else 0xFB  # and of the largest magnitude
    dev = torch.from_numpy(full).cuda()
    counts = torch.full((2,), -1, dtype=torch.int64, device="cuda")
    L = B.lib()
    import ctypes as C
    rc = L.fp8mlp_code_stats(C.c_void_p(dev.data_ptr()), shape[0], shape[1], ld, fmt, C.c_void_p(counts.data_ptr()),
                             C.c_void_p(counts.data_ptr() + 8), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == B.OK
    torch.cuda.synchronize()
    assert tuple(counts.tolist()) == oracle.code_stats(oracle.E4M3 if fmt == B.E4M3 else oracle.E5M2, full[:, :shape[1]])
