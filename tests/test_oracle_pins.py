"""Pins of the CPU oracle against things that are not the oracle.

Each test checks oracle/fp8mlp_oracle.c against something fixed by the paper or by
mathematics: the FP8 format constants (tests/golden), a library FP8/bf16 cast, fp64 brute
force, closed forms, finite differences, and invariants of the Smooth-SwiGLU construction.
"""
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from oracle import E4M3, E5M2, FLAG_NO_BF16, FLAG_Q_IDENTITY, FLAG_SMOOTH, SCALE_CURRENT, SCALE_GIVEN
from paper_2409_12517_b200 import workloads as wl

GOLDEN = Path(__file__).parent / "golden"
TORCH_FMT = {E4M3: torch.float8_e4m3fn, E5M2: torch.float8_e5m2}
ALL_CODES = np.arange(256, dtype=np.uint8)


def _torch_decode(fmt, codes):
    return torch.from_numpy(codes.copy()).view(TORCH_FMT[fmt]).to(torch.float32).numpy()


# ---------------------------------------------------------------- number formats (Section 2)

def test_format_constants_from_golden():
    for line in (GOLDEN / "fp8_format_constants.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        _, fmt_name, code_hex, value = line.split()
        fmt = E4M3 if fmt_name == "e4m3" else E5M2
        code = int(code_hex, 16)
        assert oracle.decode(fmt, np.array([code], np.uint8))[0] == np.float32(float(value))
        assert oracle.encode(fmt, np.array([float(value)], np.float32))[0] == code
    assert oracle.fmt_max(E4M3) == 448.0 and oracle.fmt_max(E5M2) == 57344.0


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_decode_matches_library_for_all_256_codes(fmt):
    mine, ref = oracle.decode(fmt, ALL_CODES), _torch_decode(fmt, ALL_CODES)
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok], ref[ok])
    assert np.array_equal(np.signbit(mine[ok]), np.signbit(ref[ok]))


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_exhaustive_round_trip(fmt):
    vals = oracle.decode(fmt, ALL_CODES)
    finite = np.isfinite(vals)
    back = oracle.encode(fmt, vals[finite])
    assert np.array_equal(back, ALL_CODES[finite])          # includes -0 -> 0x80
    # NaN codes encode to a NaN code; infinities (E5M2 only) saturate to the largest finite
    nan_back = oracle.encode(fmt, np.array([np.nan, -np.nan], np.float32))
    assert np.all(np.isnan(oracle.decode(fmt, nan_back)))
    top = {E4M3: 0x7E, E5M2: 0x7B}[fmt]
    assert list(oracle.encode(fmt, np.array([np.inf, -np.inf, 1e9, -1e9], np.float32))) == [top, top | 0x80, top, top | 0x80]


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_code_order_is_monotone(fmt):
    top = {E4M3: 0x7E, E5M2: 0x7B}[fmt]
    pos = oracle.decode(fmt, np.arange(0, top + 1, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)
    neg = oracle.decode(fmt, np.arange(0x80, 0x80 + top + 1, dtype=np.uint8))
    assert np.array_equal(neg, -pos)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_midpoints_round_to_even_and_neighbours_round_to_nearest(fmt):
    top = {E4M3: 0x7E, E5M2: 0x7B}[fmt]
    codes = np.arange(0, top + 1, dtype=np.uint8)
    v = oracle.decode(fmt, codes).astype(np.float64)
    mid = (v[:-1] + v[1:]) / 2                      # exactly representable in fp32
    even = np.where(codes[:-1] % 2 == 0, codes[:-1], codes[1:])
    assert np.array_equal(oracle.encode(fmt, mid.astype(np.float32)), even)
    assert np.array_equal(oracle.encode(fmt, (-mid).astype(np.float32)), even | 0x80)
    lo = np.nextafter(mid.astype(np.float32), np.float32(0))
    hi = np.nextafter(mid.astype(np.float32), np.float32(np.inf))
    assert np.array_equal(oracle.encode(fmt, lo), codes[:-1])
    assert np.array_equal(oracle.encode(fmt, hi), codes[1:])


def test_saturation_thresholds():
    # E4M3: 448 = 1.75*2^8, the next grid point would be 480; everything from the midpoint 464 up saturates
    assert list(oracle.encode(E4M3, np.array([448, 463.9, 464, 480, 1e30], np.float32))) == [0x7E] * 5
    assert list(oracle.encode(E5M2, np.array([57344, 6e4, 61440, 65536, 1e30], np.float32))) == [0x7B] * 5
    # subnormal grids: spacing 2^-9 and 2^-16, half of the smallest step ties to zero
    assert list(oracle.encode(E4M3, np.array([2.0**-10, 2.0**-10 * 1.0001, 3 * 2.0**-10], np.float32))) == [0, 1, 2]
    assert list(oracle.encode(E5M2, np.array([2.0**-17, 2.0**-17 * 1.0001, 3 * 2.0**-17], np.float32))) == [0, 1, 2]
    assert list(oracle.encode(E4M3, np.array([1e-30, -1e-30, 1e-45], np.float32))) == [0, 0x80, 0]


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_encode_matches_library_cast_in_range(fmt):
    rng = np.random.default_rng(11)
    mx = oracle.fmt_max(fmt)
    mag = np.exp(rng.uniform(np.log(1e-6), np.log(mx), 200000))
    v = (mag * rng.choice([-1.0, 1.0], mag.size)).astype(np.float32)
    v = v[np.abs(v) <= mx]
    ref = torch.from_numpy(v).to(TORCH_FMT[fmt]).view(torch.uint8).numpy()
    assert np.array_equal(oracle.encode(fmt, v), ref)


def test_bf16_rounding_matches_library():
    rng = np.random.default_rng(5)
    v = (rng.standard_normal(100000) * np.exp(rng.uniform(-20, 20, 100000))).astype(np.float32)
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.bf16_bits(v), ref)
    assert np.array_equal(wl.f32_to_bf16_bits(v), ref)          # the input generator's rounding too
    assert np.array_equal(oracle.bf16_to_f32(ref), wl.bf16_bits_to_f32(ref))


# ---------------------------------------------------------------- scaling

def test_per_tensor_scale_and_quantize():
    v = np.array([[0.5, -3.0, 1.25], [0.001, 2.9, -0.75]], np.float32)
    assert oracle.amax(v) == 3.0
    s = oracle.scale_from_amax(E4M3, 3.0)
    assert s == np.float32(448.0) / np.float32(3.0)
    codes, deq, a = oracle.quantize(v, E4M3, s)
    assert a == 3.0
    # the element carrying the amax lands on the largest finite code
    assert codes[0, 1] == 0xFE and deq[0, 1] == -448.0
    ref = torch.from_numpy(v * np.float32(s)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes, ref)
    assert oracle.scale_from_amax(E4M3, 0.0) == 1.0 and oracle.scale_from_amax(E5M2, np.inf) == 1.0
    # row multipliers act before the scale (W3' = diag(s^-1) W3)
    rm = np.array([0.25, 4.0], np.float32)
    codes2, deq2, a2 = oracle.quantize(v, E4M3, 2.0, row_mul=rm)
    assert a2 == 11.6 or a2 == np.float32(2.9) * 4
    assert np.array_equal(codes2, oracle.encode(E4M3, (v * rm[:, None]) * np.float32(2.0)))


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_pow2_scale_is_the_largest_power_of_two_that_fits(fmt):
    mx = oracle.fmt_max(fmt)
    rng = np.random.default_rng(3)
    amaxes = list(np.exp(rng.uniform(np.log(1e-12), np.log(1e12), 2000)).astype(np.float32))
    for k in range(-30, 31):      # exact powers of two and both sides of the 0.875 mantissa boundary
        amaxes += [np.float32(2.0**k), np.float32(0.875 * 2.0**k),
                   np.nextafter(np.float32(0.875 * 2.0**k), np.float32(np.inf)),
                   np.nextafter(np.float32(0.875 * 2.0**k), np.float32(0))]
    for a in amaxes:
        s = oracle.pow2_scale(fmt, float(a))
        m, _ = np.frexp(s)
        assert m == 0.5                                           # a power of two
        assert float(s) * float(a) <= mx < 2.0 * float(s) * float(a)
    assert oracle.pow2_scale(fmt, 0.0) == 1.0


# ---------------------------------------------------------------- GEMM against fp64 brute force

@pytest.mark.parametrize("shape", [(5, 7, 3), (17, 9, 64), (3, 33, 129)])
def test_gemm_matches_fp64_brute_force(shape):
    M, N, K = shape
    rng = np.random.default_rng(M * 1000 + N)
    A = oracle.decode(E4M3, rng.integers(0, 0x7F, (M, K)).astype(np.uint8) | (rng.integers(0, 2, (M, K)) << 7).astype(np.uint8))
    B = oracle.decode(E5M2, rng.integers(0, 0x7C, (K, N)).astype(np.uint8) | (rng.integers(0, 2, (K, N)) << 7).astype(np.uint8))
    ref = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(A[m, k]) * float(B[k, n])
            ref[m, n] = acc
    bound = K * 2.0**-23 * (np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64)) + 1e-30
    got = oracle.gemm(A, B)
    assert np.all(np.abs(got - ref) <= bound)
    # strided (transposed) operands go through the same definition
    At, Bt = np.ascontiguousarray(A.T), np.ascontiguousarray(B.T)
    assert np.array_equal(oracle.gemm(At.T, Bt.T), got)


def test_gemm_is_sequential_fp32_accumulation():
    # 2^24 + 1 + 1 in fp32 from the left stays 2^24; from the right it would be 2^24 + 2
    A = np.array([[16777216.0, 1.0, 1.0]], np.float32)
    B = np.ones((3, 1), np.float32)
    assert oracle.gemm(A, B)[0, 0] == 16777216.0
    assert oracle.gemm(A[:, ::-1], B)[0, 0] == 16777218.0


# ---------------------------------------------------------------- SwiGLU (Section 4.1)

def test_swiglu_quadratic_closed_form():
    # w1 = w2 and w1.x = 1  =>  SwiGLU(c x) = c^2 sigma(c), and SwiGLU(c x)/c^2 -> 1
    for c, sig in ((1.0, 0.7310585786300049), (5.0, 0.9933071490757153), (20.0, 0.9999999979388463), (50.0, 1.0)):
        got = oracle.swiglu(c, c)
        assert abs(got / (c * c) - sig) < 2e-7
    assert oracle.swiglu(3.0, 0.0) == 0.0
    # Swish is odd-asymmetric: large negative gate kills the output, large positive passes it
    assert abs(oracle.swiglu(2.0, -30.0)) < 1e-10 and abs(oracle.swiglu(2.0, 30.0) - 60.0) < 1e-4


def test_swiglu_grad_against_finite_differences():
    rng = np.random.default_rng(0)
    for _ in range(200):
        u, g, dh = (float(np.float32(v)) for v in rng.uniform(-4, 4, 3))
        du, dg = oracle.swiglu_grad(u, g, dh)
        h = lambda uu, gg: uu * gg / (1.0 + np.exp(-gg))
        e = 1e-6
        assert abs(du - dh * (h(u + e, g) - h(u - e, g)) / (2 * e)) < 2e-5 * max(1, abs(du))
        assert abs(dg - dh * (h(u, g + e) - h(u, g - e)) / (2 * e)) < 2e-5 * max(1, abs(dg))


# ---------------------------------------------------------------- the block: definition, derivative, Smooth-SwiGLU

def _small(seed=0, T=9, d=24, f=40, w_std=0.3, outliers=0.0):
    return wl.make("small", seed, T, d, f, w_std=w_std, channel_outlier_frac=outliers, dy_std=1.0)


def test_fp64_block_against_numpy_definition():
    w = _small()
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    H, Y = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    u, g = x @ w.W1.astype(np.float64), x @ w.W2.astype(np.float64)
    Href = u * g / (1 + np.exp(-g))
    assert np.allclose(H, Href, rtol=1e-12, atol=1e-14)
    assert np.allclose(Y, Href @ w.W3.astype(np.float64), rtol=1e-12, atol=1e-14)


def test_fp64_backward_against_finite_differences():
    w = _small(T=4, d=6, f=10)
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    dY = wl.bf16_bits_to_f32(w.dY).astype(np.float64)
    Ws = [w.W1.astype(np.float64), w.W2.astype(np.float64), w.W3.astype(np.float64)]
    dX, dW1, dW2, dW3 = oracle.mlp_f64_backward(x, *Ws, dY)
    loss = lambda xx, a, b, c: float(np.sum(oracle.mlp_f64(xx, a, b, c)[1] * dY))
    eps = 1e-6
    for which, grad in ((0, dX), (1, dW1), (2, dW2), (3, dW3)):
        args = [x.copy()] + [m.copy() for m in Ws]
        it = np.nditer(args[which], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            v = args[which][idx]
            args[which][idx] = v + eps
            lp = loss(*args)
            args[which][idx] = v - eps
            lm = loss(*args)
            args[which][idx] = v
            assert abs((lp - lm) / (2 * eps) - grad[idx]) < 1e-6 * max(1.0, abs(grad[idx]))


@pytest.mark.parametrize("smooth", [True, False])
def test_q_identity_path_reproduces_the_fp64_block_and_its_gradient(smooth):
    """With Q = identity the oracle's fp32 forward/backward code path (the same statements the
    quantised path runs) must be the fp64 block and its finite-difference-checked gradient."""
    w = _small(seed=3, T=11, d=32, f=48, outliers=0.05)
    flags = FLAG_Q_IDENTITY | FLAG_NO_BF16 | (FLAG_SMOOTH if smooth else 0)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=flags, scale_mode=SCALE_CURRENT, want_float_operands=True)
    if smooth:
        assert len(set(fw["s_h"])) > 1                       # non-trivial per-channel scales
    bw = oracle.backward(fw, w.dY, scale_mode=SCALE_CURRENT)
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    dY = wl.bf16_bits_to_f32(w.dY).astype(np.float64)
    H, Y = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    dX, dW1, dW2, dW3 = oracle.mlp_f64_backward(x, w.W1, w.W2, w.W3, dY)
    rel = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    assert rel(fw["H"], H) < 1e-5 and rel(fw["Y"], Y) < 1e-5
    for got, ref in ((bw["dX"], dX), (bw["dW1"], dW1), (bw["dW2"], dW2), (bw["dW3"], dW3)):
        assert rel(got, ref) < 1e-5


def test_smooth_swiglu_does_not_change_the_function():
    """Eq. (2) with Q = identity: scaling channel i by s_i and W3's row i by 1/s_i is the identity,
    for any positive s (<= 1e-6 relative in fp64), and the merged form (s folded into W1's columns
    and 1/s into W3's rows) is the same function again."""
    w = _small(seed=5, T=7, d=16, f=24)
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    s = np.exp(np.random.default_rng(1).uniform(-6, 6, w.f))
    _, Y0 = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    _, Ys = oracle.mlp_f64(x, w.W1, w.W2, w.W3, s=s)
    assert np.max(np.abs(Ys - Y0)) <= 1e-6 * np.max(np.abs(Y0))
    _, Ym = oracle.mlp_f64(x, w.W1.astype(np.float64) * s[None, :], w.W2, w.W3.astype(np.float64) / s[:, None])
    assert np.max(np.abs(Ym - Y0)) <= 1e-6 * np.max(np.abs(Y0))
    # power-of-two s: exactly the same numbers
    s2 = 2.0 ** np.random.default_rng(2).integers(-8, 9, w.f)
    _, Y2 = oracle.mlp_f64(x, w.W1, w.W2, w.W3, s=s2)
    assert np.array_equal(Y2, Y0)


def test_smooth_scales_put_every_channel_in_the_top_binade():
    w = wl.make("o", 7, 64, 64, 256, w_std=0.05, channel_outlier_frac=0.02)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=FLAG_SMOOTH)
    scaled_max = fw["amax_h"] * fw["s_h"]
    assert np.all((scaled_max > 224.0) & (scaled_max <= 448.0))
    assert np.array_equal(fw["amax_h"], np.abs(fw["H"]).max(axis=0))
    # no code of Hq needed saturation: every |s_i H| <= 448 before rounding
    assert np.all(np.abs(fw["H"] * fw["s_h"][None, :]) <= 448.0)
    # W3' = diag(1/s) W3 is what got quantised
    assert fw["amax_w3"] == np.float32(np.abs(w.W3 / fw["s_h"][:, None]).max())


def test_outlier_channels_hurt_per_tensor_scaling_and_not_smooth_swiglu():
    """Aligned channels (w1_i = 8 w2_i) push one per-tensor scale for H so low that ordinary
    channels lose their small values; per-channel scaling keeps them (Sections 3-4)."""
    w = wl.make("o", 9, 96, 128, 512, w_std=0.05, channel_outlier_frac=0.01)
    assert w.outlier_channels.size == 5
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    _, Y = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    on = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=FLAG_SMOOTH)
    off = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=0)
    normal = np.setdiff1d(np.arange(w.f), w.outlier_channels)
    assert np.median(on["amax_h"][w.outlier_channels]) > 8 * np.median(on["amax_h"][normal])
    zeros_on = np.count_nonzero((on["Hq"][:, normal] & 0x7F) == 0)
    zeros_off = np.count_nonzero((off["Hq"][:, normal] & 0x7F) == 0)
    assert zeros_on < zeros_off
    # With the benchmark's gain of 8 FP8's own range still absorbs the outliers; once the aligned
    # channel has also grown in norm (the paper's late-training picture) the ordinary channels
    # lose precision under one per-tensor scale and keep it under per-channel scales.
    w = wl.make("o", 9, 96, 128, 512, w_std=0.05, channel_outlier_frac=0.01, channel_gain=4096.0)
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    H, _ = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    on = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=FLAG_SMOOTH)
    off = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=0)
    herr = lambda r: (np.linalg.norm((oracle.decode(E4M3, r["Hq"]) / r["s_h"][None, :] - H)[:, normal])
                      / np.linalg.norm(H[:, normal]))
    assert herr(on) < 0.07 < 0.08 < herr(off)


@pytest.mark.parametrize("smooth", [True, False])
def test_quantised_block_stays_close_to_the_fp64_block(smooth):
    """FP8 rounding moves results by a few percent; a dropped term, a wrong sign, a transposed
    operand or a missing scale factor moves them by tens of percent or more."""
    w = wl.make("c", 21, 64, 128, 192, w_std=0.05, dy_std=1e-3)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=FLAG_SMOOTH if smooth else 0)
    bw = oracle.backward(fw, w.dY)
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    dY = wl.bf16_bits_to_f32(w.dY).astype(np.float64)
    H, Y = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    dX, dW1, dW2, dW3 = oracle.mlp_f64_backward(x, w.W1, w.W2, w.W3, dY)
    rel = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    assert rel(oracle.bf16_to_f32(fw["G"]), x @ w.W2) < 0.05
    assert rel(oracle.bf16_to_f32(fw["U"]), x @ w.W1) < 0.05
    assert rel(fw["H"], H) < 0.06 and rel(fw["Y"], Y) < 0.08
    assert rel(oracle.decode(E4M3, fw["Hq"]) / fw["s_h"][None, :], H) < 0.07
    for got, ref in ((bw["dX"], dX), (bw["dW1"], dW1), (bw["dW2"], dW2), (bw["dW3"], dW3)):
        assert rel(got, ref) < 0.12


def test_given_scales_reproduce_the_current_amax_run():
    w = wl.make("g", 4, 40, 64, 96, w_std=0.05)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    bw = oracle.backward(fw, w.dY)
    fw2 = oracle.forward(w.x, w.W1, w.W2, w.W3, scale_mode=SCALE_GIVEN, sx=fw["sx"], sw12=fw["sw12"],
                         s_h=fw["s_h"], sw3=fw["sw3"])
    bw2 = oracle.backward(fw2, w.dY, scale_mode=SCALE_GIVEN, sdy=bw["sdy"], sdz=bw["sdz"])
    for k in ("Xq", "W12q", "W3q", "Hq", "G", "U", "Y_bits", "amax_h"):
        assert np.array_equal(fw[k], fw2[k])
    for k in ("dYq", "dZq", "dX_bits", "dW1", "dW2", "dW3"):
        assert np.array_equal(bw[k], bw2[k])


def test_token_and_channel_subsets_reproduce_the_full_run():
    """Rows of Hq/Y/dZq/dX depend only on their own token, and columns/rows of Hq, dZq, dW1, dW2,
    dW3, amax_h only on their own channel, once the scales are given: full-size parity checks
    run the oracle on such subsets."""
    w = wl.make("s", 8, 48, 64, 128, w_std=0.05, channel_outlier_frac=0.02)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    bw = oracle.backward(fw, w.dY)
    given = dict(scale_mode=SCALE_GIVEN, sx=fw["sx"], sw12=fw["sw12"], sw3=fw["sw3"])
    rows = np.array([0, 5, 17, 47])
    fr = oracle.forward(w.x[rows], w.W1, w.W2, w.W3, s_h=fw["s_h"], **given)
    br = oracle.backward(fr, w.dY[rows], scale_mode=SCALE_GIVEN, sdy=bw["sdy"], sdz=bw["sdz"])
    assert np.array_equal(fr["Hq"], fw["Hq"][rows]) and np.array_equal(fr["Y_bits"], fw["Y_bits"][rows])
    assert np.array_equal(br["dZq"], bw["dZq"][rows]) and np.array_equal(br["dX_bits"], bw["dX_bits"][rows])
    ch = np.array([1, 2, 63, 100, 127])
    fc = oracle.forward(w.x, w.W1[:, ch], w.W2[:, ch], w.W3[ch, :], s_h=fw["s_h"][ch], **given)
    bc = oracle.backward(fc, w.dY, scale_mode=SCALE_GIVEN, sdy=bw["sdy"], sdz=bw["sdz"])
    assert np.array_equal(fc["Hq"], fw["Hq"][:, ch]) and np.array_equal(fc["amax_h"], fw["amax_h"][ch])
    f = w.f
    assert np.array_equal(bc["dZq"][:, :ch.size], bw["dZq"][:, ch])
    assert np.array_equal(bc["dZq"][:, ch.size:], bw["dZq"][:, f + ch])
    assert np.array_equal(bc["dW1"], bw["dW1"][:, ch]) and np.array_equal(bc["dW2"], bw["dW2"][:, ch])
    assert np.array_equal(bc["dW3"], bw["dW3"][ch, :])


def test_tiny_config_shapes_and_determinism():
    a, b = wl.make_config("tiny"), wl.make_config("tiny")
    assert a.x.shape == (128, 256) and a.W1.shape == (256, 704) and a.W3.shape == (704, 256)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.W2, b.W2) and np.array_equal(a.dY, b.dY)
    x = wl.bf16_bits_to_f32(a.x)
    assert abs(x.std() - 1.0) < 0.02 and abs(a.W1.std() - 0.02) < 5e-4 and abs(x.mean()) < 0.02
    assert abs(wl.bf16_bits_to_f32(a.dY).std() - 1e-3) < 5e-5
    o = wl.make("o", 1, 16, 32, 2000, channel_outlier_frac=0.001)
    assert o.outlier_channels.size == 2
    assert np.array_equal(o.W1[:, o.outlier_channels], np.float32(8) * o.W2[:, o.outlier_channels])
    t = wl.make("t", 4, 300, 16, 32, token_outlier_frac=0.01)
    assert t.outlier_tokens.size == 3


# ---------------------------------------------------------------- "SwiGLU output in BF16" variant (Section 4.3)
def test_h_bf16_variant_last_layer_runs_in_bf16():
    """The paper's intermediate experiment: everything FP8 except the last linear layer of the block,
    whose input (the SwiGLU output) is not quantised.  Pins: the layer's operands are the bf16
    roundings a library produces; its outputs are the brute-force fp64 contractions of exactly those
    operands; the variant sits closer to the unquantised block than plain FP8 when outlier channels
    are present; and its gradients point where the fp64 block's do."""
    import torch
    w = wl.make("hb", 9, 48, 96, 208, w_std=0.05, channel_outlier_frac=0.02)
    fl = oracle.FLAG_H_BF16
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=fl | oracle.FLAG_NO_BF16, want_float_operands=True)
    to_bf16 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(fw["hq_f"], to_bf16(fw["H"])) and np.array_equal(fw["w3q_f"], to_bf16(w.W3))
    assert fw["sw3"] == 1.0 and np.all(fw["s_h"] == 1.0)
    Y_brute = fw["hq_f"].astype(np.float64) @ fw["w3q_f"].astype(np.float64)
    assert np.abs(fw["Y"] - Y_brute).max() <= 1e-5 * np.abs(Y_brute).max()
    bw = oracle.backward(fw, w.dY)
    dy = wl.bf16_bits_to_f32(w.dY).astype(np.float64)
    assert bw["sdy"] == 1.0
    dW3_brute = fw["hq_f"].astype(np.float64).T @ dy
    assert np.abs(bw["dW3"] - dW3_brute).max() <= 1e-5 * np.abs(dW3_brute).max()
    # against the unquantised block
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    _, Y64 = oracle.mlp_f64(x, w.W1, w.W2, w.W3)
    dX64, dW1_64, dW2_64, dW3_64 = oracle.mlp_f64_backward(x, w.W1, w.W2, w.W3, dy)
    plain = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=oracle.FLAG_NO_BF16)
    err = lambda a, b: np.abs(a - b).max() / np.abs(b).max()
    assert err(fw["Y"], Y64) < err(plain["Y"], Y64)
    cos = lambda a, b: float((a * b).sum() / np.sqrt((a * a).sum() * (b * b).sum()))
    for got, ref in ((bw["dX"], dX64), (bw["dW1"], dW1_64), (bw["dW2"], dW2_64), (bw["dW3"], dW3_64)):
        assert cos(got.astype(np.float64), ref) > 0.99


def test_gu_fp8_option_saved_activations_as_e4m3_codes():
    """Option (the paper does not say how the SwiGLU inputs are kept for backward): G and U are stored as
    E4M3 codes with one per-tensor scale.  Pins: the maximum is numpy's over the fp32 G, U; the scale is
    448 / max; the codes are a library's E4M3 cast of sgu * [G | U]; the decoded values lie within half a
    spacing of G, U; the forward result does not change; backward's dZ codes equal a brute-force fp64
    evaluation of the SwiGLU derivative on the decoded activations; and the gradients still point where
    the fp64 block's do."""
    w = wl.make("gu8", 11, 40, 64, 144, w_std=0.08)
    fl = FLAG_SMOOTH | oracle.FLAG_GU_FP8
    ref = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=FLAG_SMOOTH, want_float_operands=True)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=fl, want_float_operands=True)
    G, U = fw["G_f32"], fw["U_f32"]
    agu = max(np.abs(G).max(), np.abs(U).max())
    assert fw["amax_gu"] == np.float32(agu)
    assert fw["sgu"] == np.float32(448.0) / np.float32(agu)
    scaled = np.concatenate([G, U], axis=1) * np.float32(fw["sgu"])
    lib_codes = torch.from_numpy(scaled).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(fw["GUq"], lib_codes)
    dec = _torch_decode(E4M3, fw["GUq"]).astype(np.float64) / np.float64(fw["sgu"])
    true = np.concatenate([G, U], axis=1).astype(np.float64)
    # 3 mantissa bits: half a spacing is 2^-4 relative in the normal range, 2^-10 / sgu absolute below it
    assert np.all(np.abs(dec - true) <= np.abs(true) * 2.0 ** -4 + 2.0 ** -10 / fw["sgu"] + 1e-12)
    for k in ("Xq", "W12q", "W3q", "Hq", "Y_bits"):
        assert np.array_equal(fw[k], ref[k])
    # backward: the derivative is taken at the decoded activations
    bw = oracle.backward(fw, w.dY)
    inv = np.float32(1.0) / np.float32(fw["sgu"])
    g = (_torch_decode(E4M3, fw["GUq"][:, :144]) * inv).astype(np.float64)
    u = (_torch_decode(E4M3, fw["GUq"][:, 144:]) * inv).astype(np.float64)
    dyq = _torch_decode(E5M2, bw["dYq"]).astype(np.float64) / bw["sdy"]
    w3q = _torch_decode(E4M3, fw["W3q"]).astype(np.float64) / fw["sw3"]
    dh = (dyq @ w3q.T) * fw["s_h"].astype(np.float64)[None, :]
    sig = 1.0 / (1.0 + np.exp(-g))
    dz = np.concatenate([dh * u * sig * (1.0 + g * (1.0 - sig)), dh * g * sig], axis=1)
    assert abs(bw["amax_dz"] - np.abs(dz).max()) <= 1e-5 * np.abs(dz).max()
    got = _torch_decode(E5M2, bw["dZq"]).astype(np.float64) / bw["sdz"]
    # E5M2 spacing is 2^-2 relative: the code of the fp64 value or, on a rounding tie-break, its neighbour
    assert np.all(np.abs(got - dz) <= np.abs(dz) * 2.0 ** -3 * 1.001 + 2.0 ** -17 / bw["sdz"])
    want = torch.from_numpy((dz * bw["sdz"]).astype(np.float32)).to(torch.float8_e5m2).view(torch.uint8).numpy()
    assert np.mean(want != bw["dZq"]) < 2e-3
    # against the bf16-saved run and the unquantised block
    bw_ref = oracle.backward(ref, w.dY)
    x = wl.bf16_bits_to_f32(w.x).astype(np.float64)
    dy = wl.bf16_bits_to_f32(w.dY).astype(np.float64)
    dX64, dW1_64, dW2_64, dW3_64 = oracle.mlp_f64_backward(x, w.W1, w.W2, w.W3, dy)
    assert np.array_equal(bw["dW3"], bw_ref["dW3"])              # does not involve G, U
    cos = lambda a, b: float((a * b).sum() / np.sqrt((a * a).sum() * (b * b).sum()))
    for got_, r64 in ((bw["dX"], dX64), (bw["dW1"], dW1_64), (bw["dW2"], dW2_64)):
        assert cos(got_.astype(np.float64), r64) > 0.99


def test_gu_fp8_option_is_exact_when_the_activations_are_representable():
    """When every G and U is a small integer (exact in E4M3 at a power-of-two scale and in bf16), keeping
    them as E4M3 codes or as bf16 gives bit-identical gradients; a wrong direction of the scale, a swapped
    G / U half or a dropped dequantisation would not."""
    T, d, f = 8, 16, 32
    rng = np.random.default_rng(5)
    x = np.zeros((T, d), np.float32)
    x[np.arange(T), rng.integers(0, d, T)] = 1.0                    # one-hot tokens: G, U are rows of W2, W1
    W1 = rng.integers(-7, 8, (d, f)).astype(np.float32)
    W2 = rng.integers(-7, 8, (d, f)).astype(np.float32)
    W3 = rng.standard_normal((f, d)).astype(np.float32) * 0.1
    dY = wl.f32_to_bf16_bits(rng.standard_normal((T, d)).astype(np.float32))
    xb = wl.f32_to_bf16_bits(x)
    given = dict(scale_mode=SCALE_GIVEN, sx=1.0, sw12=16.0, s_h=np.ones(f, np.float32), sw3=64.0)
    a = oracle.forward(xb, W1, W2, W3, flags=0, **given)
    b = oracle.forward(xb, W1, W2, W3, flags=oracle.FLAG_GU_FP8, sgu=4.0, **given)
    assert np.array_equal(_torch_decode(E4M3, b["GUq"][:, :f]) / 4.0, wl.bf16_bits_to_f32(a["G"]))
    assert np.array_equal(_torch_decode(E4M3, b["GUq"][:, f:]) / 4.0, wl.bf16_bits_to_f32(a["U"]))
    ba = oracle.backward(a, dY, scale_mode=SCALE_GIVEN, sdy=64.0, sdz=8.0)
    bb = oracle.backward(b, dY, scale_mode=SCALE_GIVEN, sdy=64.0, sdz=8.0)
    for k in ("dZq", "dX_bits", "dW1", "dW2", "dW3"):
        assert np.array_equal(ba[k], bb[k]), k


def test_backward_intermediates_are_what_the_codes_and_the_maximum_are_made_of():
    """The optional fp32 outputs of the backward (dH and dZ = [dG | dU] before the E5M2 cast): a library cast of
    sdz * dZ gives the stored codes, numpy's max |dZ| the reported maximum, and dZ follows from dH and the saved
    activations by the element-wise gradient routine (pinned on its own against finite differences)."""
    w = wl.make("im", 9, 24, 64, 96, w_std=0.05, channel_outlier_frac=0.02)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    bw = oracle.backward(fw, w.dY, want_intermediates=True)
    plain = oracle.backward(fw, w.dY)
    assert np.array_equal(bw["dZq"], plain["dZq"]) and np.array_equal(bw["dW1"], plain["dW1"])   # asking changes nothing
    assert np.float32(np.abs(bw["dZ"]).max()) == np.float32(bw["amax_dz"])
    lib_codes = (torch.from_numpy(bw["dZ"] * np.float32(bw["sdz"])).to(torch.float8_e5m2)).view(torch.uint8).numpy()
    assert np.array_equal(lib_codes, bw["dZq"])
    g, u = oracle.bf16_to_f32(fw["G"]), oracle.bf16_to_f32(fw["U"])
    f = w.f
    for t, i in ((0, 0), (3, 17), (23, 95), (11, 40)):
        du, dg = oracle.swiglu_grad(float(u[t, i]), float(g[t, i]), float(bw["dH"][t, i]))
        assert np.float32(dg) == bw["dZ"][t, i] and np.float32(du) == bw["dZ"][t, f + i]


def test_amax_dz_envelope_of_the_parity_tests():
    """Host logic of the tolerance the GPU tests use for the maximum of dZ: with no storage step the envelope
    collapses onto the oracle's maximum; with one bf16 step it contains it and stays within a few 2^-8."""
    from helpers import amax_dz_bounds, bf16_ulp
    w = wl.make("env", 10, 16, 64, 80, w_std=0.05)
    fw = oracle.forward(w.x, w.W1, w.W2, w.W3)
    bw = oracle.backward(fw, w.dY, want_intermediates=True)
    g, u = oracle.bf16_to_f32(fw["G"]), oracle.bf16_to_f32(fw["U"])
    lo, hi = amax_dz_bounds(g, u, bw["dH"], 0.0 * g, 0.0 * u)
    assert lo == hi and np.isclose(lo, bw["amax_dz"], rtol=1e-6)
    lo, hi = amax_dz_bounds(g, u, bw["dH"], bf16_ulp(g), bf16_ulp(u))
    assert lo <= bw["amax_dz"] <= hi and hi / lo < 1.0 + 8 * 2.0 ** -7


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_code_stats_counts_zero_and_top_codes(fmt):
    """Pins of the code statistics: among all 256 codes exactly two are zero (+0, -0) and two sit at the largest finite
    magnitude; on random values the counts equal those a library cast's values give (value == 0, |value| == format
    maximum); and a quantised tensor scaled to its own maximum has at least one top code and none beyond."""
    allc = np.arange(256, dtype=np.uint8).reshape(16, 16)
    assert oracle.code_stats(fmt, allc) == (2, 2)
    rng = np.random.default_rng(11)
    v = (rng.standard_normal((64, 48)) * rng.choice([1e-9, 1.0, 1e6], (64, 48))).astype(np.float32)
    codes, deq, _ = oracle.quantize(v, fmt, 1.0)
    tdt = torch.float8_e4m3fn if fmt == E4M3 else torch.float8_e5m2
    lib_vals = torch.from_numpy(codes).view(tdt).float().numpy()
    fmax = oracle.fmt_max(fmt)
    assert oracle.code_stats(fmt, codes) == (int(np.sum(lib_vals == 0)), int(np.sum(np.abs(lib_vals) == fmax)))
    assert oracle.code_stats(fmt, codes)[0] > 0 and oracle.code_stats(fmt, codes)[1] > 0      # the draw underflows and saturates
    own = oracle.quantize(v, fmt, oracle.scale_from_amax(fmt, oracle.amax(v)))[0]
    assert oracle.code_stats(fmt, own)[1] >= 1
