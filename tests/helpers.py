"""Shared helpers of the parity tests (no method arithmetic: comparisons and marshalling only)."""
import numpy as np
import torch


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def bf16_dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def code_rank(codes: np.ndarray) -> np.ndarray:
    """FP8 codes (sign-magnitude) -> integers that order like the values they encode."""
    c = codes.astype(np.int32)
    mag = c & 0x7F
    return np.where(c & 0x80, -mag, mag)


def code_mismatch(got: np.ndarray, ref: np.ndarray):
    """(fraction of differing codes, largest distance in code steps)."""
    diff = np.abs(code_rank(got) - code_rank(ref))
    return float(np.count_nonzero(diff)) / max(diff.size, 1), int(diff.max()) if diff.size else 0


def nmax_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |got - ref| / max |ref|."""
    ref = ref.astype(np.float64)
    denom = np.abs(ref).max()
    return float(np.abs(got.astype(np.float64) - ref).max() / (denom if denom > 0 else 1.0))


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_ulp(v: np.ndarray) -> np.ndarray:
    """Spacing of bf16 values (8 significant bits) at the magnitude of v."""
    a = np.abs(v.astype(np.float64))
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def nmax_err_bf16(got_bits: np.ndarray, ref: np.ndarray) -> float:
    """Normalised max error of a bf16 output against the oracle's, net of the output rounding:
    two fp32 results within eps of each other round to bf16 values at most eps + one bf16 spacing
    apart, so one spacing is granted per element and the rest is held to the bar on eps."""
    got = bf16_bits_to_f32(got_bits).astype(np.float64)
    ref = ref.astype(np.float64)
    excess = np.maximum(np.abs(got - ref) - bf16_ulp(ref), 0.0)
    denom = np.abs(ref).max()
    return float(excess.max() / (denom if denom > 0 else 1.0))


def frac_beyond(got: np.ndarray, ref: np.ndarray, tol: float) -> float:
    """Fraction of elements whose error exceeds tol * max |ref|."""
    ref = ref.astype(np.float64)
    return float(np.mean(np.abs(got.astype(np.float64) - ref) > tol * np.abs(ref).max()))


def check_dz_codes(name, got, ref, code_frac=1e-3, out_tol=2e-3):
    """E5M2 codes of [dG | dU] against the oracle's.  They inherit the accumulation-order differences like
    Hq does (one code step, rarely), and one more: the saved bf16 G and U may themselves differ by one bf16
    spacing between the two sides, and near the zero of the gate derivative (G about -1.28) that moves a
    small dG by more than one of its own code steps.  So: few codes differ at all, hardly any by more than
    one step, and every such difference is small against the tensor (the bar for gradient values)."""
    import oracle
    frac, worst = code_mismatch(got, ref)
    assert frac <= code_frac, f"{name}: {frac:.2e} of the codes differ"
    if worst > 1:
        many = float(np.mean(np.abs(code_rank(got) - code_rank(ref)) > 1))
        assert many <= 2e-5, f"{name}: {many:.2e} of the codes differ by more than one step"
        dv, rv = oracle.decode(oracle.E5M2, got), oracle.decode(oracle.E5M2, ref)
        far = np.argwhere(np.abs(code_rank(got) - code_rank(ref)) > 1)
        worst_at = np.unravel_index(np.argmax(np.abs(dv.astype(np.float64) - rv)), dv.shape)
        assert nmax_err(dv, rv) <= out_tol, (f"{name}: decoded difference {nmax_err(dv, rv)} at {worst_at}: got {dv[worst_at]} "
                                             f"ref {rv[worst_at]}, max |ref| {np.abs(rv).max()}; {len(far)} codes beyond one step, first at {far[:8].tolist()}")


def amax_dz_bounds(g, u, dh, g_step, u_step):
    """[lo, hi] for max(|dG|, |dU|) when every saved activation may sit one storage step beside the oracle's.

    The CUDA path keeps G and U rounded (bf16, or E4M3 codes) from fp32 values that differ from the oracle's in
    accumulation order only; where the two fp32 values straddle a rounding boundary the stored values are one
    step apart, and the gate derivative carries that step into dG, dU.  So the maximum is not held to the
    accumulation-order bar directly but to this envelope: per element the smallest and largest |dG|, |dU| over
    g in {g - step, g, g + step} x u in {u - step, u, u + step} (fp64), then the maximum over elements of each.
    Callers pass a step of zero wherever the stored value equals the oracle's, so the envelope only opens at the
    (rare) elements that really differ; elsewhere lo and hi coincide and the bar is the plain one.
    g, u, dh: the oracle's saved activations and dH; g_step, u_step: the storage spacing granted per element."""
    g, u, dh = (np.asarray(a, np.float64) for a in (g, u, dh))
    g_step, u_step = np.asarray(g_step, np.float64), np.asarray(u_step, np.float64)
    lo_e = np.full(g.shape, np.inf)
    hi_e = np.zeros(g.shape)
    for sg in (-1.0, 0.0, 1.0):
        gg = g + sg * g_step
        sig = 1.0 / (1.0 + np.exp(-gg))
        du = np.abs(dh * gg * sig)
        gate = sig * (1.0 + gg * (1.0 - sig))
        for su in (-1.0, 0.0, 1.0):
            dg = np.abs(dh * (u + su * u_step) * gate)
            m = np.maximum(du, dg)
            lo_e = np.minimum(lo_e, m)
            hi_e = np.maximum(hi_e, m)
    return float(lo_e.max()), float(hi_e.max())


def check_amax_dz(name, got, bw, g, u, g_step, u_step, rtol=1e-5, lower_only=False):
    """amax of dZ = [dG | dU] against the oracle's, by the envelope of amax_dz_bounds widened by the
    accumulation-order bar.  The envelope's centre is first checked against the oracle's own maximum (so the
    formula retyped there cannot drift from the oracle's).  lower_only: `got` is the maximum over a superset
    of the oracle's elements (a global maximum against a sample's)."""
    centre = float(np.abs(bw["dZ"]).max())
    assert np.isclose(centre, bw["amax_dz"], rtol=1e-6), f"{name}: oracle maximum {bw['amax_dz']} vs its dZ {centre}"
    lo, hi = amax_dz_bounds(g, u, bw["dH"], g_step, u_step)
    assert lo <= centre * (1 + 1e-6) and hi >= centre * (1 - 1e-6), f"{name}: envelope [{lo}, {hi}] misses {centre}"
    assert got >= lo * (1 - rtol), f"{name}: {got} below the envelope [{lo}, {hi}] of the oracle's {centre}"
    if not lower_only:
        assert got <= hi * (1 + rtol), f"{name}: {got} above the envelope [{lo}, {hi}] of the oracle's {centre}"
    return dict(got=float(got), oracle=centre, lo=lo, hi=hi)


def e4m3_step(v):
    """Spacing of E4M3 values (4 significant bits, subnormal spacing 2^-9) at the magnitude of v."""
    a = np.abs(np.asarray(v, np.float64))
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    return 2.0 ** (e - 3)


# figures the parity tests measured (see conftest.py: printed at the end of the session)
PARITY_FIGURES = []


def record_parity(test: str, **figures):
    PARITY_FIGURES.append(dict(test=test, **{k: (float(v) if isinstance(v, (np.floating, float)) else v) for k, v in figures.items()}))


def code_diff(fmt, got_codes, ref_codes):
    """dec(got) - dec(ref) in fp64: zero wherever the two sides stored the same code."""
    import oracle
    return oracle.decode(fmt, got_codes).astype(np.float64) - oracle.decode(fmt, ref_codes).astype(np.float64)
