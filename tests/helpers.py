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
        assert nmax_err(dv, rv) <= out_tol, f"{name}: decoded difference {nmax_err(dv, rv)}"
