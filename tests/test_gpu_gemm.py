"""Parity of the tcgen05 FP8 GEMM (all four operand layouts, mixed formats, ragged tiles)
with the oracle's sequential fp32 GEMM on the decoded operands."""
import numpy as np
import pytest
import torch

import oracle
from helpers import nmax_err, to_dev
from paper_2409_12517_b200 import binding as B

pytestmark = pytest.mark.gpu

# Every product of two FP8 values is exact in fp32, so only the accumulation order differs
# between the tensor core and the sequential oracle: K * 2^-24 relative to sum |a||b| at worst.
TOL = 2e-5


def _codes(rng, shape, fmt):
    top = 0x7E if fmt == B.E4M3 else 0x7B
    mag = rng.integers(0, top + 1, shape).astype(np.uint8)
    sign = (rng.integers(0, 2, shape) << 7).astype(np.uint8)
    return mag | sign


def _run(M, N, K, a_k, b_k, a_fmt, b_fmt, seed, scale=True):
    rng = np.random.default_rng(seed)
    # moderate magnitudes so that sums stay far from fp32 overflow: restrict exponents
    A = _codes(rng, (M, K), a_fmt) if a_k else _codes(rng, (K, M), a_fmt)
    Bm = _codes(rng, (N, K), b_fmt) if b_k else _codes(rng, (K, N), b_fmt)
    if a_fmt == B.E5M2:
        A &= np.uint8(0xBF)     # clear the top exponent bit: |v| < 2
    if b_fmt == B.E5M2:
        Bm &= np.uint8(0xBF)
    Af = oracle.decode(a_fmt, A)
    Bf = oracle.decode(b_fmt, Bm)
    Amk = Af if a_k else Af.T                 # [M, K] view
    Bkn = Bf.T if b_k else Bf                 # [K, N] view
    ref = oracle.gemm(Amk, Bkn)
    sa = torch.tensor([3.0], device="cuda") if scale else None
    sb = torch.tensor([0.7], device="cuda") if scale else None
    if scale:
        dq = np.float32(np.float32(1.0) / np.float32(3.0)) * np.float32(np.float32(1.0) / np.float32(0.7))
        ref = ref * np.float32(dq)
    out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    B.fp8mlp_gemm_fp8(M, N, K, to_dev(A), a_k, a_fmt, to_dev(Bm), b_k, b_fmt, sa, sb, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.all(np.isfinite(got)), "unwritten or non-finite outputs"
    return nmax_err(got, ref), got, ref


@pytest.mark.parametrize("a_k,b_k", [(True, True), (True, False), (False, False), (False, True)])
@pytest.mark.parametrize("shape", [(128, 256, 128), (16, 16, 16), (144, 272, 400), (384, 768, 1024)])
def test_gemm_layouts(a_k, b_k, shape):
    M, N, K = shape
    err, _, _ = _run(M, N, K, a_k, b_k, B.E4M3, B.E4M3, seed=M + N + K)
    assert err <= TOL, f"normalised max error {err}"


@pytest.mark.parametrize("a_fmt,b_fmt", [(B.E5M2, B.E4M3), (B.E4M3, B.E5M2), (B.E5M2, B.E5M2)])
@pytest.mark.parametrize("a_k,b_k", [(True, True), (False, False)])
def test_gemm_mixed_formats(a_fmt, b_fmt, a_k, b_k):
    err, _, _ = _run(256, 256, 256, a_k, b_k, a_fmt, b_fmt, seed=7)
    assert err <= TOL, f"normalised max error {err}"


def test_gemm_many_tiles_persistent_loop_and_long_k():
    """More tiles than SMs (each CTA loops over several tiles, both accumulators in use) and a
    contraction long enough to wrap the shared-memory ring many times."""
    err, _, _ = _run(2176, 2560, 2304, True, False, B.E4M3, B.E4M3, seed=1, scale=False)
    assert err <= TOL, f"normalised max error {err}"
    err, _, _ = _run(128, 256, 16384, False, False, B.E4M3, B.E5M2, seed=2)
    assert err <= 8 * TOL, f"normalised max error {err}"
