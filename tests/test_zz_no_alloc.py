"""fp8mlp_forward_static: the forward for callers that cannot allocate device memory.

Such callers (a plug-in inside an application whose pool owns the whole GPU, a serving loop that
must avoid the stalls of cudaMalloc / cudaFree) have no context; the library's fixed 4 MiB scratch
array takes its place.  This checks, through the C ABI, that the entry point gives what
fp8mlp_forward gives, on two calls in a row (the array keeps the first call's leftovers), and that
shapes beyond the array are refused before anything runs.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

from helpers import bf16_bits_to_f32, bf16_dev_to_bits, nmax_err, to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import build as libbuild
from paper_2409_12517_b200 import workloads as wl

OUT_TOL = 2e-3      # the bar the other parity tests use for outputs


def _forward_with_context(w, flags, mode, sc, am):
    ctx = B.fp8mlp_create(w.T, w.d, w.f, flags)
    try:
        y = torch.zeros((w.T, w.d), dtype=torch.bfloat16, device="cuda")
        B.fp8mlp_forward(ctx, w.T, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3), mode, sc, am, y)
        assert B.fp8mlp_status(ctx) == B.OK
        return bf16_dev_to_bits(y)
    finally:
        B.fp8mlp_destroy(ctx)


@pytest.mark.gpu
def test_static_forward_matches_the_context_forward_twice_in_a_row():
    # two different problems back to back: the second finds the first one's data in the scratch
    problems = [(wl.make_config("tiny"), B.SMOOTH), (wl.make("second", 5, 200, 128, 400, w_std=0.05), B.SMOOTH),
                (wl.make_config("tiny"), 0)]
    for w, flags in problems:
        sc_ref, am_ref = B.new_scales(w.f), B.new_amax(w.f)
        y_ref = _forward_with_context(w, flags, B.SCALE_FROM_CURRENT_AMAX, sc_ref, am_ref)
        for mode in (B.SCALE_FROM_CURRENT_AMAX, B.SCALE_GIVEN):
            sc, am = B.new_scales(w.f), B.new_amax(w.f)
            if mode == B.SCALE_GIVEN:
                for k in sc:
                    sc[k].copy_(sc_ref[k])
            y = torch.full((w.T, w.d), float("nan"), dtype=torch.bfloat16, device="cuda")
            B.fp8mlp_forward_static(w.T, w.d, w.f, flags, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3),
                                    mode, sc, am, y)
            torch.cuda.synchronize()
            got = bf16_bits_to_f32(bf16_dev_to_bits(y))
            assert np.all(np.isfinite(got))
            assert nmax_err(got, bf16_bits_to_f32(y_ref)) <= OUT_TOL
            for k in ("x", "w12", "w3", "h"):
                assert torch.allclose(sc[k], sc_ref[k], rtol=1e-5, atol=0)
            for k in ("x", "w1", "w2", "w3", "h"):
                assert torch.allclose(am[k], am_ref[k], rtol=1e-5, atol=0)


def test_static_forward_rejects_what_does_not_fit():
    libbuild.build()
    L = B.lib()
    n0 = L.fp8mlp_launch_count()
    # the 7B shape needs ~135 MB of FP8 weights alone
    assert L.fp8mlp_forward_static(4096, 4096, 11008, B.SMOOTH, 256, 256, 256, 256, 0, None, None, 256, None) == B.ERR_TOO_LARGE
    assert L.fp8mlp_forward_static(16, 24, 16, B.SMOOTH, 256, 256, 256, 256, 0, None, None, 256, None) == B.ERR_SHAPE
    assert L.fp8mlp_forward_static(16, 16, 16, B.SAVE_FOR_BWD, 256, 256, 256, 256, 0, None, None, 256, None) == B.ERR_ARG
    assert L.fp8mlp_launch_count() == n0
    assert b"scratch" in L.fp8mlp_strerror(B.ERR_TOO_LARGE)
