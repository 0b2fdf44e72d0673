"""fp8mlp_forward_static: the forward for callers that cannot allocate device memory.

Such callers (a plug-in inside an application whose pool owns the whole GPU, a serving loop that
must avoid the stalls of cudaMalloc / cudaFree) have no context; the library's fixed 4 MiB scratch
array takes its place.  This checks, through the C ABI, that the entry point gives exactly what
fp8mlp_forward gives (bit for bit, and within the oracle's bar), on calls in a row (the array keeps the previous
call's leftovers), that a call leaves the amount of free device memory unchanged, and that shapes beyond the
array and bad arguments are refused before anything runs.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f32, bf16_dev_to_bits, nmax_err, to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import build as libbuild
from paper_2409_12517_b200 import workloads as wl

OUT_TOL = 2e-3      # the bar the other parity tests use for outputs against the oracle


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
    """Same kernels on the same data: the result must equal fp8mlp_forward's bit for bit (outputs, scales and
    maxima), in both scale modes, and the first problem's result must also meet the oracle's bar."""
    # different problems back to back: each finds the previous one's data in the scratch
    problems = [(wl.make_config("tiny"), B.SMOOTH), (wl.make("second", 5, 200, 128, 400, w_std=0.05), B.SMOOTH),
                (wl.make_config("tiny"), 0)]
    for n, (w, flags) in enumerate(problems):
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
            got_bits = bf16_dev_to_bits(y)
            assert np.array_equal(got_bits, y_ref), "output differs from fp8mlp_forward's"
            for k in ("x", "w12", "w3", "h"):
                assert torch.equal(sc[k], sc_ref[k]), f"scale {k}"
            for k in ("x", "w1", "w2", "w3", "h"):
                assert torch.equal(am[k], am_ref[k]), f"maximum {k}"
            if n == 0 and mode == B.SCALE_FROM_CURRENT_AMAX:      # and against the CPU oracle, once
                fw = oracle.forward(w.x, w.W1, w.W2, w.W3, flags=oracle.FLAG_SMOOTH)
                assert np.array_equal(sc["h"].cpu().numpy(), fw["s_h"])
                assert nmax_err(bf16_bits_to_f32(got_bits), fw["Y"]) <= OUT_TOL


@pytest.mark.gpu
def test_static_forward_leaves_device_memory_as_it_found_it():
    """The promise to callers that cannot allocate: once the library is loaded and the kernels have run once,
    a call takes no device memory - the free bytes the driver reports are the same before and after."""
    w = wl.make_config("tiny")
    x, W1, W2, W3 = to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3)
    sc, am = B.new_scales(w.f), B.new_amax(w.f)
    y = torch.zeros((w.T, w.d), dtype=torch.bfloat16, device="cuda")
    call = lambda: B.fp8mlp_forward_static(w.T, w.d, w.f, B.SMOOTH, x, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
    call()                                   # warm-up: the runtime loads the kernels and sets the array up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    call()
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, f"device memory in use changed by {free_before - free_after} bytes across the call"
    # a bad argument (here: x not 16-byte aligned, then no scales) is refused before anything is enqueued
    n0 = B.fp8mlp_launch_count()
    with pytest.raises(B.Fp8MlpError) as ei:
        B.fp8mlp_forward_static(w.T, w.d, w.f, B.SMOOTH, x.view(-1)[4:4 + w.T * w.d], W1, W2, W3, B.SCALE_GIVEN, sc, am, y)
    assert ei.value.code == B.ERR_ALIGN
    assert B.lib().fp8mlp_forward_static(w.T, w.d, w.f, B.SMOOTH, x.data_ptr(), W1.data_ptr(), W2.data_ptr(), W3.data_ptr(),
                                         B.SCALE_GIVEN, None, None, y.data_ptr(), None) == B.ERR_ARG
    assert B.fp8mlp_launch_count() == n0


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
