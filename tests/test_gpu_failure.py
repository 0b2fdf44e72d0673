"""The failure path on the GPU, without faulting or hanging anything: every wait inside the kernels
is bounded; a wait that runs out raises the context's status word and the kernel ends normally.
The self-test kernel waits on a barrier that nothing completes (a flag that nothing sets)."""
import time

import pytest
import torch

from helpers import to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_reports_timeout_and_leaves_the_context_usable():
    w = wl.make_config("tiny")
    ctx = B.fp8mlp_create(w.T, w.d, w.f, B.SMOOTH)
    try:
        assert B.fp8mlp_status(ctx) == B.OK
        t0 = time.time()
        B.fp8mlp_selftest_wait_timeout(ctx, 20000)                 # 20 ms limit
        assert time.time() - t0 < 5.0
        assert B.fp8mlp_status(ctx) == B.ERR_TIMEOUT               # reported once ...
        assert B.fp8mlp_status(ctx) == B.OK                        # ... and cleared
        # the CUDA context and this library context still work
        sc, am = B.new_scales(w.f), B.new_amax(w.f)
        y = torch.zeros((w.T, w.d), dtype=torch.bfloat16, device="cuda")
        B.fp8mlp_forward(ctx, w.T, to_dev_bf16(w.x), to_dev(w.W1), to_dev(w.W2), to_dev(w.W3),
                         B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        assert B.fp8mlp_status(ctx) == B.OK
        assert bool(torch.isfinite(y.float()).all()) and float(y.float().abs().max()) > 0
        with pytest.raises(B.Fp8MlpError):
            B.fp8mlp_selftest_wait_timeout(ctx, 0)                 # limit out of range: refused before any launch
    finally:
        B.fp8mlp_destroy(ctx)
