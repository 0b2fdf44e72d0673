"""The step gives the same bits every time.

Every kernel of the path is deterministic by construction (maxima by atomic max, split contractions added in a fixed
order, no floating-point atomics), so repeating a step on the same inputs must reproduce every buffer bit for bit.
That makes repetition a detector for races that the parity tests are too coarse to see: a hand-over of shared
memory between the epilogue's loads and the bulk-copy engine that lacked a proxy fence corrupted a few 16-byte
pieces per 10^9 - within every tolerance of a sampled comparison, but never twice the same."""
import pytest
import torch

from paper_2409_12517_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d,f,flags,reps", [
    (16384, 4096, 11008, B.SMOOTH | B.SAVE_FOR_BWD, 60),                 # the benchmark's 7B step
    (8192, 8192, 28672, B.SMOOTH | B.SAVE_FOR_BWD, 30),                  # the 70B shape
    (16384, 4096, 11008, B.SMOOTH | B.SAVE_FOR_BWD | B.GU_FP8, 30),      # saved activations as E4M3 codes
    (512, 4096, 11008, B.SMOOTH | B.SAVE_FOR_BWD, 100),                  # split contractions, staged stores
    (2520, 4048, 1040, B.SAVE_FOR_BWD, 60),                              # ragged tiles, Smooth-SwiGLU off
    (4096, 4096, 11008, B.SAVE_FOR_BWD | B.H_BF16, 30),                  # the last layer in bf16 (16-bit operand path)
])
def test_step_is_bitwise_repeatable(T, d, f, flags, reps):
    gen = torch.Generator(device="cuda").manual_seed(T + f)
    x = torch.randn(T, d, device="cuda", generator=gen).to(torch.bfloat16)
    dy = (torch.randn(T, d, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16)
    W1, W2, W3 = (torch.randn(*s, device="cuda", generator=gen) * 0.02 for s in ((d, f), (d, f), (f, d)))
    y, dx = torch.empty_like(x), torch.empty_like(x)
    dW1, dW2, dW3 = torch.empty_like(W1), torch.empty_like(W2), torch.empty_like(W3)
    ctx = B.fp8mlp_create(T, d, f, flags)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        B.fp8mlp_forward(ctx, T, x, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        B.fp8mlp_backward(ctx, T, dy, B.SCALE_FROM_CURRENT_AMAX, sc, am, dx, dW1, dW2, dW3)
        gu_dtype = torch.uint8 if flags & B.GU_FP8 else torch.int16

        def snapshot():
            ws = lambda which, shape, dt=torch.uint8: B.workspace_tensor(ctx, which, shape, dt)
            h = ws(B.WS_HB, (T, f), torch.int16) if flags & B.H_BF16 else ws(B.WS_HQ, (T, f))
            return dict(H=h, GU=ws(B.WS_GU, (T, 2 * f), gu_dtype), dZq=ws(B.WS_DZQ, (T, 2 * f)),
                        Y=y.view(torch.int16).clone(), dX=dx.view(torch.int16).clone(), dW1=dW1.view(torch.int32).clone(),
                        dW2=dW2.view(torch.int32).clone(), dW3=dW3.view(torch.int32).clone(),
                        maxima=torch.cat([v.view(-1) for v in am.values()]).view(torch.int32).clone())

        first = None
        for rep in range(reps):
            for which in (B.WS_HB if flags & B.H_BF16 else B.WS_HQ, B.WS_GU, B.WS_DZQ):   # nothing survives from the previous repetition
                B.workspace_fill(ctx, which, 0x7F)
            B.fp8mlp_forward(ctx, T, x, W1, W2, W3, B.SCALE_GIVEN, sc, am, y)
            B.fp8mlp_backward(ctx, T, dy, B.SCALE_GIVEN, sc, am, dx, dW1, dW2, dW3)
            torch.cuda.synchronize()
            now = snapshot()
            if first is None:
                first = now
                continue
            for name in now:
                if not torch.equal(now[name], first[name]):
                    where = (now[name] != first[name]).nonzero()
                    raise AssertionError(f"repetition {rep}: {name} differs from the first run in {where.shape[0]} elements, "
                                         f"first at {where[:4].tolist()}")
        assert B.fp8mlp_status(ctx) == B.OK
    finally:
        B.fp8mlp_destroy(ctx)


def test_just_in_time_step_and_merged_forward_are_bitwise_repeatable():
    """The same for the step with every scale derived from the current data (calibration passes, scale kernels) and
    for the inference form on merged weights."""
    T, d, f = 4096, 4096, 11008
    gen = torch.Generator(device="cuda").manual_seed(7)
    x = torch.randn(T, d, device="cuda", generator=gen).to(torch.bfloat16)
    dy = (torch.randn(T, d, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16)
    W1, W2, W3 = (torch.randn(*s, device="cuda", generator=gen) * 0.02 for s in ((d, f), (d, f), (f, d)))
    y, dx = torch.empty_like(x), torch.empty_like(x)
    dW1, dW2, dW3 = torch.empty_like(W1), torch.empty_like(W2), torch.empty_like(W3)
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        first = None
        for rep in range(12):
            for t in (y, dx, dW1, dW2, dW3):
                t.fill_(float("nan"))
            B.fp8mlp_forward(ctx, T, x, W1, W2, W3, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
            B.fp8mlp_backward(ctx, T, dy, B.SCALE_FROM_CURRENT_AMAX, sc, am, dx, dW1, dW2, dW3)
            torch.cuda.synchronize()
            now = [t.view(torch.int16).clone() for t in (y, dx)] + [t.view(torch.int32).clone() for t in (dW1, dW2, dW3)] + \
                  [torch.cat([v.view(-1) for v in list(sc.values()) + list(am.values())]).view(torch.int32).clone()]
            if first is None:
                first = now
            else:
                assert all(torch.equal(a, b) for a, b in zip(now, first)), f"just-in-time step, repetition {rep}"
        s = sc["h"].clone()
        B.fp8mlp_merge_weights(ctx, W1, W2, W3, s, B.SCALE_FROM_CURRENT_AMAX, sc, am)
        B.fp8mlp_forward_merged(ctx, T, x, B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        first = None
        for rep in range(30):
            y.fill_(float("nan"))
            B.fp8mlp_forward_merged(ctx, T, x, B.SCALE_GIVEN, sc, None, y)
            torch.cuda.synchronize()
            now = y.view(torch.int16).clone()
            if first is None:
                first = now
            else:
                assert torch.equal(now, first), f"merged forward, repetition {rep}"
        assert B.fp8mlp_status(ctx) == B.OK
    finally:
        B.fp8mlp_destroy(ctx)
