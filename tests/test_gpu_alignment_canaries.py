"""Pointers that are only 16-byte aligned (what the C ABI promises) and guard zones around every output.

The kernels use 32-byte loads and stores where rows and bases allow it and fall back to 16-byte
accesses otherwise; here every caller-owned tensor starts 16 bytes past a 32-byte boundary, sits
between two guard zones filled with a canary pattern, and the results must equal those of the
aligned run bit for bit with every canary intact (no out-of-bounds write on ragged shapes)."""
import numpy as np
import pytest
import torch

from helpers import to_dev, to_dev_bf16
from paper_2409_12517_b200 import binding as B
from paper_2409_12517_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes on each side
CANARY = 0x5A


class Guarded:
    """A tensor of `shape`/`dtype` carved out of a canary-filled byte buffer, 16 bytes past a 32-byte boundary."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((GUARD + 16 + n + GUARD + 32,), CANARY, dtype=torch.uint8, device="cuda")
        base = self.raw.data_ptr()
        self.off = (-base) % 32 + GUARD + 16            # 32-byte boundary + guard + 16
        self.n = n
        self.t = self.raw[self.off:self.off + n].view(dtype).view(shape)
        assert self.t.data_ptr() % 32 == 16
        if fill is not None:
            self.t.copy_(fill)

    def intact(self):
        before = self.raw[:self.off]
        after = self.raw[self.off + self.n:]
        return bool((before == CANARY).all()) and bool((after == CANARY).all())


def _run(w, aligned):
    T, d, f = w.T, w.d, w.f
    mk = (lambda shape, dt, fill=None: Guarded(shape, dt, fill)) if not aligned else None
    x_src, dy_src = to_dev_bf16(w.x), to_dev_bf16(w.dY)
    W_src = [to_dev(a) for a in (w.W1, w.W2, w.W3)]
    if aligned:
        x, dy, Ws = x_src, dy_src, W_src
        y, dx = torch.zeros_like(x_src), torch.zeros_like(x_src)
        dWs = [torch.zeros_like(a) for a in W_src]
        guards = []
    else:
        gx, gdy = mk((T, d), torch.bfloat16, x_src), mk((T, d), torch.bfloat16, dy_src)
        gW = [mk(tuple(a.shape), torch.float32, a) for a in W_src]
        gy, gdx = mk((T, d), torch.bfloat16), mk((T, d), torch.bfloat16)
        gdW = [mk(tuple(a.shape), torch.float32) for a in W_src]
        x, dy, Ws, y, dx, dWs = gx.t, gdy.t, [g.t for g in gW], gy.t, gdx.t, [g.t for g in gdW]
        guards = [gx, gdy, *gW, gy, gdx, *gdW]
    ctx = B.fp8mlp_create(T, d, f, B.SMOOTH | B.SAVE_FOR_BWD)
    try:
        sc, am = B.new_scales(f), B.new_amax(f)
        B.fp8mlp_forward(ctx, T, x, Ws[0], Ws[1], Ws[2], B.SCALE_FROM_CURRENT_AMAX, sc, am, y)
        B.fp8mlp_backward(ctx, T, dy, B.SCALE_FROM_CURRENT_AMAX, sc, am, dx, dWs[0], dWs[1], dWs[2])
        assert B.fp8mlp_status(ctx) == B.OK
        # Adam on the same (mis)aligned weights and gradients
        n = Ws[0].numel()
        if aligned:
            m, v = torch.zeros(n, dtype=torch.uint8, device="cuda"), torch.zeros(n, dtype=torch.uint8, device="cuda")
        else:
            gm, gv = mk((n,), torch.uint8), mk((n,), torch.uint8)
            gm.t.zero_(); gv.t.zero_()
            m, v = gm.t, gv.t
            guards += [gm, gv]
        one = lambda: torch.ones(1, device="cuda")
        w_adam = Ws[0].clone() if aligned else mk(tuple(Ws[0].shape), torch.float32, Ws[0])
        if not aligned:
            guards.append(w_adam)
            w_adam = w_adam.t
        st = dict(w=w_adam.view(-1), g=dWs[0].view(-1), m=m, v=v, scale_m_in=one(), scale_v_in=one(), scale_m_out=one(),
                  scale_v_out=one(), amax_m=torch.zeros(1, device="cuda"), amax_v=torch.zeros(1, device="cuda"))
        B.fp8mlp_adam_step([st], lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.01, step=1)
        torch.cuda.synchronize()
        out = [t.clone() for t in (y, dx, *dWs, w_adam, m, v)]
    finally:
        B.fp8mlp_destroy(ctx)
    return out, guards


@pytest.mark.parametrize("shape", [(200, 320, 272), (130, 144, 528), (128, 256, 704)])
def test_sixteen_byte_aligned_pointers_and_guard_zones(shape):
    T, d, f = shape
    w = wl.make("al", 41, T, d, f, w_std=0.05, channel_outlier_frac=0.01)
    ref, _ = _run(w, aligned=True)
    got, guards = _run(w, aligned=False)
    for a, b in zip(ref, got):
        assert torch.equal(a.view(torch.uint8), b.contiguous().view(torch.uint8))
    assert all(g.intact() for g in guards), "a guard zone was written"
