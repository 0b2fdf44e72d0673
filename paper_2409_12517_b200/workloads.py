"""Seeded synthetic inputs for the FP8 Smooth-SwiGLU MLP block.

This module only *draws inputs*; it holds none of the method's arithmetic (no FP8
encoding, no scaling, no SwiGLU).  Both the CPU oracle's tests and the CUDA path's
tests feed on it so that they see identical bits.

The paper trains Llama2 on a public web corpus; those activations and trained weights
are not available, so the inputs here stand in for them: Gaussian activations and
weights at the Llama2 MLP shapes, plus the outlier structure the paper describes for
late training (Section 4.2, Theorem 1 and the weight-correlation figures): a few d_ff
channels whose linear-branch column w1_i is aligned with the gate column w2_i and has
a larger norm, so that the SwiGLU output of those channels is far above typical.

Generator: counter-based.  Element n of stream s under seed k is a pure function of
(k, s, n): a SplitMix64 finaliser of the counter gives 2x24 uniform bits, Box-Muller
turns them into one normal deviate (fp64 maths), which is then rounded to the stated
dtype (bf16 by round-to-nearest-even, carried as uint16 bit patterns; or fp32).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# stream ids
_S_X, _S_W1, _S_W2, _S_W3, _S_DY, _S_CH, _S_TOK = 1, 2, 3, 4, 5, 6, 7


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed) * _GOLDEN + np.uint64(stream)], dtype=np.uint64))
    return k[0]


def raw_bits(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """64 random bits for counters start .. start+count-1 of a stream."""
    with np.errstate(over="ignore"):
        n = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        return _mix(_key(seed, stream) + n * _GOLDEN)


def _normals_chunk(seed: int, stream: int, lo: int, c: int, std: float, out: np.ndarray) -> None:
    r = raw_bits(seed, stream, lo, c)
    u1 = ((r >> np.uint64(40)).astype(np.float64) + 1.0) * (1.0 / 16777216.0)  # (0, 1]
    u2 = ((r >> np.uint64(8)) & np.uint64(0xFFFFFF)).astype(np.float64) * (1.0 / 16777216.0)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    out[lo:lo + c] = (z * std).astype(np.float32)


def normals(seed: int, stream: int, count: int, std: float = 1.0, chunk: int = 1 << 20) -> np.ndarray:
    """count normal deviates N(0, std^2) as float32 (Box-Muller on 24-bit uniforms).

    Chunks are independent (counter-based), so large draws are spread over host threads;
    the result does not depend on the number of threads.
    """
    out = np.empty(count, dtype=np.float32)
    starts = list(range(0, count, chunk))
    if len(starts) <= 2:
        for lo in starts:
            _normals_chunk(seed, stream, lo, min(chunk, count - lo), std, out)
        return out
    from concurrent.futures import ThreadPoolExecutor
    import os
    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as pool:
        list(pool.map(lambda lo: _normals_chunk(seed, stream, lo, min(chunk, count - lo), std, out), starts))
    return out


def f32_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(v, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    with np.errstate(over="ignore"):
        r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _pick(seed: int, stream: int, population: int, count: int) -> np.ndarray:
    """count distinct indices out of population, chosen by smallest hash (seeded)."""
    if count <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.argsort(raw_bits(seed, stream, 0, population), kind="stable")
    return np.sort(order[:count]).astype(np.int64)


@dataclass
class Workload:
    name: str
    seed: int
    T: int
    d: int
    f: int
    x: np.ndarray            # uint16 bf16 bits [T, d]
    W1: np.ndarray           # float32 [d, f]  linear branch
    W2: np.ndarray           # float32 [d, f]  gate (Swish) branch
    W3: np.ndarray           # float32 [f, d]  last linear layer
    dY: np.ndarray | None    # uint16 bf16 bits [T, d]
    outlier_channels: np.ndarray = field(default_factory=lambda: np.zeros(0, dtype=np.int64))
    outlier_tokens: np.ndarray = field(default_factory=lambda: np.zeros(0, dtype=np.int64))


def make(name: str, seed: int, T: int, d: int, f: int, *, w_std: float = 0.02,
         channel_outlier_frac: float = 0.0, channel_gain: float = 8.0,
         token_outlier_frac: float = 0.0, token_gain: float = 50.0,
         dy_std: float = 1e-3, with_dy: bool = True) -> Workload:
    """Draw one workload.

    x ~ N(0,1) in bf16 (a fraction token_outlier_frac of the rows multiplied by token_gain
    before rounding); W1, W2, W3 ~ N(0, w_std^2) in fp32, except that in a fraction
    channel_outlier_frac of the d_ff channels column i of W1 is channel_gain * column i
    of W2; dY ~ N(0, dy_std^2) in bf16.
    """
    x = normals(seed, _S_X, T * d).reshape(T, d)
    toks = _pick(seed, _S_TOK, T, int(np.floor(token_outlier_frac * T)))
    if toks.size:
        x[toks, :] *= np.float32(token_gain)
    W1 = normals(seed, _S_W1, d * f, w_std).reshape(d, f)
    W2 = normals(seed, _S_W2, d * f, w_std).reshape(d, f)
    W3 = normals(seed, _S_W3, f * d, w_std).reshape(f, d)
    chans = _pick(seed, _S_CH, f, int(np.floor(channel_outlier_frac * f)))
    if chans.size:
        W1[:, chans] = np.float32(channel_gain) * W2[:, chans]
    dY = f32_to_bf16_bits(normals(seed, _S_DY, T * d, dy_std)).reshape(T, d) if with_dy else None
    return Workload(name, seed, T, d, f, f32_to_bf16_bits(x).reshape(T, d), W1, W2, W3, dY, chans, toks)


# The benchmark configurations (shapes, distributions and seeds as the benchmark
# definition states them).  "sweep" entries are the token-count sweep at the 7B shape.
CONFIGS = {
    "tiny":       dict(seed=0, T=128,   d=256,  f=704),
    "7b_fwd":     dict(seed=1, T=4096,  d=4096, f=11008, channel_outlier_frac=0.001, with_dy=False),
    "7b":         dict(seed=2, T=16384, d=4096, f=11008, channel_outlier_frac=0.001),
    "70b":        dict(seed=3, T=8192,  d=8192, f=28672, w_std=0.01, channel_outlier_frac=0.0005),
    "sweep_512":  dict(seed=4, T=512,   d=4096, f=11008, token_outlier_frac=0.01),
    "sweep_2048": dict(seed=5, T=2048,  d=4096, f=11008, token_outlier_frac=0.01),
    "sweep_8192": dict(seed=6, T=8192,  d=4096, f=11008, token_outlier_frac=0.01),
    "sweep_32768": dict(seed=7, T=32768, d=4096, f=11008, token_outlier_frac=0.01),
}


def make_config(name: str, **override) -> Workload:
    kw = dict(CONFIGS[name])
    kw.update(override)
    return make(name, **kw)
