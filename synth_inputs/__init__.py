"""Seeded synthetic inputs for the cached causal Conv3D tests and benchmarks.

This module serves both the CPU oracle and the CUDA path and therefore holds
none of the method's arithmetic: it only draws numbers and rounds them to the
storage type.  Every element is a pure function of (seed, tensor id, flat
element index) through a 64-bit counter-based mixing hash, so any slice of any
tensor can be regenerated without generating the rest.

Storage conventions on the host:
  * fp32 tensors are ``numpy.float32`` arrays;
  * bf16 tensors are ``numpy.uint16`` arrays holding the bf16 bit patterns
    (round-to-nearest-even from the fp32 draw).

Distributions follow the benchmark configurations: ``N(0, a)`` is read with
``a`` as the VARIANCE (weights: variance 1/(Cin*kt*kh*kw), i.e. fan-in scaling;
bias: variance 0.1).
"""
from __future__ import annotations

import math
import numpy as np

F32 = 0
BF16 = 1

# tensor ids (sub-streams); layer l of a chain uses id + 16*l
TID_X, TID_CACHE, TID_W, TID_B = 1, 2, 3, 4

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_CHUNK = 1 << 22


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tid: int, lane: int) -> np.uint64:
    k = (seed * 0x632BE59BD9B4E019 + tid * 0xD1B54A32D192ED03 + lane * 0x8CB92BA72F3D8DD7 + 0x1234567) % (1 << 64)
    return np.uint64(k)


def _uniform01(seed: int, tid: int, lane: int, start: int, count: int) -> np.ndarray:
    """count doubles in (0,1), element i at flat index start+i."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64)
        z = _mix(_mix(idx * _GOLD + _key(seed, tid, lane)))
    return ((z >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def to_bf16_bits(a32: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    bits = np.ascontiguousarray(a32, dtype=np.float32).view(np.uint32)
    r = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b16: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b16, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of a stored tensor (fp32 array or bf16 bit patterns)."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


def _store(vals64: np.ndarray, dtype: int) -> np.ndarray:
    a32 = vals64.astype(np.float32)
    return to_bf16_bits(a32) if dtype == BF16 else a32


def uniform(shape, lo: float, hi: float, dtype: int, seed: int, tid: int) -> np.ndarray:
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if dtype == BF16 else np.float32)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        u = _uniform01(seed, tid, 0, s, c)
        out[s:s + c] = _store(lo + (hi - lo) * u, dtype)
    return out.reshape(shape)


def normal(shape, std: float, dtype: int, seed: int, tid: int) -> np.ndarray:
    """N(0, std^2) by Box-Muller on two independent hashed uniforms per element."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if dtype == BF16 else np.float32)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        u1 = _uniform01(seed, tid, 0, s, c)
        u2 = _uniform01(seed, tid, 1, s, c)
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * math.pi) * u2)
        out[s:s + c] = _store(std * z, dtype)
    return out.reshape(shape)


def zeros(shape, dtype: int) -> np.ndarray:
    return np.zeros(shape, dtype=np.uint16 if dtype == BF16 else np.float32)


def conv_case(N, Cin, Cout, T, H, W, k=(3, 3, 3), dtype=BF16, seed=0, x_dist="normal",
              cache="random", bias=True, layer=0):
    """One causal-conv problem: dict with x, cache, w, b (host arrays) and the sizes.

    x_dist: "normal" -> N(0,1); "uniform" -> U(-1,1) (the fp32 configuration).
    cache : "random" (same distribution as x), "zeros", or None (first chunk).
    """
    kt, kh, kw = k
    off = 16 * layer
    draw = (lambda shp, tid: normal(shp, 1.0, dtype, seed, tid)) if x_dist == "normal" else \
           (lambda shp, tid: uniform(shp, -1.0, 1.0, dtype, seed, tid))
    x = draw((N, Cin, T, H, W), TID_X + off)
    if kt > 1 and cache == "random":
        c = draw((N, Cin, kt - 1, H, W), TID_CACHE + off)
    elif kt > 1 and cache == "zeros":
        c = zeros((N, Cin, kt - 1, H, W), dtype)
    else:
        c = None
    w = normal((Cout, Cin, kt, kh, kw), 1.0 / math.sqrt(Cin * kt * kh * kw), dtype, seed, TID_W + off)
    b = normal((Cout,), math.sqrt(0.1), dtype, seed, TID_B + off) if bias else None
    return dict(x=x, cache=c, w=w, b=b, N=N, Cin=Cin, Cout=Cout, T=T, H=H, W=W, k=k, dtype=dtype)


# The benchmark configurations (sizes only; see conv_case for the distributions).
CONFIGS = {
    "cfg1_f32_16": dict(N=1, Cin=16, Cout=16, T=2, H=16, W=16, k=(3, 3, 3), dtype=F32, x_dist="uniform"),
    "cfg2_bf16_384": dict(N=1, Cin=384, Cout=384, T=1, H=44, W=80, k=(3, 3, 3), dtype=BF16),
    "cfg3_bf16_192": dict(N=1, Cin=192, Cout=192, T=4, H=352, W=640, k=(3, 3, 3), dtype=BF16),
    "cfg4a_bf16_96": dict(N=1, Cin=96, Cout=96, T=4, H=704, W=1280, k=(3, 3, 3), dtype=BF16),
    "cfg4b_bf16_192_96": dict(N=1, Cin=192, Cout=96, T=4, H=704, W=1280, k=(3, 3, 3), dtype=BF16),
    "cfg4c_bf16_pw_192_96": dict(N=1, Cin=192, Cout=96, T=4, H=704, W=1280, k=(1, 1, 1), dtype=BF16),
}


def conv_flops(N, Cin, Cout, T, H, W, k):
    return 2.0 * N * Cout * Cin * k[0] * k[1] * k[2] * T * H * W


def conv_bytes(N, Cin, Cout, T, H, W, k, elem=2, out_elem=2):
    """Algorithmic bytes of one call: x, cache, w, b read once; out, new_cache written once."""
    px = N * H * W
    tc = k[0] - 1
    return (px * Cin * T * elem + 2 * px * Cin * tc * elem + Cout * Cin * k[0] * k[1] * k[2] * elem
            + Cout * elem + px * Cout * T * out_elem)
