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

import ctypes
import math
import os
import subprocess

import numpy as np

F32 = 0
BF16 = 1

# tensor ids (sub-streams); layer l of a chain uses id + 16*l
TID_X, TID_CACHE, TID_W, TID_B = 1, 2, 3, 4

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libsynth_inputs.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the generator (gcc, OpenMP, no fast-math); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB + ".tmp", _SRC, "-lm"],
                       check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _fill(shape, kind: int, a: float, b: float, dtype: int, seed: int, tid: int) -> np.ndarray:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.synth_fill.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_double,
                                    ctypes.c_double, ctypes.c_int, ctypes.c_uint64, ctypes.c_uint64]
        _lib.synth_fill.restype = None
    out = np.empty(shape, dtype=np.uint16 if dtype == BF16 else np.float32)
    _lib.synth_fill(out.ctypes.data_as(ctypes.c_void_p), 0, out.size, kind, a, b, dtype, seed, tid)
    return out


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


def uniform(shape, lo: float, hi: float, dtype: int, seed: int, tid: int) -> np.ndarray:
    return _fill(shape, 0, lo, hi, dtype, seed, tid)


def normal(shape, std: float, dtype: int, seed: int, tid: int) -> np.ndarray:
    """N(0, std^2) by Box-Muller on two independent hashed uniforms per element."""
    return _fill(shape, 1, std, 0.0, dtype, seed, tid)


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
