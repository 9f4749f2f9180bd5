"""CPU oracle for the cached causal Conv3D (TEST INFRASTRUCTURE ONLY).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product never does.  It wraps ``ccv3d_oracle.c`` (the plain
fp64 definition, Section 4.1-4.2, Eq. (1)-(2)) through ctypes, and adds
restatements of different structure used to pin it:

  * ``brute_force``       - materialises the zero-padded Z volume and loops
                            output-outermost in pure Python/numpy (tiny shapes);
  * ``tap_intervals``     - the interval algebra of Eq. (4) alone (which output
                            frames a temporal tap reaches, and from where), held
                            against direct enumeration of Eq. (1) in the tests.

``forward_general`` / ``brute_force_general`` are the operator with the layer's own
spatial stride, padding, dilation and a temporal dilation (Eq. (1)-(2) as printed).

Host tensors: fp32 arrays, or uint16 arrays of bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ccv3d_oracle.c")
_LIB = os.path.join(_HERE, "libccv3d_oracle.so")

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-o", _LIB + ".tmp", _SRC]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


_lib = None


class _Geom(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "Cin", "Cout", "T", "H", "W", "kt", "kh", "kw", "sh", "sw", "ph", "pw",
                                            "dh", "dw", "dil_t", "cf", "st")]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i, p = ctypes.c_int, ctypes.c_void_p
        lib.ccv3d_oracle_forward.argtypes = [i, p, p, p, p] + [i] * 9 + [p, p]
        lib.ccv3d_oracle_forward.restype = i
        lib.ccv3d_oracle_points.argtypes = [i, p, p, p, p] + [i] * 9 + [p, ctypes.c_int64, p]
        lib.ccv3d_oracle_points.restype = i
        lib.ccv3d_oracle_num_threads.restype = i
        lib.ccv3d_oracle_cache_update.argtypes = [i, p, p] + [i] * 6 + [p]
        lib.ccv3d_oracle_cache_update.restype = i
        lib.ccv3d_oracle_forward_general.argtypes = [i, p, p, p, p, ctypes.POINTER(_Geom), p, p]
        lib.ccv3d_oracle_forward_general.restype = i
        lib.ccv3d_oracle_out_dims.argtypes = [ctypes.POINTER(_Geom), ctypes.POINTER(i), ctypes.POINTER(i), ctypes.POINTER(i)]
        lib.ccv3d_oracle_out_dims.restype = i
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().ccv3d_oracle_num_threads())


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    raise TypeError("oracle tensors are float32 arrays or uint16 bf16 bit patterns")


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _prep(x, cache, w, b):
    dt = _dtype_of(x)
    x = np.ascontiguousarray(x)
    w = np.ascontiguousarray(w)
    assert _dtype_of(w) == dt
    N, Cin, T, H, W = x.shape
    Cout, Cin2, kt, kh, kw = w.shape
    assert Cin2 == Cin
    if cache is not None:
        cache = np.ascontiguousarray(cache)
        assert _dtype_of(cache) == dt and cache.shape == (N, Cin, kt - 1, H, W)
    if b is not None:
        b = np.ascontiguousarray(b)
        assert _dtype_of(b) == dt and b.shape == (Cout,)
    return dt, x, cache, w, b, (N, Cin, Cout, T, H, W, kt, kh, kw)


def forward(x, cache, w, b, want_cache: bool = True):
    """Returns (out float64 [N,Cout,T,H,W], new_cache in the storage dtype or None)."""
    dt, x, cache, w, b, dims = _prep(x, cache, w, b)
    N, Cin, Cout, T, H, W, kt, kh, kw = dims
    out = np.empty((N, Cout, T, H, W), dtype=np.float64)
    nc = np.empty((N, Cin, kt - 1, H, W), dtype=x.dtype) if (want_cache and kt > 1) else None
    rc = _load().ccv3d_oracle_forward(dt, _ptr(x), _ptr(cache), _ptr(w), _ptr(b), *dims, _ptr(out), _ptr(nc))
    if rc != 0:
        raise ValueError("ccv3d_oracle_forward rejected its arguments")
    return out, nc


def points(x, cache, w, b, flat_idx):
    """Oracle value of the sampled output elements flat_idx (into [N,Cout,T,H,W])."""
    dt, x, cache, w, b, dims = _prep(x, cache, w, b)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    vals = np.empty(idx.shape, dtype=np.float64)
    rc = _load().ccv3d_oracle_points(dt, _ptr(x), _ptr(cache), _ptr(w), _ptr(b), *dims, _ptr(idx), idx.size,
                                     _ptr(vals))
    if rc != 0:
        raise ValueError("ccv3d_oracle_points rejected its arguments")
    return vals


def forward_general(x, cache, w, b, stride=(1, 1), pad=None, dil=(1, 1), dil_t=1, want_cache: bool = True, stride_t=1):
    """The operator with the paper's full supported contract (Eq. (1)-(2) with s, p, d and d_t; unit temporal
    stride): spatial stride/padding/dilation per tap, temporal dilation, a cache of up to d_t (kt-1) frames
    (fewer = older history absent).  pad None = ((kh-1) d_h / 2, (kw-1) d_w / 2).  stride_t > 1 (outside the
    paper's method, which rejects it): output frame o reads Z frames o s_t + k d_t, T_o = floor((T-1)/s_t) + 1.
    Returns (out float64 [N,Cout,T_o,H_o,W_o], new_cache [N,Cin,d_t (kt-1),H,W] or None)."""
    dt = _dtype_of(x)
    x, w = np.ascontiguousarray(x), np.ascontiguousarray(w)
    assert _dtype_of(w) == dt
    N, Cin, T, H, W = x.shape
    Cout, Cin2, kt, kh, kw = w.shape
    assert Cin2 == Cin
    if pad is None:
        pad = ((kh - 1) * dil[0] // 2, (kw - 1) * dil[1] // 2)
    tc = dil_t * (kt - 1)
    cf = 0
    if cache is not None and tc > 0:
        cache = np.ascontiguousarray(cache)
        cf = cache.shape[2]
        assert _dtype_of(cache) == dt and cache.shape == (N, Cin, cf, H, W) and 0 < cf <= tc
    else:
        cache = None
    if b is not None:
        b = np.ascontiguousarray(b)
        assert _dtype_of(b) == dt and b.shape == (Cout,)
    g = _Geom(N, Cin, Cout, T, H, W, kt, kh, kw, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1], dil_t, cf, stride_t)
    to, ho, wo = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    if _load().ccv3d_oracle_out_dims(ctypes.byref(g), ctypes.byref(to), ctypes.byref(ho), ctypes.byref(wo)) != 0:
        raise ValueError("bad geometry")
    out = np.empty((N, Cout, to.value, ho.value, wo.value), dtype=np.float64)
    nc = np.empty((N, Cin, tc, H, W), dtype=x.dtype) if (want_cache and tc > 0) else None
    rc = _load().ccv3d_oracle_forward_general(dt, _ptr(x), _ptr(cache), _ptr(w), _ptr(b), ctypes.byref(g), _ptr(out),
                                              _ptr(nc))
    if rc != 0:
        raise ValueError("ccv3d_oracle_forward_general rejected its arguments")
    return out, nc


def brute_force_general(x, cache, w, b, stride=(1, 1), pad=(0, 0), dil=(1, 1), dil_t=1, stride_t=1):
    """The same contract on a materialised, zero-padded Z volume with strided slicing per tap (pure numpy,
    tap-outermost: structurally different from the C routine).  Tiny shapes only."""
    xd, cd, wd, bd = _widen(x), _widen(cache), _widen(w), _widen(b)
    N, Cin, T, H, W = xd.shape
    Cout, _, kt, kh, kw = wd.shape
    tc = dil_t * (kt - 1)
    ph, pw = pad
    Zp = np.zeros((N, Cin, tc + T, H + 2 * ph, W + 2 * pw))
    if cd is not None and tc > 0:
        cf = cd.shape[2]
        Zp[:, :, tc - cf:tc, ph:ph + H, pw:pw + W] = cd
    Zp[:, :, tc:, ph:ph + H, pw:pw + W] = xd
    Ho = (H + 2 * ph - dil[0] * (kh - 1) - 1) // stride[0] + 1
    Wo = (W + 2 * pw - dil[1] * (kw - 1) - 1) // stride[1] + 1
    To = (T - 1) // stride_t + 1
    out = np.zeros((N, Cout, To, Ho, Wo))
    if bd is not None:
        out += bd[None, :, None, None, None]
    for k in range(kt):
        for a in range(kh):
            for c in range(kw):
                src = Zp[:, :, k * dil_t:k * dil_t + (To - 1) * stride_t + 1:stride_t,
                         a * dil[0]:a * dil[0] + (Ho - 1) * stride[0] + 1:stride[0],
                         c * dil[1]:c * dil[1] + (Wo - 1) * stride[1] + 1:stride[1]]          # [N,Cin,T,Ho,Wo]
                out += np.einsum("nithw,oi->nothw", src, wd[:, :, k, a, c])
    Zt = Zp[:, :, :, ph:ph + H, pw:pw + W]
    return out, Zt[:, :, T:T + tc]


def cache_update(x, cache, kt: int):
    """new_cache = last kt-1 frames of [cache ; x] (zeros where there is no history); storage dtype, bit copy."""
    dt = _dtype_of(x)
    x = np.ascontiguousarray(x)
    N, Cin, T, H, W = x.shape
    if cache is not None:
        cache = np.ascontiguousarray(cache)
        assert cache.shape == (N, Cin, kt - 1, H, W) and cache.dtype == x.dtype
    nc = np.empty((N, Cin, kt - 1, H, W), dtype=x.dtype)
    rc = _load().ccv3d_oracle_cache_update(dt, _ptr(x), _ptr(cache), N, Cin, T, H, W, kt, _ptr(nc))
    if rc != 0:
        raise ValueError("ccv3d_oracle_cache_update rejected its arguments")
    return nc


# --------------------------------------------------------------------------------------
# Second opinions (pure numpy / Python, float64, tiny shapes only)
# --------------------------------------------------------------------------------------
def _widen(a):
    if a is None:
        return None
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def brute_force(x, cache, w, b):
    """Definition evaluated on a materialised zero-padded Z volume, output-outermost."""
    xd, cd, wd, bd = _widen(x), _widen(cache), _widen(w), _widen(b)
    N, Cin, T, H, W = xd.shape
    Cout, _, kt, kh, kw = wd.shape
    ph, pw = (kh - 1) // 2, (kw - 1) // 2
    Zp = np.zeros((N, Cin, kt - 1 + T, H + 2 * ph, W + 2 * pw))
    if cd is not None and kt > 1:
        Zp[:, :, :kt - 1, ph:ph + H, pw:pw + W] = cd
    Zp[:, :, kt - 1:, ph:ph + H, pw:pw + W] = xd
    out = np.zeros((N, Cout, T, H, W))
    for n in range(N):
        for co in range(Cout):
            for t in range(T):
                for h in range(H):
                    for ww in range(W):
                        patch = Zp[n, :, t:t + kt, h:h + kh, ww:ww + kw]
                        out[n, co, t, h, ww] = (bd[co] if bd is not None else 0.0) + float(np.sum(patch * wd[co]))
    Zt = Zp[:, :, :, ph:ph + H, pw:pw + W]
    return out, Zt[:, :, T:T + kt - 1]


def tap_intervals(kt: int, cache_frames: int, T: int, dil_t: int = 1):
    """Eq. (4): per temporal tap k the valid output interval [o_l, o_h) and its
    source interval [z_l, z_h) in Z = [C ; X], with p_l^base = d_t (kt-1),
    p_l = p_l^base - |C|, p_r = 0 and unit temporal stride.  Returns (T_o, list)."""
    p_base = dil_t * (kt - 1)
    p_l = p_base - cache_frames
    zlen = cache_frames + T
    T_o = (zlen + p_l + 0 - dil_t * (kt - 1) - 1) // 1 + 1
    taps = []
    for k in range(kt):
        delta = k * dil_t - p_l
        o_l = max(0, -delta)
        o_h = min(T_o, zlen - delta)
        taps.append((k, o_l, o_h, o_l + delta, o_h + delta))
    return T_o, taps
