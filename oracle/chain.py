"""Oracle of the streamed synthetic decoder chain (TEST INFRASTRUCTURE ONLY).

Quantisation-matched: every convolution is the FP64 definition (oracle.forward) followed by one
round-to-nearest-even to BF16, every residual add is an exact FP64 sum of two BF16 values followed by one RNE to
BF16, and the glue (nearest-neighbour 2x upsample, frame repeat) moves values exactly - the points at which
the GPU chain stores BF16.  Host tensors are uint16 BF16 bit patterns.
"""
import numpy as np

from . import forward

LAYERS = ("A1", "A2", "PA", "B1", "B2", "PB", "C1", "C2")


def _f64_to_bf16_bits(a):
    """float64 -> bf16 bit patterns, round to nearest even, decided on the double itself (going through float32
    first would round twice)."""
    a = np.ascontiguousarray(a, dtype=np.float64)
    trunc = a.astype(np.float32).view(np.uint32) & np.uint32(0xFFFF0000)      # a bf16 neighbour of a
    # the two bf16 values that bracket |a| around that neighbour
    n0 = trunc.view(np.float32).astype(np.float64)
    n_up = (trunc + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    n_dn = (trunc - np.uint32(0x10000)).view(np.float32).astype(np.float64)
    aa = np.abs(a)
    lo_is_dn = np.abs(n0) > aa                       # float32 rounding went up past a: bracket is [n_dn, n0]
    lo = np.where(lo_is_dn, n_dn, n0)
    hi = np.where(lo_is_dn, n0, n_up)
    lo_bits = np.where(lo_is_dn, trunc - np.uint32(0x10000), trunc)
    mid = 0.5 * (np.abs(lo) + np.abs(hi))
    lo_odd = ((lo_bits >> np.uint32(16)) & np.uint32(1)) == 1
    up = (aa > mid) | ((aa == mid) & lo_odd)
    out = np.where(up, lo_bits + np.uint32(0x10000), lo_bits)
    return (out >> np.uint32(16)).astype(np.uint16)


def _bf16_to_f64(b):
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _add(a, b):
    return _f64_to_bf16_bits(_bf16_to_f64(a) + _bf16_to_f64(b))


def _up(x, rt):
    return np.ascontiguousarray(np.repeat(np.repeat(np.repeat(x, rt, axis=2), 2, axis=3), 2, axis=4))


class ChainOracle:
    def __init__(self, weights, biases, trace=None):
        """trace: optional list that receives (layer, x, cache_in, out_bf16, new_cache) of every convolution call."""
        self.w, self.b = weights, biases
        self.trace = trace
        self.reset()

    def reset(self):
        self.caches = {n: None for n in LAYERS}

    def _conv(self, name, x):
        x = np.ascontiguousarray(x)
        out, nc = forward(x, self.caches[name], self.w[name], self.b[name])
        ob = _f64_to_bf16_bits(out)
        if self.trace is not None:
            self.trace.append((name, x, self.caches[name], ob, nc))
        self.caches[name] = nc
        return ob

    def step(self, a):
        a = _add(a, self._conv("A2", self._conv("A1", a)))
        b = _up(self._conv("PA", a), 4)
        b = _add(b, self._conv("B2", self._conv("B1", b)))
        c = _up(self._conv("PB", b), 1)
        c = _add(c, self._conv("C2", self._conv("C1", c)))
        return c
