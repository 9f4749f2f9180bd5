"""Streamed synthetic decoder chain built on the ccv3d C-ABI (every arithmetic step runs in the library).

Three resolution stages of a causal video-VAE-decoder-shaped stack, BF16 between layers, per-layer temporal
caches carried across chunks:

    stage A (C_a ch, H x W,   T frames):   a <- a + convA2(convA1(a))
    1x1x1 conv C_a -> C_b, nearest 2x spatial upsample, each frame repeated 4x
    stage B (C_b ch, 2H x 2W, 4T frames):  b <- b + convB2(convB1(b))
    1x1x1 conv C_b -> C_c, nearest 2x spatial upsample
    stage C (C_c ch, 4H x 4W, 4T frames):  c <- c + convC2(convC1(c))

The six 3x3x3 convolutions are cached causal convolutions (zero history before the first chunk).  No
normalisation or non-linearity: the chain exists to exercise streaming, caches and layer shapes.
"""
from __future__ import annotations

from . import CausalConv3d, Ccv3dError, OK, ccv3d_add_bf16, ccv3d_upsample_bf16

LAYERS = ("A1", "A2", "PA", "B1", "B2", "PB", "C1", "C2")


class DecoderChain:
    def __init__(self, weights: dict, biases: dict):
        """weights/biases: dicts over LAYERS of contiguous CUDA BF16 tensors ([Cout,Cin,kt,kh,kw] / [Cout])."""
        import torch
        self.torch = torch
        self.layers = {n: CausalConv3d(weights[n], biases[n]) for n in LAYERS}
        self.reset()

    def reset(self):
        """Forget all temporal state (next chunk is a first chunk)."""
        self.caches = {n: None for n in LAYERS}

    def _conv(self, name, x):
        out, new_cache = self.layers[name](x, self.caches[name])
        self.caches[name] = new_cache          # a fresh buffer every call: the old cache is never overwritten in place
        return out

    def _add(self, a, b):
        y = self.torch.empty_like(a)
        s = ccv3d_add_bf16(a.data_ptr(), b.data_ptr(), y.data_ptr(), a.numel(),
                           self.torch.cuda.current_stream().cuda_stream)
        if s != OK:
            raise Ccv3dError(s, "ccv3d_add_bf16")
        return y

    def _up(self, x, rt):
        N, C, T, H, W = x.shape
        y = self.torch.empty((N, C, T * rt, 2 * H, 2 * W), dtype=x.dtype, device=x.device)
        s = ccv3d_upsample_bf16(x.data_ptr(), y.data_ptr(), N, C, T, H, W, rt,
                                self.torch.cuda.current_stream().cuda_stream)
        if s != OK:
            raise Ccv3dError(s, "ccv3d_upsample_bf16")
        return y

    def step(self, a):
        """One chunk: a [N,C_a,T,H,W] BF16 -> [N,C_c,4T,4H,4W] BF16."""
        a = self._add(a, self._conv("A2", self._conv("A1", a)))
        b = self._up(self._conv("PA", a), 4)
        b = self._add(b, self._conv("B2", self._conv("B1", b)))
        c = self._up(self._conv("PB", b), 1)
        c = self._add(c, self._conv("C2", self._conv("C1", c)))
        return c

    def close(self):
        for l in self.layers.values():
            l.close()
