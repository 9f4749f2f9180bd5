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

from . import CausalConv3d, Ccv3dError, FrameRing, OK, ccv3d_add_bf16, ccv3d_upsample_bf16

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


class ResidentDecoderChain:
    """The same chain with every activation between the chunk input and the chunk output resident in frame rings
    (channels-last blocks, the order the tensor-core kernel reads): a layer writes straight into the next layer's
    ring, the temporal history of a layer is whatever earlier chunks left in its ring (no cache tensors, no cache
    update), the residual additions run in the convolution epilogues and the two upsamples in the stores of the
    1x1x1 layers.  Per chunk: one layout move for the input and eight convolution kernels.  Results are
    bit-identical to DecoderChain."""

    def __init__(self, weights: dict, biases: dict):
        import torch
        self.torch = torch
        self.layers = {n: CausalConv3d(weights[n], biases[n]) for n in LAYERS}
        self.ch = {n: (weights[n].shape[1], weights[n].shape[0]) for n in LAYERS}   # (cin, cout)
        self.geom = None
        self.reset()

    def reset(self):
        """Forget all temporal state (next chunk is a first chunk)."""
        self.seen = 0            # latent frames consumed since the last reset
        self.slot = {"A": 0, "B": 0, "C": 0}

    def _alloc(self, N, T, H, W):
        ca, cb, cc = self.ch["A1"][0], self.ch["B1"][0], self.ch["C1"][0]
        R = FrameRing
        self.rings = {
            "A1": R(N, ca, T + 2, H, W), "A2": R(N, ca, T + 2, H, W), "PA": R(N, ca, T, H, W),
            "B1": R(N, cb, 4 * T + 2, 2 * H, 2 * W), "B2": R(N, cb, 4 * T + 2, 2 * H, 2 * W),
            "PB": R(N, cb, 4 * T, 2 * H, 2 * W),
            "C1": R(N, cc, 4 * T + 2, 4 * H, 4 * W), "C2": R(N, cc, 4 * T + 2, 4 * H, 4 * W),
        }
        self.geom = (N, T, H, W)

    def _block(self, first, second, nxt, slot, hist, T, out=None):
        """x <- x + conv2(conv1(x)) with x in ring `first`: the sum goes to ring `nxt` (slot 0) or to NCTHW `out`."""
        r, L = self.rings, self.layers
        L[first].forward_ring(r[first], slot, hist, T, out_ring=r[second], out_slot=slot)
        if out is None:
            L[second].forward_ring(r[second], slot, hist, T, out_ring=r[nxt], out_slot=0, res=r[first], res_slot=slot)
        else:
            L[second].forward_ring(r[second], slot, hist, T, out=out, res=r[first], res_slot=slot)

    def step(self, a, out=None):
        """One chunk: a [N,C_a,T,H,W] BF16 -> [N,C_c,4T,4H,4W] BF16 (T at most the first chunk's T after a reset
        or a change of geometry)."""
        N, C, T, H, W = a.shape
        if self.geom is None or self.geom[0] != N or self.geom[2:] != (H, W) or T > self.geom[1]:
            self._alloc(N, T, H, W)
            self.reset()
        r, L = self.rings, self.layers
        if out is None:
            out = self.torch.empty((N, self.ch["C2"][1], 4 * T, 4 * H, 4 * W), dtype=a.dtype, device=a.device)
        sa, sb, sc = self.slot["A"], self.slot["B"], self.slot["C"]
        ha, hb = min(2, self.seen), min(2, 4 * self.seen)
        r["A1"].load(sa, a)
        self._block("A1", "A2", "PA", sa, ha, T)
        L["PA"].forward_ring(r["PA"], 0, 0, T, out_ring=r["B1"], out_slot=sb, up_rt=4)      # 1x1x1, upsample in the store
        self._block("B1", "B2", "PB", sb, hb, 4 * T)
        L["PB"].forward_ring(r["PB"], 0, 0, 4 * T, out_ring=r["C1"], out_slot=sc, up_rt=1)
        self._block("C1", "C2", None, sc, hb, 4 * T, out=out)
        self.seen += T
        self.slot = {"A": (sa + T) % r["A1"].F, "B": (sb + 4 * T) % r["B1"].F, "C": (sc + 4 * T) % r["C1"].F}
        return out

    def close(self):
        for l in self.layers.values():
            l.close()
