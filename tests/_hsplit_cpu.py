"""Stand-ins that let the height-split host logic run without a GPU: row copies by slicing, the layer by the oracle.
Test infrastructure only."""
import numpy as np
import torch

import oracle


class TorchRowOps:
    def empty(self, shape, like):
        return torch.full(shape, float("nan"), dtype=like.dtype)      # a row nobody wrote would poison the result

    def rows_copy(self, dst, dst_row0, src, src_row0, rows):
        dst[..., dst_row0:dst_row0 + rows, :] = 0 if src is None else src[..., src_row0:src_row0 + rows, :]


class OracleConv:
    """(slab, cache_slab) -> (out float64, new_cache) with pad_h = 0, as the height-split layer asks of its inner layer."""

    def __init__(self, w, b, pad_w, stride=(1, 1, 1), dilation=(1, 1, 1)):
        self.w, self.b, self.pad_w, self.stride, self.dil = w, b, pad_w, stride, dilation

    def __call__(self, slab, cache_slab):
        out, nc = oracle.forward_general(slab.numpy(), None if cache_slab is None else cache_slab.numpy(), self.w, self.b,
                                         stride=(1, self.stride[2]), pad=(0, self.pad_w), dil=(self.dil[1], self.dil[2]),
                                         dil_t=self.dil[0], stride_t=self.stride[0])
        return torch.from_numpy(out), None if nc is None else torch.from_numpy(nc)


def case_tensors(seed, N, Cin, Cout, T, H, W, k):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((N, Cin, T, H, W)).astype(np.float32)
    w = (rng.standard_normal((Cout, Cin) + tuple(k)) / np.sqrt(Cin * np.prod(k))).astype(np.float32)
    b = rng.standard_normal(Cout).astype(np.float32)
    return x, w, b
