"""Python binding of the ccv3d C-ABI library (cached causal Conv3D for B200).

Argument marshalling only: every step of the operator runs inside
``libccv3d.so`` (hand-written CUDA for sm_100a).  The functions below carry the
names of the C entry points declared in ``include/ccv3d.h`` and take raw
addresses; ``CausalConv3d`` is a thin convenience wrapper that takes torch
tensors (torch is used for device memory and streams, nothing else).

There is no CPU or library fallback: importing this package without the built
library raises.
"""
from __future__ import annotations

import ctypes
import os

from . import _build

F32, BF16 = 0, 1
FLAG_FORCE_SIMT = 0x1
FLAG_TC_PER_TAP_A = 0x2
FLAG_OVERLAP = 0x4
FLAG_FUSED = 0x8
FLAG_TWO_KERNELS = 0x10
FLAG_F32_TENSOR = 0x20
FLAG_NO_PAIR = 0x40
FLAG_EPI_SILU = 0x80
FLAG_NO_TAIL_SPLIT = 0x100

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_ALIAS, ERR_ARCH, ERR_NOMEM, ERR_CUDA, \
    ERR_DEVICE_TIMEOUT = range(9)


class Desc(ctypes.Structure):
    _fields_ = [("cin", ctypes.c_int32), ("cout", ctypes.c_int32),
                ("kt", ctypes.c_int32), ("kh", ctypes.c_int32), ("kw", ctypes.c_int32),
                ("pad_t", ctypes.c_int32), ("pad_h", ctypes.c_int32), ("pad_w", ctypes.c_int32),
                ("stride", ctypes.c_int32 * 3), ("dilation", ctypes.c_int32 * 3), ("groups", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class Counters(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in ("calls", "ok", "tcgen05_bf16", "tcgen05_f32", "pointwise", "simt", "unsupported", "invalid",
                                               "cuda_error", "device_timeout", "kernel_launches")]


class Ring(ctypes.Structure):
    """ccv3d_ring: a frame ring [N][F][C/KB][H][W][KB] of BF16 activations on the device."""
    _fields_ = [("base", ctypes.c_void_p), ("N", ctypes.c_int32), ("C", ctypes.c_int32), ("F", ctypes.c_int32),
                ("H", ctypes.c_int32), ("W", ctypes.c_int32), ("KB", ctypes.c_int32)]


EXPORTS = ("ccv3d_create", "ccv3d_forward", "ccv3d_forward_host", "ccv3d_workspace_bytes", "ccv3d_destroy",
           "ccv3d_get_counters", "ccv3d_device_status", "ccv3d_status_string", "ccv3d_add_bf16",
           "ccv3d_upsample_bf16", "ccv3d_profile_enable", "ccv3d_profile_read", "ccv3d_forward_static", "ccv3d_selftest_wait_timeout", "ccv3d_forward_ex",
           "ccv3d_ring_kb", "ccv3d_ring_bytes", "ccv3d_ring_load", "ccv3d_ring_store", "ccv3d_upsample_ring",
           "ccv3d_forward_ring", "ccv3d_out_dims", "ccv3d_forward_ring_up", "ccv3d_rows_copy",
           "ccv3d_forward_host_stream", "ccv3d_set_workspace")


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                          "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(path)
    vp, i32, u64p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_uint64)
    lib.ccv3d_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Desc), vp, vp, vp]
    lib.ccv3d_forward.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.ccv3d_forward_ex.argtypes = [vp, vp, vp, i32, vp, vp, i32, i32, i32, i32, vp]
    lib.ccv3d_forward_static.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.ccv3d_forward_host.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.ccv3d_forward_host_stream.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
    lib.ccv3d_workspace_bytes.argtypes = [vp, i32, i32, i32, i32, u64p]
    lib.ccv3d_set_workspace.argtypes = [vp, vp, ctypes.c_uint64]
    lib.ccv3d_destroy.argtypes = [vp]
    lib.ccv3d_get_counters.argtypes = [vp, ctypes.POINTER(Counters)]
    lib.ccv3d_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.ccv3d_status_string.argtypes = [ctypes.c_int]
    lib.ccv3d_status_string.restype = ctypes.c_char_p
    lib.ccv3d_profile_enable.argtypes = [vp, i32]
    lib.ccv3d_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                       ctypes.POINTER(ctypes.c_int64)]
    lib.ccv3d_selftest_wait_timeout.argtypes = [vp, i32, vp]
    lib.ccv3d_add_bf16.argtypes = [vp, vp, vp, ctypes.c_int64, vp]
    lib.ccv3d_upsample_bf16.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, vp]
    lib.ccv3d_rows_copy.argtypes = [vp, i32, i32, vp, i32, i32, ctypes.c_int64, i32, ctypes.c_int64, vp]
    i32p = ctypes.POINTER(ctypes.c_int32)
    lib.ccv3d_out_dims.argtypes = [vp, i32, i32, i32, i32p, i32p, i32p, i32p]
    rp = ctypes.POINTER(Ring)
    lib.ccv3d_ring_kb.argtypes = [i32]
    lib.ccv3d_ring_bytes.argtypes = [rp]
    lib.ccv3d_ring_load.argtypes = [rp, i32, vp, i32, vp]
    lib.ccv3d_ring_store.argtypes = [rp, i32, vp, i32, vp]
    lib.ccv3d_upsample_ring.argtypes = [rp, i32, rp, i32, i32, i32, vp]
    lib.ccv3d_forward_ring.argtypes = [vp, rp, i32, i32, rp, i32, rp, i32, vp, i32, vp]
    lib.ccv3d_forward_ring_up.argtypes = [vp, rp, i32, i32, rp, i32, rp, i32, i32, i32, vp]
    for name in EXPORTS:
        if name not in ("ccv3d_status_string", "ccv3d_ring_bytes"):
            getattr(lib, name).restype = ctypes.c_int
    lib.ccv3d_ring_bytes.restype = ctypes.c_uint64
    return lib


lib = _load()


class Ccv3dError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)}")


def status_string(s: int) -> str:
    return lib.ccv3d_status_string(int(s)).decode()


def make_desc(cin, cout, k=(3, 3, 3), dtype=BF16, out_dtype=None, flags=0, stride=(1, 1, 1), dilation=(1, 1, 1),
              groups=1, pad=None) -> Desc:
    kt, kh, kw = k
    pad = pad if pad is not None else ((kt - 1) // 2, (kh - 1) // 2, (kw - 1) // 2)
    d = Desc()
    d.cin, d.cout, d.kt, d.kh, d.kw = cin, cout, kt, kh, kw
    d.pad_t, d.pad_h, d.pad_w = pad
    d.stride[:] = stride
    d.dilation[:] = dilation
    d.groups = groups
    d.dtype = dtype
    d.out_dtype = dtype if out_dtype is None else out_dtype
    d.flags = flags
    return d


# ---- the C entry points, same names, raw addresses (ints) ----
def ccv3d_create(desc: Desc, w_dev: int, b_dev: int | None, stream: int = 0):
    h = ctypes.c_void_p()
    s = lib.ccv3d_create(ctypes.byref(h), ctypes.byref(desc), w_dev, b_dev, stream)
    return s, (h.value if s == OK else None)


def ccv3d_forward(h, x, cache, out, new_cache, N, T, H, W, stream=0) -> int:
    return lib.ccv3d_forward(h, x, cache, out, new_cache, N, T, H, W, stream)


def ccv3d_forward_ex(h, x, cache, cache_frames, out, new_cache, N, T, H, W, stream=0) -> int:
    """ccv3d_forward with a cache of cache_frames <= kt-1 frames (older history absent = zero)."""
    return lib.ccv3d_forward_ex(h, x, cache, cache_frames, out, new_cache, N, T, H, W, stream)


def ccv3d_forward_static(h, x, cache, out, new_cache, N, T, H, W, stream=0) -> int:
    """ccv3d_forward for callers that cannot allocate: the staging copy lives in a fixed 32 MiB device array."""
    return lib.ccv3d_forward_static(h, x, cache, out, new_cache, N, T, H, W, stream)


def ccv3d_forward_host(h, x, cache, out, new_cache, N, T, H, W, stream=0) -> int:
    return lib.ccv3d_forward_host(h, x, cache, out, new_cache, N, T, H, W, stream)


def ccv3d_forward_host_stream(h, x, out, reset, N, T, H, W, stream=0) -> int:
    """x/out are HOST pointers; the history stays on the device between calls."""
    return lib.ccv3d_forward_host_stream(h, x, out, 1 if reset else 0, N, T, H, W, stream)


def ccv3d_out_dims(h, T, H, W):
    """(status, T_o, H_o, W_o, history frames) of a layer for a T x H x W input."""
    t, a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    s = lib.ccv3d_out_dims(h, T, H, W, ctypes.byref(t), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    return s, t.value, a.value, b.value, c.value


def ccv3d_workspace_bytes(h, N, T, H, W):
    b = ctypes.c_uint64()
    s = lib.ccv3d_workspace_bytes(h, N, T, H, W, ctypes.byref(b))
    return s, b.value


def ccv3d_set_workspace(h, ws_dev, nbytes) -> int:
    """Lend the handle a caller-owned staging workspace (DEVICE address, 256-byte aligned); None/0 takes it back."""
    return lib.ccv3d_set_workspace(h, ws_dev, nbytes)


def ccv3d_destroy(h) -> int:
    return lib.ccv3d_destroy(h)


def ccv3d_get_counters(h) -> dict:
    c = Counters()
    s = lib.ccv3d_get_counters(h, ctypes.byref(c))
    if s != OK:
        raise Ccv3dError(s, "ccv3d_get_counters")
    return {n: int(getattr(c, n)) for n, _ in Counters._fields_}


def ccv3d_device_status(h):
    d = ctypes.c_uint32()
    s = lib.ccv3d_device_status(h, ctypes.byref(d))
    return s, d.value


def ccv3d_profile_enable(h, enable: bool) -> int:
    return lib.ccv3d_profile_enable(h, 1 if enable else 0)


def ccv3d_profile_read(h):
    """(status, staging-kernel ms, convolution-kernel ms, calls) summed since the last read; sync the stream first."""
    a, b, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_int64()
    s = lib.ccv3d_profile_read(h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(n))
    return s, a.value, b.value, n.value


def ccv3d_selftest_wait_timeout(h, limit_ms: int, stream=0) -> int:
    return lib.ccv3d_selftest_wait_timeout(h, limit_ms, stream)


def ccv3d_add_bf16(a, b, y, n, stream=0) -> int:
    return lib.ccv3d_add_bf16(a, b, y, n, stream)


def ccv3d_upsample_bf16(x, y, N, C, T, H, W, rt, stream=0) -> int:
    return lib.ccv3d_upsample_bf16(x, y, N, C, T, H, W, rt, stream)


def ccv3d_rows_copy(dst, dst_H, dst_row0, src, src_H, src_row0, planes, rows, row_bytes, stream=0) -> int:
    return lib.ccv3d_rows_copy(dst, dst_H, dst_row0, src, src_H, src_row0, planes, rows, row_bytes, stream)


def ccv3d_ring_kb(C: int) -> int:
    return lib.ccv3d_ring_kb(C)


def ccv3d_ring_bytes(ring: Ring) -> int:
    return int(lib.ccv3d_ring_bytes(ctypes.byref(ring)))


def ccv3d_ring_load(ring: Ring, slot0: int, x: int, T: int, stream=0) -> int:
    return lib.ccv3d_ring_load(ctypes.byref(ring), slot0, x, T, stream)


def ccv3d_ring_store(ring: Ring, slot0: int, y: int, T: int, stream=0) -> int:
    return lib.ccv3d_ring_store(ctypes.byref(ring), slot0, y, T, stream)


def ccv3d_upsample_ring(rin: Ring, in_slot0: int, rout: Ring, out_slot0: int, T: int, rt: int, stream=0) -> int:
    return lib.ccv3d_upsample_ring(ctypes.byref(rin), in_slot0, ctypes.byref(rout), out_slot0, T, rt, stream)


def ccv3d_forward_ring(h, rin: Ring, x_slot: int, hist_frames: int, res: Ring | None, res_slot: int,
                       out_ring: Ring | None, out_slot: int, out_ncthw: int | None, T: int, stream=0) -> int:
    return lib.ccv3d_forward_ring(h, ctypes.byref(rin), x_slot, hist_frames,
                                  None if res is None else ctypes.byref(res), res_slot,
                                  None if out_ring is None else ctypes.byref(out_ring), out_slot, out_ncthw, T, stream)


def ccv3d_forward_ring_up(h, rin: Ring, x_slot: int, hist_frames: int, res: Ring | None, res_slot: int, out_ring: Ring,
                          out_slot: int, rt: int, T: int, stream=0) -> int:
    return lib.ccv3d_forward_ring_up(h, ctypes.byref(rin), x_slot, hist_frames,
                                     None if res is None else ctypes.byref(res), res_slot, ctypes.byref(out_ring),
                                     out_slot, rt, T, stream)


class FrameRing:
    """A frame ring on the current CUDA device: torch owns the memory, `c` is the struct the C calls take."""

    def __init__(self, N, C, F, H, W, zero=False):
        import torch
        kb = ccv3d_ring_kb(C)
        if kb == 0:
            raise ValueError(f"{C} channels cannot live in a frame ring (need a multiple of 32)")
        self.N, self.C, self.F, self.H, self.W, self.KB = N, C, F, H, W, kb
        alloc = torch.zeros if zero else torch.empty
        self.buf = alloc((N, F, C // kb, H, W, kb), dtype=torch.bfloat16, device="cuda")
        self.c = Ring(self.buf.data_ptr(), N, C, F, H, W, kb)
        self._stream = lambda: torch.cuda.current_stream().cuda_stream

    def load(self, slot0, x):
        """x [N,C,T,H,W] -> slots slot0.. (mod F)."""
        assert x.is_cuda and x.is_contiguous() and x.shape[:2] == (self.N, self.C) and x.shape[3:] == (self.H, self.W)
        s = ccv3d_ring_load(self.c, slot0, x.data_ptr(), x.shape[2], self._stream())
        if s != OK:
            raise Ccv3dError(s, "ccv3d_ring_load")

    def store(self, slot0, T, y=None):
        """slots slot0.. (mod F) -> y [N,C,T,H,W]."""
        import torch
        if y is None:
            y = torch.empty((self.N, self.C, T, self.H, self.W), dtype=torch.bfloat16, device="cuda")
        s = ccv3d_ring_store(self.c, slot0, y.data_ptr(), T, self._stream())
        if s != OK:
            raise Ccv3dError(s, "ccv3d_ring_store")
        return y


class CausalConv3d:
    """One cached causal Conv3D layer on the current CUDA device (torch tensors in, torch tensors out)."""

    def __init__(self, w, b=None, out_dtype=None, flags=0, stride=(1, 1, 1), dilation=(1, 1, 1), pad=None):
        import torch
        assert w.is_cuda and w.is_contiguous() and w.dim() == 5
        self.torch = torch
        self.dtype = BF16 if w.dtype == torch.bfloat16 else F32
        assert w.dtype in (torch.bfloat16, torch.float32)
        cout, cin, kt, kh, kw = w.shape
        self.k, self.cin, self.cout = (kt, kh, kw), cin, cout
        self.out_dtype = self.dtype if out_dtype is None else out_dtype
        if pad is None:          # size-preserving spatial padding; the temporal entry only has to describe the causal total
            pad = (dilation[0] * (kt - 1) // 2, dilation[1] * (kh - 1) // 2, dilation[2] * (kw - 1) // 2)
        self.desc = make_desc(cin, cout, self.k, self.dtype, self.out_dtype, flags, stride=stride, dilation=dilation,
                              pad=pad)
        self.tc = dilation[0] * (kt - 1)
        if b is not None:
            assert b.is_cuda and b.is_contiguous() and b.dtype == w.dtype and b.shape == (cout,)
        s, h = ccv3d_create(self.desc, w.data_ptr(), None if b is None else b.data_ptr(),
                            torch.cuda.current_stream().cuda_stream)
        if s != OK:
            raise Ccv3dError(s, "ccv3d_create")
        self.h = h

    def forward(self, x, cache=None, out=None, new_cache=None, want_cache=True):
        torch = self.torch
        N, C, T, H, W = x.shape
        assert C == self.cin and x.is_contiguous() and x.is_cuda
        tc = self.tc
        odt = torch.bfloat16 if self.out_dtype == BF16 else torch.float32
        if out is None:
            _, To, Ho, Wo, _ = ccv3d_out_dims(self.h, T, H, W)
            out = torch.empty((N, self.cout, To, Ho, Wo), dtype=odt, device=x.device)
        if new_cache is None and want_cache and tc:
            new_cache = torch.empty((N, C, tc, H, W), dtype=x.dtype, device=x.device)
        cf = 0
        if cache is not None:
            cf = cache.shape[2]      # a cache shorter than the full history: the older frames do not exist yet
            assert cache.is_contiguous() and cache.shape == (N, C, cf, H, W) and cache.dtype == x.dtype and 0 < cf <= tc
        s = ccv3d_forward_ex(self.h, x.data_ptr(), None if cache is None else cache.data_ptr(), cf, out.data_ptr(),
                             None if new_cache is None else new_cache.data_ptr(), N, T, H, W,
                             torch.cuda.current_stream().cuda_stream)
        if s != OK:
            raise Ccv3dError(s, "ccv3d_forward_ex")
        return out, new_cache

    __call__ = forward

    def forward_ring(self, rin: FrameRing, x_slot, hist_frames, T, out_ring: FrameRing | None = None, out_slot=0,
                     out=None, res: FrameRing | None = None, res_slot=0, up_rt=0):
        """The layer on resident activations (see ccv3d_forward_ring): reads `rin`, writes `out_ring` or NCTHW `out`.
        up_rt > 0: `out_ring` is 2H x 2W and receives the 2x2-upsampled output, every frame up_rt times."""
        st = self.torch.cuda.current_stream().cuda_stream
        if up_rt > 0:
            s = ccv3d_forward_ring_up(self.h, rin.c, x_slot, hist_frames, None if res is None else res.c, res_slot,
                                      out_ring.c, out_slot, up_rt, T, st)
        else:
            s = ccv3d_forward_ring(self.h, rin.c, x_slot, hist_frames, None if res is None else res.c, res_slot,
                                   None if out_ring is None else out_ring.c, out_slot,
                                   None if out is None else out.data_ptr(), T, st)
        if s != OK:
            raise Ccv3dError(s, "ccv3d_forward_ring")
        return out_ring if out_ring is not None else out

    def counters(self):
        return ccv3d_get_counters(self.h)

    def device_status(self):
        return ccv3d_device_status(self.h)

    def close(self):
        if getattr(self, "h", None):
            ccv3d_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
