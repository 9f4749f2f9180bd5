"""One cached causal Conv3D layer split by image rows across ranks (one process per GPU).

Every output element of the layer depends on its inputs only, and the per-tap 2-D correlation of Eq. (2) is
local in h: output row i reads input rows i - pad_h + dh * d_h.  So rank r of `world` owns a band of image rows
[r0, r1) of input and output alike (the layer must keep the height: 2 pad_h = d_h (kh - 1), as every layer of
a decoder does), keeps its input as a slab of rows [r0 - pad_h, r1 + pad_h) with the pad_h halo rows on either
side taken from its two neighbours (zeros at the image edge, which is the layer's zero padding), and runs
the unchanged single-GPU layer on the slab with pad_h = 0: the result is exactly the band's rows of the
unsplit layer, with the same order of accumulation per output element.  The temporal cache is kept per rank as
a slab *with* its halo rows (the new cache is the last frames of the slab that was just assembled), so there is
one neighbour exchange per layer and chunk - the halo rows of x - and none for the cache.

The exchange is the only communication: point-to-point sends of contiguous buffers through torch.distributed
(NCCL send/recv between GPUs, into this GPU's own memory first; the convolution kernel never reads a peer's
memory).  Packing, unpacking and slab assembly are `ccv3d_rows_copy` launches.  Height-split needs unit
stride in h; stride in t and w, dilation and padding in w are the layer's own.
"""
from __future__ import annotations

from dataclasses import dataclass

from . import CausalConv3d, Ccv3dError, OK, ccv3d_rows_copy


def band(H: int, world: int, rank: int):
    """Rows [r0, r1) of rank `rank`: H rows dealt out as evenly as possible, the first H % world bands one row taller."""
    base, rem = divmod(H, world)
    r0 = rank * base + min(rank, rem)
    return r0, r0 + base + (1 if rank < rem else 0)


@dataclass(frozen=True)
class HaloPlan:
    H: int
    world: int
    rank: int
    top: int          # halo rows above the band (from rank - 1, or zeros)
    bot: int          # halo rows below the band (from rank + 1, or zeros)
    r0: int
    r1: int

    @property
    def rows(self):
        return self.r1 - self.r0

    @property
    def slab_rows(self):
        return self.top + self.rows + self.bot

    @property
    def up(self):
        """Rank that owns the rows above this band, or None at the top of the image."""
        return self.rank - 1 if self.rank > 0 else None

    @property
    def down(self):
        return self.rank + 1 if self.rank < self.world - 1 else None


def halo_plan(H: int, world: int, rank: int, kh: int, pad_h: int, dil_h: int = 1) -> HaloPlan:
    if world < 1 or not 0 <= rank < world or H < 1 or kh < 1 or dil_h < 1 or pad_h < 0:
        raise ValueError("bad height-split arguments")
    if 2 * pad_h != dil_h * (kh - 1):
        raise ValueError("height-split needs a layer that keeps the height: 2 pad_h = d_h (kh - 1)")
    top = bot = pad_h
    if world > 1 and H // world < max(top, bot, 1):
        raise ValueError("bands are shorter than the halo: a halo row would come from beyond the neighbour")
    r0, r1 = band(H, world, rank)
    return HaloPlan(H, world, rank, top, bot, r0, r1)


class CudaRowOps:
    """Device buffers through torch, every copy through the library."""

    def empty(self, shape, like):
        import torch
        return torch.empty(shape, dtype=like.dtype, device=like.device)

    def rows_copy(self, dst, dst_row0, src, src_row0, rows):
        """dst[..., dst_row0 : dst_row0+rows, :] <- src[..., src_row0 : src_row0+rows, :] (src None: zeros)."""
        import torch
        assert dst.is_cuda and dst.is_contiguous() and (src is None or (src.is_cuda and src.is_contiguous()))
        W = dst.shape[-1]
        planes = dst.numel() // (dst.shape[-2] * W)
        if src is not None:
            assert src.shape[-1] == W and src.dtype == dst.dtype and src.numel() // (src.shape[-2] * W) == planes
        s = ccv3d_rows_copy(dst.data_ptr(), dst.shape[-2], dst_row0, None if src is None else src.data_ptr(),
                            0 if src is None else src.shape[-2], src_row0, planes, rows, W * dst.element_size(),
                            torch.cuda.current_stream().cuda_stream)
        if s != OK:
            raise Ccv3dError(s, "ccv3d_rows_copy")


class DistTransport:
    """Neighbour exchange over a torch.distributed process group (NCCL between GPUs)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group

    def _peer(self, r):
        return r if self.group is None else self.dist.get_global_rank(self.group, r)

    def exchange(self, plan: HaloPlan, to_up, to_down, from_up, from_down):
        """Sends `to_up` / `to_down` to the neighbours and fills `from_up` / `from_down` (each may be None)."""
        d, ops = self.dist, []
        for buf, peer, op in ((to_up, plan.up, d.isend), (from_up, plan.up, d.irecv),
                              (to_down, plan.down, d.isend), (from_down, plan.down, d.irecv)):
            if buf is not None and peer is not None:
                ops.append(d.P2POp(op, buf, self._peer(peer), self.group))
        if ops:
            for req in d.batch_isend_irecv(ops):
                req.wait()


class HSplitCausalConv3d:
    """The band of one layer that rank `rank` of `world` computes.

    forward(x_band [N,Cin,T,rows,W], cache_slab) -> (out_band [N,Cout,T_o,rows,W_o], new_cache_slab); the cache
    slab is [N,Cin,d_t(kt-1),slab_rows,W] and only ever comes from a previous call (None on the first chunk).
    `conv`, `ops` and `transport` exist so that the host logic can be exercised without GPUs; by default the
    layer is the library's, the copies are the library's and the exchange is torch.distributed's.
    """

    def __init__(self, w, b, H, rank, world, transport=None, ops=None, conv=None, out_dtype=None, flags=0,
                 stride=(1, 1, 1), dilation=(1, 1, 1), pad=None):
        kt, kh, kw = w.shape[2:]
        if stride[1] != 1:
            raise ValueError("height-split needs unit stride in h")
        if pad is None:
            pad = (dilation[0] * (kt - 1) // 2, dilation[1] * (kh - 1) // 2, dilation[2] * (kw - 1) // 2)
        self.plan = halo_plan(H, world, rank, kh, pad[1], dilation[1])
        self.ops = ops if ops is not None else CudaRowOps()
        self.transport = transport if transport is not None else (DistTransport() if world > 1 else None)
        self.conv = conv if conv is not None else CausalConv3d(w, b, out_dtype=out_dtype, flags=flags, stride=stride,
                                                               dilation=dilation, pad=(pad[0], 0, pad[2]))

    # -- the three steps of a call; forward_all_local drives them for several ranks held by one process --
    def pack(self, x_band):
        """Contiguous copies of the rows the neighbours need: (to_up, to_down), None where nothing is sent."""
        p, o = self.plan, self.ops
        assert x_band.shape[-2] == p.rows, "x_band must hold exactly this rank's rows"
        lead = tuple(x_band.shape[:-2])
        W = x_band.shape[-1]
        to_up = to_down = None
        if p.up is not None and p.bot > 0:            # my first rows are the upper neighbour's bottom halo
            to_up = o.empty(lead + (p.bot, W), x_band)
            o.rows_copy(to_up, 0, x_band, 0, p.bot)
        if p.down is not None and p.top > 0:          # my last rows are the lower neighbour's top halo
            to_down = o.empty(lead + (p.top, W), x_band)
            o.rows_copy(to_down, 0, x_band, p.rows - p.top, p.top)
        return to_up, to_down

    def recv_buffers(self, x_band):
        p, o = self.plan, self.ops
        lead, W = tuple(x_band.shape[:-2]), x_band.shape[-1]
        from_up = o.empty(lead + (p.top, W), x_band) if (p.up is not None and p.top > 0) else None
        from_down = o.empty(lead + (p.bot, W), x_band) if (p.down is not None and p.bot > 0) else None
        return from_up, from_down

    def assemble(self, x_band, from_up, from_down):
        """[halo above ; band ; halo below]; a halo with no neighbour behind it is the layer's zero padding."""
        p, o = self.plan, self.ops
        slab = o.empty(tuple(x_band.shape[:-2]) + (p.slab_rows, x_band.shape[-1]), x_band)
        if p.top > 0:
            o.rows_copy(slab, 0, from_up, 0, p.top)
        o.rows_copy(slab, p.top, x_band, 0, p.rows)
        if p.bot > 0:
            o.rows_copy(slab, p.top + p.rows, from_down, 0, p.bot)
        return slab

    def forward(self, x_band, cache_slab=None):
        to_up, to_down = self.pack(x_band)
        from_up, from_down = self.recv_buffers(x_band)
        if self.transport is not None:
            self.transport.exchange(self.plan, to_up, to_down, from_up, from_down)
        return self.conv(self.assemble(x_band, from_up, from_down), cache_slab)

    __call__ = forward

    def close(self):
        if hasattr(self.conv, "close"):
            self.conv.close()


def forward_all_local(layers, x_bands, cache_slabs=None):
    """All ranks of one height-split layer held by one process (one GPU, or a test): the neighbour exchange is a
    hand-over of the packed buffers, everything else is the per-rank path.  Returns (out_bands, new_cache_slabs)."""
    world = len(layers)
    assert all(l.plan.world == world and l.plan.rank == r for r, l in enumerate(layers)) and len(x_bands) == world
    cache_slabs = cache_slabs if cache_slabs is not None else [None] * world
    packed = [l.pack(x) for l, x in zip(layers, x_bands)]
    outs, caches = [], []
    for r, (l, x) in enumerate(zip(layers, x_bands)):
        from_up = packed[r - 1][1] if r > 0 else None                # the upper neighbour's to_down
        from_down = packed[r + 1][0] if r < world - 1 else None      # the lower neighbour's to_up
        o, c = l.conv(l.assemble(x, from_up, from_down), cache_slabs[r])
        outs.append(o)
        caches.append(c)
    return outs, caches


# ------------------------------------------------------------------------------------------------------------------
# Height-split on resident activations (frame rings)
# ------------------------------------------------------------------------------------------------------------------
# A rank's rings hold its slab (halo rows included) instead of the whole image, and a layer is the unchanged ring
# call with its own zero padding on the slab.  The layer's output rows at halo positions come out wrong (they saw
# zero padding where the neighbour's rows belong) - but those are exactly the rows the next layer must get from the
# neighbours anyway: after every layer the band's edge rows are sent, the halo rows of the output ring are
# overwritten with what the neighbours sent (zeros where the image ends), and the ring is a valid input slab.  No
# slab assembly, no cache: the temporal history is whatever earlier chunks left in the ring, halos included.  Cost
# per layer over the unsplit share: 2 * halo extra rows of convolution and four small row copies.

def _frame_runs(slot0, T, F):
    """Slots slot0 .. slot0+T-1 (mod F) as contiguous runs [(first slot, frames, first frame index)]."""
    s = slot0 % F
    first = min(T, F - s)
    runs = [(s, first, 0)]
    if first < T:
        runs.append((0, T - first, first))
    return runs


def ring_rows_copy(ring, slot0, T, row0, rows, buf, to_ring):
    """Rows row0 .. row0+rows-1 of frames slot0.. of `ring`  <->  buf [N][T][C/KB][rows][W][KB] (contiguous).
    to_ring with buf None writes zeros."""
    import torch
    st = torch.cuda.current_stream().cuda_stream
    CB = ring.C // ring.KB
    row_bytes = ring.W * ring.KB * 2
    for n in range(ring.N):
        for s, cnt, t0 in _frame_runs(slot0, T, ring.F):
            rp = ring.buf.data_ptr() + ((n * ring.F + s) * CB) * ring.H * row_bytes
            bp = None if buf is None else buf.data_ptr() + ((n * T + t0) * CB) * rows * row_bytes
            if to_ring:
                st_ = ccv3d_rows_copy(rp, ring.H, row0, bp, rows, 0, cnt * CB, rows, row_bytes, st)
            else:
                st_ = ccv3d_rows_copy(bp, rows, 0, rp, ring.H, row0, cnt * CB, rows, row_bytes, st)
            if st_ != OK:
                raise Ccv3dError(st_, "ccv3d_rows_copy")


class HSplitRingConv3d:
    """One layer of a height-split stage on frame rings.  All layers that share rings share the slab geometry, so
    `halo` is the stage's (the largest (kh-1)/2 of its layers; a 1x1x1 layer in a 3x3 stage runs with halo 1)."""

    def __init__(self, w, b, H, rank, world, halo=None, transport=None, flags=0):
        kt, kh, kw = w.shape[2:]
        own = (kh - 1) // 2
        halo = own if halo is None else halo
        if kh % 2 == 0 or halo < own:
            raise ValueError("the stage's halo must cover this layer's reach in h")
        self.plan = halo_plan(H, world, rank, 2 * halo + 1, halo)
        self.transport = transport if transport is not None else (DistTransport() if world > 1 else None)
        self.conv = CausalConv3d(w, b, flags=flags)           # standard geometry: zero padding on the slab

    def ring(self, N, C, F, W):
        from . import FrameRing
        return FrameRing(N, C, F, self.plan.slab_rows, W, zero=True)

    def _buf(self, ring, T, rows):
        import torch
        return torch.empty((ring.N, T, ring.C // ring.KB, rows, ring.W, ring.KB), dtype=torch.bfloat16, device="cuda")

    def pack(self, ring, slot0, T):
        """The band's edge rows of frames slot0.. as contiguous buffers (to_up, to_down); None where nothing is sent."""
        p = self.plan
        assert ring.H == p.slab_rows
        to_up = to_down = None
        if p.up is not None and p.bot > 0:
            to_up = self._buf(ring, T, p.bot)
            ring_rows_copy(ring, slot0, T, p.top, p.bot, to_up, to_ring=False)
        if p.down is not None and p.top > 0:
            to_down = self._buf(ring, T, p.top)
            ring_rows_copy(ring, slot0, T, p.top + p.rows - p.top, p.top, to_down, to_ring=False)
        return to_up, to_down

    def recv_buffers(self, ring, T):
        p = self.plan
        return (self._buf(ring, T, p.top) if (p.up is not None and p.top > 0) else None,
                self._buf(ring, T, p.bot) if (p.down is not None and p.bot > 0) else None)

    def unpack(self, ring, slot0, T, from_up, from_down):
        """Halo rows of frames slot0.. <- the neighbours' rows; zeros where the image ends."""
        p = self.plan
        if p.top > 0:
            ring_rows_copy(ring, slot0, T, 0, p.top, from_up if p.up is not None else None, to_ring=True)
        if p.bot > 0:
            ring_rows_copy(ring, slot0, T, p.top + p.rows, p.bot, from_down if p.down is not None else None, to_ring=True)

    def exchange(self, ring, slot0, T):
        to_up, to_down = self.pack(ring, slot0, T)
        from_up, from_down = self.recv_buffers(ring, T)
        if self.transport is not None:
            self.transport.exchange(self.plan, to_up, to_down, from_up, from_down)
        self.unpack(ring, slot0, T, from_up, from_down)

    def load_band(self, ring, slot0, x_band, exchange=True):
        """Chunk input: NCTHW band -> the band rows of ring slots slot0.., then the halo exchange (exchange=False:
        the caller runs it, e.g. ring_exchange_all_local)."""
        import torch
        p = self.plan
        N, C, T, rows, W = x_band.shape
        assert rows == p.rows and ring.H == p.slab_rows
        slab = torch.zeros((N, C, T, p.slab_rows, W), dtype=x_band.dtype, device=x_band.device)
        CudaRowOps().rows_copy(slab, p.top, x_band, 0, p.rows)
        ring.load(slot0, slab)
        if exchange:
            self.exchange(ring, slot0, T)

    def forward(self, rin, x_slot, hist_frames, T, out_ring, out_slot=0, res=None, res_slot=0):
        """The layer on this rank's slab rings; `out_ring` leaves as a valid input slab of the next layer."""
        self.conv.forward_ring(rin, x_slot, hist_frames, T, out_ring=out_ring, out_slot=out_slot, res=res, res_slot=res_slot)
        self.exchange(out_ring, out_slot, T)
        return out_ring

    def forward_out(self, rin, x_slot, hist_frames, T, res=None, res_slot=0):
        """Last layer of a stage: the band as NCTHW [N,Cout,T,rows,W] (no exchange: nobody reads its halo)."""
        import torch
        p = self.plan
        slab = torch.empty((rin.N, self.conv.cout, T, p.slab_rows, rin.W), dtype=torch.bfloat16, device="cuda")
        self.conv.forward_ring(rin, x_slot, hist_frames, T, out=slab, res=res, res_slot=res_slot)
        band = torch.empty((rin.N, self.conv.cout, T, p.rows, rin.W), dtype=torch.bfloat16, device="cuda")
        CudaRowOps().rows_copy(band, 0, slab, p.top, p.rows)
        return band

    def close(self):
        self.conv.close()


def ring_exchange_all_local(layers, rings, slot0, T):
    """The halo exchange of all ranks held by one process: pack everywhere, hand the buffers over, unpack."""
    world = len(layers)
    packed = [l.pack(r, slot0, T) for l, r in zip(layers, rings)]
    for k, (l, r) in enumerate(zip(layers, rings)):
        l.unpack(r, slot0, T, packed[k - 1][1] if k > 0 else None, packed[k + 1][0] if k < world - 1 else None)


def ring_forward_all_local(layers, rins, x_slot, hist_frames, T, out_rings, out_slot=0, res_rings=None, res_slot=0):
    """One layer for all ranks held by one process: every rank's ring call, then the exchange by hand-over."""
    for k, l in enumerate(layers):
        l.conv.forward_ring(rins[k], x_slot, hist_frames, T, out_ring=out_rings[k], out_slot=out_slot,
                            res=None if res_rings is None else res_rings[k], res_slot=res_slot)
    ring_exchange_all_local(layers, out_rings, out_slot, T)
    return out_rings
