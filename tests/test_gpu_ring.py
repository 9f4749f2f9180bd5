"""GPU tests of the resident-activation entry points (frame rings): the layout moves are bit-exact permutations,
and a layer run on rings - history left in place by earlier calls, output written channels-last for the next
layer, optional residual in the epilogue - computes what the oracle's definition computes on the whole sequence."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from _util import as_f64, bits, check, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ccv():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as m
    torch.cuda.set_device(0)
    return m


def _rand_bf16(shape, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16).cuda()


def _ring_view(ring, slot, T):
    """Frames slot.. (mod F) of a ring as NCTHW, by indexing the ring's own buffer (pure permutation in torch)."""
    idx = [(slot + t) % ring.F for t in range(T)]
    b = ring.buf[:, idx]                                   # [N, T, CB, H, W, KB]
    return b.permute(0, 2, 5, 1, 3, 4).reshape(ring.N, ring.C, T, ring.H, ring.W).contiguous()


# ---------------------------------------------------------------------------- layout moves
@pytest.mark.parametrize("N,C,F,H,W,slot,T", [
    (1, 64, 3, 5, 8, 0, 3),       # 64-channel blocks
    (2, 96, 5, 7, 21, 3, 4),      # 32-channel blocks, odd width, slots wrap around
    (1, 192, 4, 17, 70, 2, 1),    # more than one 64-pixel span per row, ragged
    (1, 32, 2, 3, 3, 1, 2),
])
def test_ring_load_and_store_are_exact_inverses(ccv, N, C, F, H, W, slot, T):
    x = _rand_bf16((N, C, T, H, W), 1)
    ring = ccv.FrameRing(N, C, F, H, W, zero=True)
    ring.load(slot, x)
    torch.cuda.synchronize()
    assert torch.equal(_ring_view(ring, slot, T), x)                      # the stated layout, not just a round trip
    untouched = [s for s in range(F) if s not in [(slot + t) % F for t in range(T)]]
    assert not ring.buf[:, untouched].any()                               # no other slot is written
    y = ring.store(slot, T)
    torch.cuda.synchronize()
    assert torch.equal(y, x)


@pytest.mark.parametrize("N,C,H,W,T,rt", [(1, 64, 5, 6, 1, 4), (2, 96, 3, 7, 2, 1), (1, 32, 4, 4, 3, 2)])
def test_ring_upsample_is_nearest_neighbour_repeat(ccv, N, C, H, W, T, rt):
    x = _rand_bf16((N, C, T, H, W), 2)
    rin = ccv.FrameRing(N, C, T + 1, H, W, zero=True)
    rout = ccv.FrameRing(N, C, T * rt + 2, 2 * H, 2 * W, zero=True)
    rin.load(1, x)
    s = ccv.ccv3d_upsample_ring(rin.c, 1, rout.c, T * rt, T, rt, torch.cuda.current_stream().cuda_stream)
    assert s == ccv.OK
    torch.cuda.synchronize()
    want = x.repeat_interleave(rt, dim=2).repeat_interleave(2, dim=3).repeat_interleave(2, dim=4)
    assert torch.equal(_ring_view(rout, T * rt, T * rt), want)


# ---------------------------------------------------------------------------- the layer on rings
RING_CASES = [
    # N, Cin, Cout, H, W, k, chunk lengths, ring frames beyond the minimum
    (1, 64, 64, 20, 24, (3, 3, 3), [2, 2, 2], 0),       # 64-channel blocks, F = T + kt - 1: every slot is reused
    (1, 96, 96, 18, 21, (3, 3, 3), [1, 1, 1, 1], 0),    # 32-channel blocks, odd width, T < kt - 1
    (2, 128, 64, 33, 40, (3, 3, 3), [3, 3], 2),         # batch, F larger than needed, 3 row bands
    (1, 64, 384, 16, 16, (3, 3, 3), [2, 2], 0),         # two output-channel tiles of 192
    (1, 192, 96, 12, 16, (1, 1, 1), [2, 2], 0),         # 1x1x1: no history
    (1, 64, 32, 16, 40, (2, 3, 3), [2, 1, 2], 1),       # even temporal extent: one history frame
]


@pytest.mark.parametrize("N,Cin,Cout,H,W,k,chunks,extra", RING_CASES)
def test_layer_on_rings_matches_the_oracle_on_the_whole_sequence(ccv, N, Cin, Cout, H, W, k, chunks, extra):
    """Chunked calls on rings (history in place) against one oracle run over the whole sequence from an empty
    history; the ring output and the NCTHW output of the same call sequence are bit-identical, and both are
    bit-identical to the cache-carrying entry point."""
    Ttot, tc = sum(chunks), k[0] - 1
    c = si.conv_case(N, Cin, Cout, Ttot, H, W, k=k, cache=None, seed=21)
    ref, _ = oracle.forward(c["x"], None, c["w"], c["b"])
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x = to_dev(c["x"])
    Tmax = max(chunks)
    rin = ccv.FrameRing(N, Cin, Tmax + tc + extra, H, W)
    rout = ccv.FrameRing(N, Cout, Tmax + 1, H, W)
    rin.buf.fill_(float("nan"))                           # absent history must never be read
    outs_ring, outs_ncthw, outs_abi = [], [], []
    slot, oslot, pos, cache = 0, 0, 0, None
    for T in chunks:
        xc = x[:, :, pos:pos + T].contiguous()
        rin.load(slot, xc)
        hist = min(tc, pos)
        layer.forward_ring(rin, slot, hist, T, out_ring=rout, out_slot=oslot)
        outs_ring.append(rout.store(oslot, T))
        o = torch.full((N, Cout, T, H, W), float("nan"), dtype=torch.bfloat16, device="cuda")
        layer.forward_ring(rin, slot, hist, T, out=o)
        outs_ncthw.append(o)
        o2, cache = layer(xc, cache)
        outs_abi.append(o2)
        slot, oslot, pos = (slot + T) % rin.F, (oslot + T) % rout.F, pos + T
    torch.cuda.synchronize()
    st, detail = layer.device_status()
    assert st == ccv.OK, (ccv.status_string(st), hex(detail))
    got_ring, got_ncthw, got_abi = (torch.cat(v, dim=2) for v in (outs_ring, outs_ncthw, outs_abi))
    check(as_f64(got_ring), ref, "bf16")
    assert torch.equal(got_ring, got_ncthw)
    assert torch.equal(got_ring, got_abi)
    ctr = layer.counters()
    assert ctr["calls"] == ctr["ok"] and ctr["unsupported"] == ctr["invalid"] == ctr["cuda_error"] == 0
    layer.close()


@pytest.mark.parametrize("N,C,H,W,to_ring", [(1, 64, 20, 24, True), (1, 96, 18, 21, True), (1, 64, 20, 24, False),
                                              (2, 96, 17, 19, False)])
def test_residual_in_the_epilogue_equals_convolution_then_addition(ccv, N, C, H, W, to_ring):
    """out = bf16(float(bf16(conv + b)) + float(res)): checked bit for bit against the un-fused composition (the
    ring call without residual, then a BF16 addition written out in torch), and against the oracle within the
    tolerance of two roundings."""
    T, k = 2, (3, 3, 3)
    c = si.conv_case(N, C, C, T, H, W, k=k, cache="random", seed=22)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    rin = ccv.FrameRing(N, C, T + 2, H, W)
    rin.load(1, cache)                                     # history in slots 1, 2; x in slots 3, 0
    rin.load(3, x)
    plain = torch.empty((N, C, T, H, W), dtype=torch.bfloat16, device="cuda")
    layer.forward_ring(rin, 3, 2, T, out=plain)
    if to_ring:
        rout = ccv.FrameRing(N, C, T, H, W)
        layer.forward_ring(rin, 3, 2, T, out_ring=rout, out_slot=1, res=rin, res_slot=3)
        got = rout.store(1, T)
    else:
        got = torch.full_like(plain, float("nan"))
        layer.forward_ring(rin, 3, 2, T, out=got, res=rin, res_slot=3)
    torch.cuda.synchronize()
    assert torch.equal(got, (plain.float() + x.float()).to(torch.bfloat16))
    ref, _ = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    ref = ref + as_f64(x)
    m = check(as_f64(got), ref, "bf16")
    assert m["max"] <= 2e-2
    layer.close()


@pytest.mark.parametrize("Cin,Cout,H,W,k,T,rt", [(64, 64, 20, 24, (1, 1, 1), 1, 4), (192, 96, 12, 21, (1, 1, 1), 4, 1),
                                                 (64, 32, 18, 20, (3, 3, 3), 2, 2)])
def test_upsample_fused_into_the_store_equals_store_then_upsample(ccv, Cin, Cout, H, W, k, T, rt):
    """ccv3d_forward_ring_up (4*rt strided TMA stores of the epilogue tile) against ccv3d_forward_ring followed by
    ccv3d_upsample_ring: the same bits in the same slots, nothing else of the output ring touched."""
    tc = k[0] - 1
    c = si.conv_case(1, Cin, Cout, T, H, W, k=k, cache="random", seed=25)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    rin = ccv.FrameRing(1, Cin, T + tc, H, W)
    if tc:
        rin.load(0, to_dev(c["cache"]))
    rin.load(tc, to_dev(c["x"]))
    small = ccv.FrameRing(1, Cout, T, H, W)
    want = ccv.FrameRing(1, Cout, T * rt + 1, 2 * H, 2 * W, zero=True)
    got = ccv.FrameRing(1, Cout, T * rt + 1, 2 * H, 2 * W, zero=True)
    st = torch.cuda.current_stream().cuda_stream
    layer.forward_ring(rin, tc, tc, T, out_ring=small)
    assert ccv.ccv3d_upsample_ring(small.c, 0, want.c, 1, T, rt, st) == ccv.OK
    layer.forward_ring(rin, tc, tc, T, out_ring=got, out_slot=1, up_rt=rt)
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK
    assert torch.equal(got.buf, want.buf)
    assert ccv.ccv3d_forward_ring_up(layer.h, rin.c, tc, tc, None, 0, small.c, 0, 1, T, st) == ccv.ERR_INVALID_ARG   # not 2H x 2W
    layer.close()


def test_cta_pairs_on_rings(ccv):
    """192 output channels and enough tiles: the ring calls run on CTA pairs.  Output into a ring, into NCTHW, with
    the residual epilogue and with the upsample fused into the store - each bit for bit what the single-CTA kernel
    writes."""
    c = si.conv_case(1, 192, 192, 2, 90, 100, seed=26)
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    got = {}
    for flags in (0, ccv.FLAG_NO_PAIR):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
        rin = ccv.FrameRing(1, 192, 4, 90, 100)
        rin.load(0, cache)
        rin.load(2, x)
        r1, r2 = ccv.FrameRing(1, 192, 2, 90, 100, zero=True), ccv.FrameRing(1, 192, 2, 180, 200, zero=True)
        out = torch.zeros((1, 192, 2, 90, 100), dtype=torch.bfloat16, device="cuda")
        layer.forward_ring(rin, 2, 2, 2, out_ring=r1, res=rin, res_slot=2)
        layer.forward_ring(rin, 2, 2, 2, out=out)
        layer.forward_ring(rin, 2, 2, 2, out_ring=r2, up_rt=1)
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        got[flags] = (r1.buf.clone(), out.clone(), r2.buf.clone())
        layer.close()
    for a, b in zip(got[0], got[ccv.FLAG_NO_PAIR]):
        assert torch.equal(a, b)
    ref, _ = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    check(as_f64(got[0][1]), ref, "bf16")


@pytest.mark.parametrize("Cin,Cout,T,H,W", [
    (192, 192, 4, 88, 160),     # 240 pair tiles on 74 pairs: three whole waves, then 18 tiles as 36 half-width items
    (64, 384, 2, 64, 96),       # two co-tiles per pixel tile: 96 items, 74 + 22 -> 74 full-width and 44 half-width
    (128, 128, 3, 60, 100),     # 84 items: 74 + 10 -> 20 half-width; ragged tile rows and columns
])
def test_half_width_tail_on_rings(ccv, Cin, Cout, T, H, W):
    """A call whose last wave of tiles would be at most half full finishes with half-width output-channel tiles in
    the same launch.  Ring output with the residual epilogue (where channel counts allow), NCTHW output and the
    upsampling store: bit for bit what the launch without the tail writes, and within tolerance of the oracle."""
    c = si.conv_case(1, Cin, Cout, T, H, W, seed=31)
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    got = {}
    for flags in (0, ccv.FLAG_NO_TAIL_SPLIT):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
        rin = ccv.FrameRing(1, Cin, T + 2, H, W)
        rin.load(0, cache)
        rin.load(2, x)
        r1, r2 = ccv.FrameRing(1, Cout, T, H, W, zero=True), ccv.FrameRing(1, Cout, T, 2 * H, 2 * W, zero=True)
        out = torch.zeros((1, Cout, T, H, W), dtype=torch.bfloat16, device="cuda")
        res = rin if Cin == Cout else None
        layer.forward_ring(rin, 2, 2, T, out_ring=r1, res=res, res_slot=2)
        layer.forward_ring(rin, 2, 2, T, out=out)
        layer.forward_ring(rin, 2, 2, T, out_ring=r2, up_rt=1)
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        got[flags] = (r1.buf.clone(), out.clone(), r2.buf.clone())
        layer.close()
    for a, b in zip(got[0], got[ccv.FLAG_NO_TAIL_SPLIT]):
        assert torch.equal(a, b)
    ref, _ = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    check(as_f64(got[0][1]), ref, "bf16")


def test_ring_argument_errors(ccv):
    c = si.conv_case(1, 64, 64, 2, 16, 16, seed=23)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    rin = ccv.FrameRing(1, 64, 4, 16, 16, zero=True)
    rout = ccv.FrameRing(1, 64, 2, 16, 16)
    out = torch.empty((1, 64, 2, 16, 16), dtype=torch.bfloat16, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    call = lambda *a: ccv.ccv3d_forward_ring(layer.h, *a, st)
    assert call(rin.c, 0, 2, None, 0, rout.c, 0, out.data_ptr(), 2) == ccv.ERR_INVALID_ARG      # two outputs
    assert call(rin.c, 0, 2, None, 0, None, 0, None, 2) == ccv.ERR_INVALID_ARG                  # no output
    assert call(rin.c, 0, 3, None, 0, rout.c, 0, None, 2) == ccv.ERR_INVALID_ARG                # history > kt-1
    assert call(rin.c, 4, 2, None, 0, rout.c, 0, None, 2) == ccv.ERR_INVALID_ARG                # slot out of range
    assert call(rin.c, 0, 2, None, 0, rout.c, 0, None, 3) == ccv.ERR_INVALID_ARG                # F < T + kt - 1
    assert call(rin.c, 0, 2, None, 0, rin.c, 0, None, 2) == ccv.ERR_ALIAS                       # output ring = input ring
    small = ccv.FrameRing(1, 64, 4, 8, 16)
    assert call(rin.c, 0, 2, small.c, 0, rout.c, 0, None, 2) == ccv.ERR_INVALID_ARG             # residual geometry
    r32 = ccv.Ring(rin.buf.data_ptr(), 1, 64, 4, 16, 16, 32)
    assert call(r32, 0, 2, None, 0, rout.c, 0, None, 2) == ccv.ERR_UNSUPPORTED                  # wrong channel block
    assert call(rin.c, 0, 2, None, 0, rout.c, 0, None, 2) == ccv.OK
    torch.cuda.synchronize()
    ctr = layer.counters()
    assert ctr["calls"] == 9 and ctr["ok"] == 1 and ctr["invalid"] == 7 and ctr["unsupported"] == 1
    # the FP32-FMA route has no ring form
    simt = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=ccv.FLAG_FORCE_SIMT)
    assert ccv.ccv3d_forward_ring(simt.h, rin.c, 0, 2, None, 0, rout.c, 0, None, 2, st) == ccv.ERR_UNSUPPORTED
    # layout moves
    assert ccv.ccv3d_ring_load(rin.c, 0, out.data_ptr(), 5, st) == ccv.ERR_INVALID_ARG          # T > F
    assert ccv.ccv3d_ring_store(rin.c, 0, rin.buf.data_ptr(), 2, st) == ccv.ERR_ALIAS
    assert ccv.ccv3d_upsample_ring(rin.c, 0, rout.c, 0, 1, 1, st) == ccv.ERR_INVALID_ARG        # not twice the size
    torch.cuda.synchronize()
    simt.close()
    layer.close()


def test_ring_calls_can_be_captured_in_a_cuda_graph(ccv):
    """The ring entry points allocate nothing and synchronise nothing, so a block of layers can be captured once
    and replayed: layout move, convolution with programmatic dependent launch, convolution with residual,
    upsample.  The replay reproduces the eager result bit for bit, also on new input data."""
    c = si.conv_case(1, 64, 64, 2, 20, 24, seed=24)
    l1 = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    l2 = ccv.CausalConv3d(to_dev(c["w"]), None)
    r1, r2 = ccv.FrameRing(1, 64, 4, 20, 24, zero=True), ccv.FrameRing(1, 64, 4, 20, 24, zero=True)
    r3, r4 = ccv.FrameRing(1, 64, 2, 20, 24), ccv.FrameRing(1, 64, 2, 40, 48)
    xin = to_dev(c["x"]).clone()

    def block():
        r1.load(2, xin)
        l1.forward_ring(r1, 2, 2, 2, out_ring=r2, out_slot=2)
        l2.forward_ring(r2, 2, 2, 2, out_ring=r3, out_slot=0, res=r1, res_slot=2)
        assert ccv.ccv3d_upsample_ring(r3.c, 0, r4.c, 0, 2, 1, torch.cuda.current_stream().cuda_stream) == ccv.OK

    block()
    torch.cuda.synchronize()
    eager = r4.store(0, 2).clone()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(g, stream=side):
        block()
    r4.buf.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(r4.store(0, 2), eager)
    xin.copy_(xin * 0.5)                                   # same graph, new data in the captured buffers
    block()
    torch.cuda.synchronize()
    eager2 = r4.store(0, 2).clone()
    r4.buf.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(r4.store(0, 2), eager2) and not torch.equal(eager2, eager)
    for l in (l1, l2):
        assert l.device_status()[0] == ccv.OK
        l.close()
