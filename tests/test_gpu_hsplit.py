"""Height-split on the CUDA path: all ranks of a layer held by one process on one GPU (the neighbour exchange is a
hand-over of the packed buffers; packing, slab assembly and the layer are the library's).  A band must be
bit-identical to the same rows of the unsplit layer (same kernel, same order of accumulation per output element)
and the whole within the oracle tolerances, over two streamed chunks; plus ccv3d_rows_copy on its own."""
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


@pytest.mark.parametrize("dtype,W,rows,d0,s0", [("bf16", 24, 3, 2, 1), ("bf16", 7, 2, 0, 3), ("f32", 5, 1, 4, 0),
                                                ("f32", 8, 4, 1, 1)])
def test_rows_copy(ccv, dtype, W, rows, d0, s0):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    g = torch.Generator(device="cuda:0").manual_seed(3)
    src = torch.randn((2, 3, 2, 6, W), device="cuda:0", generator=g).to(tdt)
    dst = torch.randn((2, 3, 2, 9, W), device="cuda:0", generator=g).to(tdt)
    want = dst.clone()
    want[..., d0:d0 + rows, :] = src[..., s0:s0 + rows, :]
    st = torch.cuda.current_stream().cuda_stream
    es = src.element_size()
    assert ccv.ccv3d_rows_copy(dst.data_ptr(), 9, d0, src.data_ptr(), 6, s0, 12, rows, W * es, st) == ccv.OK
    assert torch.equal(dst.view(torch.int16 if es == 2 else torch.int32), want.view(torch.int16 if es == 2 else torch.int32))
    want[..., d0:d0 + rows, :] = 0
    assert ccv.ccv3d_rows_copy(dst.data_ptr(), 9, d0, None, 0, 0, 12, rows, W * es, st) == ccv.OK
    assert torch.equal(dst.view(torch.int16 if es == 2 else torch.int32), want.view(torch.int16 if es == 2 else torch.int32))
    # row ranges outside their planes are refused before anything is launched
    assert ccv.ccv3d_rows_copy(dst.data_ptr(), 9, 8, src.data_ptr(), 6, 0, 12, 2, W * es, st) == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_rows_copy(dst.data_ptr(), 9, 0, src.data_ptr(), 6, 5, 12, 2, W * es, st) == ccv.ERR_INVALID_ARG


CASES = [
    # Cin, Cout, T, H, W, k, dilation, dtype, worlds
    (64, 64, 2, 40, 48, (3, 3, 3), (1, 1, 1), si.BF16, (2, 3)),
    (192, 96, 2, 44, 64, (3, 3, 3), (1, 1, 1), si.BF16, (2, 4)),       # bands of 11 rows: slabs of 13
    (32, 64, 3, 30, 40, (3, 5, 3), (1, 2, 1), si.BF16, (3,)),          # dilated 5 taps in h: halo of 4 rows
    (16, 24, 2, 18, 20, (3, 3, 3), (1, 1, 1), si.F32, (2,)),
    (64, 64, 2, 24, 32, (3, 1, 1), (1, 1, 1), si.BF16, (2,)),          # temporal-only kernel: nothing exchanged
    (64, 64, 8, 320, 256, (3, 3, 3), (1, 1, 1), si.BF16, (2,)),        # slabs of 162 rows: large enough for the cooperative schedule
]


@pytest.mark.parametrize("Cin,Cout,T,H,W,k,dil,dtype,worlds", CASES)
def test_bands_equal_unsplit_layer(ccv, Cin, Cout, T, H, W, k, dil, dtype, worlds):
    from paper_2609_31938_b200.hsplit import HSplitCausalConv3d, forward_all_local
    c = si.conv_case(1, Cin, Cout, 2 * T, H, W, k=k, dtype=dtype, cache=None, seed=21,
                     x_dist="uniform" if dtype == si.F32 else "normal")
    pad = tuple(d * (kk - 1) // 2 for d, kk in zip(dil, k))
    kw = dict(pad=(pad[1], pad[2]), dil=(dil[1], dil[2]), dil_t=dil[0])
    x = c["x"]
    ref0, rc = oracle.forward_general(x[:, :, :T], None, c["w"], c["b"], **kw)
    ref1, _ = oracle.forward_general(x[:, :, T:], rc, c["w"], c["b"], **kw)
    ref = np.concatenate([ref0, ref1], axis=2)
    w, b, xd = to_dev(c["w"]), to_dev(c["b"]), to_dev(x)
    whole = ccv.CausalConv3d(w, b, dilation=dil)
    o0, cache = whole(xd[:, :, :T].contiguous(), None)
    o1, _ = whole(xd[:, :, T:].contiguous(), cache)
    unsplit = torch.cat([o0, o1], dim=2)
    check(as_f64(unsplit), ref, "f32" if dtype == si.F32 else "bf16")
    for world in worlds:
        layers = [HSplitCausalConv3d(w, b, H, r, world, dilation=dil) for r in range(world)]
        caches, got = None, []
        for ch in range(2):
            xs = [xd[:, :, ch * T:(ch + 1) * T, l.plan.r0:l.plan.r1].contiguous() for l in layers]
            outs, caches = forward_all_local(layers, xs, caches)
            got.append(torch.cat(outs, dim=3))
        got = torch.cat(got, dim=2)
        torch.cuda.synchronize()
        assert got.shape == unsplit.shape
        assert np.array_equal(bits(got), bits(unsplit)), f"world {world}: bands differ from the unsplit layer"
        for l in layers:
            assert l.conv.device_status()[0] == ccv.OK
            if H >= 320:      # the slab layer (no padding in h) runs on the cooperative schedule, like the unsplit one
                cnt = l.conv.counters()
                assert cnt["calls"] == 2 and cnt["kernel_launches"] == whole.counters()["kernel_launches"], cnt
            l.close()
    whole.close()


@pytest.mark.parametrize("world,C,H,W,spare", [(2, 64, 40, 48, 0), (3, 96, 51, 40, 1), (4, 192, 64, 32, 0), (2, 64, 33, 24, 1)])
def test_ring_block_bands_equal_unsplit(ccv, world, C, H, W, spare):
    """x <- x + conv2(conv1(x)) on frame rings, streamed over three chunks: every rank's band (its rings hold only its
    slab; halo rows re-exchanged after each layer, residual added in the epilogue) is bit-identical to the same rows
    of the unsplit ring path."""
    from paper_2609_31938_b200.hsplit import (HSplitRingConv3d, ring_exchange_all_local, ring_forward_all_local)
    T, chunks = 2, 3
    cs = [si.conv_case(1, C, C, T * chunks, H, W, k=(3, 3, 3), dtype=si.BF16, cache=None, seed=30 + i) for i in range(2)]
    w = [to_dev(c["w"]) for c in cs]
    b = [to_dev(c["b"]) for c in cs]
    x = to_dev(cs[0]["x"])
    F = T + 2 + spare        # spare = 1: five slots, two frames per chunk - the third chunk wraps around inside a call
    # unsplit reference on full-height rings
    L = [ccv.CausalConv3d(w[i], b[i]) for i in range(2)]
    r1, r2 = ccv.FrameRing(1, C, F, H, W, zero=True), ccv.FrameRing(1, C, F, H, W, zero=True)
    ref, slot = [], 0
    for c in range(chunks):
        hist = min(2, c * T)
        r1.load(slot, x[:, :, c * T:(c + 1) * T].contiguous())
        L[0].forward_ring(r1, slot, hist, T, out_ring=r2, out_slot=slot)
        out = torch.empty((1, C, T, H, W), dtype=torch.bfloat16, device="cuda:0")
        L[1].forward_ring(r2, slot, hist, T, out=out, res=r1, res_slot=slot)
        ref.append(out)
        slot = (slot + T) % F
    ref = torch.cat(ref, dim=2)
    # the same block, every rank on its slab
    S = [[HSplitRingConv3d(w[i], b[i], H, r, world) for r in range(world)] for i in range(2)]
    R1 = [l.ring(1, C, F, W) for l in S[0]]
    R2 = [l.ring(1, C, F, W) for l in S[0]]
    got, slot = [], 0
    for c in range(chunks):
        hist = min(2, c * T)
        for r, l in enumerate(S[0]):       # chunk input: the band rows of each rank's ring, then the halos by hand-over
            l.load_band(R1[r], slot, x[:, :, c * T:(c + 1) * T, l.plan.r0:l.plan.r1].contiguous(), exchange=False)
        ring_exchange_all_local(S[0], R1, slot, T)
        ring_forward_all_local(S[0], R1, slot, hist, T, R2, slot)
        got.append(torch.cat([l.forward_out(R2[r], slot, hist, T, res=R1[r], res_slot=slot) for r, l in enumerate(S[1])], dim=3))
        slot = (slot + T) % F
    got = torch.cat(got, dim=2)
    torch.cuda.synchronize()
    assert np.array_equal(bits(got), bits(ref))
    for l in L + S[0] + S[1]:
        assert l.conv.device_status()[0] == ccv.OK if hasattr(l, "conv") else l.device_status()[0] == ccv.OK
        l.close()
