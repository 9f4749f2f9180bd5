"""GPU parity for the paper's full supported contract (Eq. (1)-(2) as printed): the layer's own spatial stride,
padding and dilation inside each temporal tap, temporal dilation in the source time, unit temporal stride - on the
FP32-FMA kernel (FP32 layers, BF16 reference route) and on the tensor-core kernel (halo tiles with dilated tap
offsets; spatial stride through one strided TMA box per tap).  Same tolerances as the standard geometry; the cache
update (d_t (kt-1) frames) is bit-exact."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from _util import as_f64, bits, check, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

GUARD = 64


@pytest.fixture(scope="module")
def ccv():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as m
    torch.cuda.set_device(0)
    return m


def _guarded(shape, dtype):
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), float("nan"), dtype=dtype, device="cuda:0")
    return buf, buf[GUARD:GUARD + n].view(shape)


def _intact(buf):
    return bool(torch.isnan(buf[:GUARD]).all() and torch.isnan(buf[-GUARD:]).all())


def _case(N, Cin, Cout, T, H, W, k, dtype, cf, seed):
    c = si.conv_case(N, Cin, Cout, T, H, W, k=k, dtype=dtype, cache=None, seed=seed,
                     x_dist="uniform" if dtype == si.F32 else "normal")
    draw = (lambda shp: si.uniform(shp, -1.0, 1.0, dtype, seed, si.TID_CACHE)) if dtype == si.F32 else \
           (lambda shp: si.normal(shp, 1.0, dtype, seed, si.TID_CACHE))
    c["cache"] = draw((N, Cin, cf, H, W)) if cf else None
    return c


def run_general(ccv, c, stride, pad, dil, dil_t, flags=0, kind=None, stride_t=1):
    kt, kh, kw = c["k"]
    ref, ref_nc = oracle.forward_general(c["x"], c["cache"], c["w"], c["b"], stride=stride, pad=pad, dil=dil, dil_t=dil_t,
                                         stride_t=stride_t)
    tc = dil_t * (kt - 1)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=(stride_t, *stride),
                             dilation=(dil_t, *dil), pad=(tc // 2, *pad))
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    N, Cin, T, H, W = c["x"].shape
    s, To, Ho, Wo, frames = ccv.ccv3d_out_dims(layer.h, T, H, W)
    assert s == ccv.OK and (To, Ho, Wo) == ref.shape[2:] and frames == tc
    odt = torch.float32 if c["dtype"] == si.F32 else torch.bfloat16
    obuf, out = _guarded(ref.shape, odt)
    nbuf, nc = (_guarded((N, Cin, tc, H, W), x.dtype) if tc else (None, None))
    layer(x, cache, out=out, new_cache=nc)
    torch.cuda.synchronize()
    st, detail = layer.device_status()
    assert st == ccv.OK, (ccv.status_string(st), hex(detail))
    assert _intact(obuf) and (nbuf is None or _intact(nbuf)), "guard band overwritten"
    m = check(as_f64(out), ref, kind or ("f32" if c["dtype"] == si.F32 else "bf16"))
    if tc:
        assert np.array_equal(bits(nc), ref_nc), "cache update is not bit-exact"
    ctr = layer.counters()
    assert ctr["calls"] == ctr["ok"] == 1 and ctr["unsupported"] == ctr["invalid"] == ctr["cuda_error"] == 0
    layer.close()
    return m, ctr


GEOMS = [  # k, stride, pad, dil, dil_t
    ((3, 3, 3), (1, 1), (2, 2), (2, 2), 1),     # dilation 2, size preserved
    ((3, 3, 3), (1, 1), (0, 0), (1, 1), 1),     # no padding: output shrinks
    ((3, 3, 3), (1, 1), (1, 1), (1, 1), 2),     # temporal dilation 2: 4 history frames
    ((3, 3, 3), (2, 2), (1, 1), (1, 1), 1),     # spatial stride 2 (downsampling layer)
    ((3, 3, 3), (2, 1), (0, 2), (1, 2), 2),     # everything at once
    ((1, 3, 3), (3, 2), (1, 0), (1, 1), 1),
    ((2, 2, 2), (1, 1), (1, 0), (1, 1), 3),     # even kernels
    ((3, 1, 1), (2, 2), (0, 0), (1, 1), 1),     # strided temporal-only kernel
    ((1, 1, 1), (2, 2), (0, 0), (1, 1), 1),     # strided 1x1x1 (a downsampling shortcut)
    ((3, 5, 3), (1, 2), (3, 1), (1, 1), 1),
]


@pytest.mark.parametrize("k,stride,pad,dil,dil_t", GEOMS)
@pytest.mark.parametrize("cache_mode", ["full", "short", "none"])
def test_fp32_general_geometry(ccv, k, stride, pad, dil, dil_t, cache_mode):
    tc = dil_t * (k[0] - 1)
    cf = {"full": tc, "short": tc // 2, "none": 0}[cache_mode]
    c = _case(2, 5, 7, 3, 13, 18, k, si.F32, cf, seed=31)
    m, ctr = run_general(ccv, c, stride, pad, dil, dil_t)
    assert ctr["simt"] == 1


@pytest.mark.parametrize("k,stride,pad,dil,dil_t", GEOMS)
@pytest.mark.parametrize("Cin,Cout,H,W,cache_mode", [(64, 64, 37, 40, "full"), (96, 48, 20, 27, "short"), (32, 200, 18, 33, "none")])
def test_bf16_tensor_core_general_geometry(ccv, k, stride, pad, dil, dil_t, Cin, Cout, H, W, cache_mode):
    tc = dil_t * (k[0] - 1)
    cf = {"full": tc, "short": tc // 2, "none": 0}[cache_mode]
    c = _case(1, Cin, Cout, 3, H, W, k, si.BF16, cf, seed=32)
    m, ctr = run_general(ccv, c, stride, pad, dil, dil_t)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0


@pytest.mark.parametrize("k,stride,pad,dil,dil_t", [GEOMS[0], GEOMS[3], GEOMS[4]])
def test_bf16_fma_route_general_geometry(ccv, k, stride, pad, dil, dil_t):
    c = _case(1, 24, 20, 2, 11, 14, k, si.BF16, dil_t * (k[0] - 1), seed=33)
    m, ctr = run_general(ccv, c, stride, pad, dil, dil_t, flags=ccv.FLAG_FORCE_SIMT)
    assert ctr["simt"] == 1


@pytest.mark.parametrize("k,stride,pad,dil,dil_t", [GEOMS[2], GEOMS[3], GEOMS[4], GEOMS[7], ((3, 3, 3), (1, 1), (1, 1), (1, 1), 1)])
@pytest.mark.parametrize("stride_t,T", [(2, 4), (2, 5), (3, 4)])
@pytest.mark.parametrize("route", ["f32", "bf16_tc", "bf16_fma"])
def test_temporal_stride(ccv, k, stride, pad, dil, dil_t, stride_t, T, route):
    """Temporal stride (the encoder's temporal downsampling layers; outside the paper's method, which hands them
    back to the framework): output frame o reads Z frames o s_t + k d_t, T_o = floor((T-1)/s_t) + 1."""
    tc = dil_t * (k[0] - 1)
    if route == "f32":
        c = _case(1, 5, 6, T, 9, 12, k, si.F32, tc, seed=37)
    else:
        c = _case(1, 64, 48, T, 20, 24, k, si.BF16, tc // 2 if T == 5 else tc, seed=38)
    m, ctr = run_general(ccv, c, stride, pad, dil, dil_t, flags=ccv.FLAG_FORCE_SIMT if route == "bf16_fma" else 0,
                         stride_t=stride_t)
    assert ctr["tcgen05_bf16" if route == "bf16_tc" else "simt"] == 1


def test_spatial_stride_with_two_samples_and_three_by_two_phases(ccv):
    """The phase-decomposed path with N = 2 and a stride of (3, 2): six phase images per channel block, some with a
    single tap, image extents that are not multiples of the stride."""
    c = _case(2, 64, 48, 3, 29, 38, (3, 3, 3), si.BF16, 2, seed=48)
    m, ctr = run_general(ccv, c, (3, 2), (1, 1), (1, 1), 1)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0


@pytest.mark.parametrize("H,W", [(512, 640), (511, 637)])
def test_spatial_stride_on_many_tiles(ccv, H, W):
    """A downsampling layer (3x3x3, spatial stride 2) on an image of hundreds of tiles: the staging kernel writes the
    phase-decomposed copy (four phase images per channel block; zero rows and columns where the image is not a whole
    number of phases, as with the odd extents here), the convolution kernel reads one halo tile per phase.  Against the
    oracle, cache bit-exact."""
    c = _case(1, 64, 64, 4, H, W, (3, 3, 3), si.BF16, 2, seed=47)
    m, ctr = run_general(ccv, c, (2, 2), (1, 1), (1, 1), 1)
    assert ctr["tcgen05_bf16"] == 1 and ctr["kernel_launches"] == 4            # weight pack, bias, staging, convolution
    print("stride 2,", (H, W), m)


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,cf", [
    (1, 96, 192, 3, 131, 202, 2),      # 32-channel blocks, two pixel blocks per CTA, one accumulator buffer
    (2, 64, 192, 2, 100, 150, 1),      # 64-channel blocks, one pixel block per CTA; two samples, a short cache
    (1, 32, 48, 4, 90, 140, 0),        # narrow tiles with two accumulator buffers; no history at all
    (1, 96, 320, 2, 67, 133, 2),       # two output-channel tiles
])
def test_spatial_stride_two_on_cta_pairs(ccv, N, Cin, Cout, T, H, W, cf):
    """3x3x3 layers with spatial stride 2 and padding 1 that have tiles for the CTA pairs: their convolution kernel takes
    the nine taps in phase order as straight-line code (four halo tiles per channel block, one per phase image).
    Against the oracle, cache bit-exact; and bit for bit the output of the same layer on single CTAs (run-time tap
    loop), whose accumulation order it shares."""
    c = _case(N, Cin, Cout, T, H, W, (3, 3, 3), si.BF16, cf, seed=52 + Cin)
    m, ctr = run_general(ccv, c, (2, 2), (1, 1), (1, 1), 1)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0
    outs = []
    for flags in (0, ccv.FLAG_NO_PAIR):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=(1, 2, 2), pad=(1, 1, 1))
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        outs.append((o, nc))
        layer.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,cf", [
    (1, 96, 48, 16, 252, 320, 2),      # 32-channel blocks, two pixel blocks per CTA (16 KB stager tasks); ragged last tile row
    (1, 64, 192, 16, 128, 160, 1),     # 64-channel blocks, one pixel block per CTA (8 KB tasks); a short cache
    (2, 64, 64, 8, 256, 320, 0),       # two samples, no history
    (1, 64, 64, 1, 896, 1408, 0),      # one frame without history: the absent frame of the updated cache is written as zeros
])
def test_spatial_stride_two_cooperative_staging(ccv, N, Cin, Cout, T, H, W, cf):
    """Stride-2 layers with enough tiles for the default schedule to stage inside the convolution kernel: the stager
    warps write the four phase images of every channel block (even H and W), band by band of 16 input rows ahead of
    the tiles that read them.  Against the oracle, cache bit-exact, and the same bits as the two-kernel schedule on
    single CTAs."""
    c = _case(N, Cin, Cout, T, H, W, (3, 3, 3), si.BF16, cf, seed=61 + Cout)
    m, ctr = run_general(ccv, c, (2, 2), (1, 1), (1, 1), 1)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0
    outs = []
    for flags in (0, ccv.FLAG_TWO_KERNELS | ccv.FLAG_NO_PAIR):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=(1, 2, 2), pad=(1, 1, 1))
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        outs.append((o, nc))
        layer.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


@pytest.mark.parametrize("Cin,Cout,T,H,W,cf", [
    (64, 128, 6, 176, 320, 1),         # few tiles: staging kernel, then the convolution kernel
    (64, 64, 8, 512, 640, 2),          # eight waves of tiles: cooperative staging
])
def test_downsampling_in_time_and_space_on_cta_pairs(ccv, Cin, Cout, T, H, W, cf):
    """Stride (2, 2, 2): the stride-2 kernel on CTA pairs reads Z frame 2 t + dt for output frame t, on both schedules.
    Against the oracle, cache bit-exact, and the same bits as the two-kernel schedule on single CTAs."""
    c = _case(1, Cin, Cout, T, H, W, (3, 3, 3), si.BF16, cf, seed=71)
    m, ctr = run_general(ccv, c, (2, 2), (1, 1), (1, 1), 1, stride_t=2)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0
    outs = []
    for flags in (0, ccv.FLAG_TWO_KERNELS | ccv.FLAG_NO_PAIR):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=(2, 2, 2), pad=(1, 1, 1))
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        outs.append((o, nc))
        layer.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_temporal_stride_cooperative_staging(ccv):
    """A temporal downsampling layer (stride (2, 1, 1), 3x3x3) with enough tiles for the cooperative schedule: all input
    frames are staged inside the kernel, output frame t reads Z frames 2 t + dt.  Against the oracle, cache bit-exact,
    and the same bits as the two-kernel schedule on single CTAs."""
    c = _case(1, 64, 64, 8, 256, 320, (3, 3, 3), si.BF16, 2, seed=83)
    m, ctr = run_general(ccv, c, (1, 1), (1, 1), (1, 1), 1, stride_t=2)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0
    outs = []
    for flags in (0, ccv.FLAG_TWO_KERNELS | ccv.FLAG_NO_PAIR):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=(2, 1, 1))
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        outs.append((o, nc))
        layer.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_streaming_with_temporal_stride_on_gpu(ccv):
    c = _case(1, 64, 32, 8, 20, 24, (3, 3, 3), si.BF16, 0, seed=39)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), stride=(2, 1, 1))
    x = to_dev(c["x"])
    whole, whole_nc = layer(x, None)
    assert whole.shape[2] == 4
    cache, outs = None, []
    for pos, n in ((0, 2), (2, 4), (6, 2)):
        o, cache = layer(x[:, :, pos:pos + n].contiguous(), cache)
        outs.append(o)
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(outs, dim=2), whole) and torch.equal(cache, whole_nc)
    ref, ref_nc = oracle.forward_general(c["x"], None, c["w"], c["b"], stride_t=2)
    check(as_f64(whole), ref, "bf16")
    assert np.array_equal(bits(cache), ref_nc)
    layer.close()


def test_tensor_core_equals_fma_route_closely_on_a_strided_dilated_layer(ccv):
    """Two independent kernels on the same general layer: both within tolerance of the oracle (above), and within
    BF16 rounding of each other."""
    k, stride, pad, dil, dil_t = GEOMS[4]
    c = _case(1, 64, 64, 3, 33, 40, k, si.BF16, dil_t * (k[0] - 1), seed=34)
    outs = []
    for flags in (0, 1):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=(1, *stride), dilation=(dil_t, *dil),
                                 pad=(dil_t * (k[0] - 1) // 2, *pad))
        o, _ = layer(to_dev(c["x"]), to_dev(c["cache"]))
        outs.append(as_f64(o))
        layer.close()
    rms = float(np.sqrt(np.mean(outs[1] ** 2)))
    assert np.abs(outs[0] - outs[1]).max() <= 2e-2 * rms


@pytest.mark.parametrize("chunks", [[1] * 6, [4, 2], [2, 1, 3]])
def test_streaming_equivalence_with_temporal_dilation_on_gpu(ccv, chunks):
    k, dil_t = (3, 3, 3), 2
    c = _case(1, 64, 32, 6, 20, 24, k, si.BF16, 0, seed=35)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), dilation=(dil_t, 1, 1))
    x = to_dev(c["x"])
    whole, whole_nc = layer(x, None)
    cache, outs, pos = None, [], 0
    for n in chunks:
        o, cache = layer(x[:, :, pos:pos + n].contiguous(), cache)
        outs.append(o)
        pos += n
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(outs, dim=2), whole) and torch.equal(cache, whole_nc)
    ref, ref_nc = oracle.forward_general(c["x"], None, c["w"], c["b"], dil_t=dil_t)
    check(as_f64(whole), ref, "bf16")
    assert np.array_equal(bits(cache), ref_nc)
    layer.close()


def test_general_geometry_is_refused_by_the_standard_only_entry_points(ccv):
    c = _case(1, 64, 64, 2, 16, 16, (3, 3, 3), si.BF16, 2, seed=36)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), stride=(1, 2, 2))
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    out = torch.empty((1, 64, 2, 8, 8), dtype=torch.bfloat16, device="cuda")
    nc = torch.empty_like(cache)
    st = torch.cuda.current_stream().cuda_stream
    assert ccv.ccv3d_forward_static(layer.h, x.data_ptr(), cache.data_ptr(), out.data_ptr(), nc.data_ptr(), 1, 2, 16, 16,
                                    st) == ccv.ERR_UNSUPPORTED
    rin, rout = ccv.FrameRing(1, 64, 4, 16, 16, zero=True), ccv.FrameRing(1, 64, 2, 16, 16)
    assert ccv.ccv3d_forward_ring(layer.h, rin.c, 2, 2, None, 0, rout.c, 0, None, 2, st) == ccv.ERR_UNSUPPORTED
    # an input the kernel does not fit into
    tiny = torch.empty((1, 64, 2, 1, 1), dtype=torch.bfloat16, device="cuda")
    valid = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), pad=(1, 0, 0))
    assert ccv.ccv3d_forward(valid.h, tiny.data_ptr(), None, out.data_ptr(), None, 1, 2, 1, 1, st) == ccv.ERR_INVALID_ARG
    torch.cuda.synchronize()
    layer.close()
    valid.close()


# ---------------------------------------------------------------------------- FP32 layers on the tensor cores (3xTF32)
F32_TC_CASES = [
    # N, Cin, Cout, T, H, W, k, cache frames, stride, pad, dil, dil_t, stride_t
    (1, 32, 32, 2, 20, 24, (3, 3, 3), 2, (1, 1), (1, 1), (1, 1), 1, 1),
    (2, 48, 40, 3, 17, 19, (3, 3, 3), 1, (1, 1), (1, 1), (1, 1), 1, 1),      # channels off the block size, short cache, odd W
    (1, 16, 300, 1, 33, 40, (3, 3, 3), 0, (1, 1), (1, 1), (1, 1), 1, 1),     # two output-channel tiles, no history
    (1, 64, 64, 4, 16, 32, (1, 1, 1), 0, (1, 1), (0, 0), (1, 1), 1, 1),      # 1x1x1
    (1, 40, 24, 3, 21, 26, (3, 3, 3), 4, (2, 2), (1, 1), (1, 1), 2, 1),      # strided, temporal dilation
    (1, 32, 48, 4, 18, 20, (2, 3, 3), 1, (1, 1), (2, 2), (2, 2), 1, 2),      # dilated, temporal stride
    (1, 96, 96, 2, 40, 48, (3, 3, 3), 2, (1, 1), (1, 1), (1, 1), 1, 1),      # K = 2592
]


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cf,stride,pad,dil,dil_t,stride_t", F32_TC_CASES)
def test_fp32_on_tensor_cores_3xtf32(ccv, N, Cin, Cout, T, H, W, k, cf, stride, pad, dil, dil_t, stride_t):
    """FP32 layers as three TF32 tensor-core products per FP32 product (hi*hi + hi*lo + lo*hi, FP32 accumulate):
    within the FP32 tolerance (max <= 1e-4 x RMS) of the oracle, cache update bit-exact."""
    c = _case(N, Cin, Cout, T, H, W, k, si.F32, cf, seed=41)
    m, ctr = run_general(ccv, c, stride, pad, dil, dil_t, flags=ccv.FLAG_F32_TENSOR, stride_t=stride_t)
    assert ctr["tcgen05_f32"] == 1 and ctr["tcgen05_bf16"] == 0 and ctr["simt"] == 0
    print("3xTF32", (N, Cin, Cout, T, H, W, k), "K =", Cin * k[0] * k[1] * k[2], m)


def test_fp32_route_selection_by_size(ccv):
    """FP32 calls go to the tensor cores (3xTF32) when they are large (0.2 GFLOP and more) or when K is long enough
    (256 and more) for the FMA kernel's serial walk to lose; short-K small calls stay on the FMA kernel.  Both routes
    within tolerance and close to each other."""
    c = _case(1, 64, 64, 4, 44, 80, (3, 3, 3), si.F32, 2, seed=42)          # 3.1 GFLOP
    ref, ref_nc = oracle.forward_general(c["x"], c["cache"], c["w"], c["b"])
    outs = {}
    for name, flags in (("auto", 0), ("fma", ccv.FLAG_FORCE_SIMT)):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        small, _ = layer(to_dev(c["x"])[:, :, :1, :8, :8].contiguous(), None)    # 2.8 MFLOP, but K = 1728: tensor cores too
        torch.cuda.synchronize()
        ctr = layer.counters()
        assert (ctr["tcgen05_f32"], ctr["simt"], ctr["tcgen05_bf16"]) == ((2, 0, 0) if name == "auto" else (0, 2, 0))
        check(as_f64(o), ref, "f32")
        assert np.array_equal(bits(nc), ref_nc)
        outs[name] = as_f64(o)
        layer.close()
    rms = float(np.sqrt(np.mean(ref ** 2)))
    assert np.abs(outs["auto"] - outs["fma"]).max() <= 1e-4 * rms
    # K = 8 x 27 = 216 and a small call: the FMA kernel
    c2 = _case(1, 8, 16, 2, 12, 20, (3, 3, 3), si.F32, 2, seed=43)
    ref2, _ = oracle.forward_general(c2["x"], c2["cache"], c2["w"], c2["b"])
    layer = ccv.CausalConv3d(to_dev(c2["w"]), to_dev(c2["b"]))
    o2, _ = layer(to_dev(c2["x"]), to_dev(c2["cache"]))
    torch.cuda.synchronize()
    assert layer.counters()["simt"] == 1 and layer.counters()["tcgen05_f32"] == 0
    check(as_f64(o2), ref2, "f32")
    layer.close()


@pytest.mark.parametrize("dist", ["normal", "uniform", "one_sign"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_fp32_default_route_just_under_the_k_limit(ccv, dist, seed):
    """The longest K the automatic FP32 route sends to the tensor cores (K <= 8192; here Cin = 300, 3x3x3: K = 8100)
    on three kinds of data: normal, uniform, and activations and weights all of one sign - the worst case for an
    accumulation that truncates, since the accumulator then sits at full size along the whole chain.  Each within
    the FP32 tolerance of the oracle (max <= 1e-4 x RMS), cache bit-exact; one more channel pair (K = 8208) takes
    the FMA kernel."""
    N, Cin, Cout, T, H, W = 1, 300, 16, 2, 12, 16
    c = _case(N, Cin, Cout, T, H, W, (3, 3, 3), si.F32, 2, seed=80 + seed)
    if dist == "normal":                                       # (the FP32 cases of this file draw uniform activations)
        rng = np.random.default_rng(seed)
        c["x"] = rng.standard_normal(c["x"].shape).astype(np.float32)
        c["cache"] = rng.standard_normal(c["cache"].shape).astype(np.float32)
    elif dist == "one_sign":
        for n in ("x", "cache", "w"):
            c[n] = np.abs(c[n])
    m, ctr = run_general(ccv, c, (1, 1), (1, 1), (1, 1), 1)
    assert ctr["tcgen05_f32"] == 1 and ctr["simt"] == 0
    print("3xTF32 at K = 8100,", dist, seed, m)
    if dist == "normal" and seed == 0:
        c2 = _case(N, 304, Cout, T, H, W, (3, 3, 3), si.F32, 2, seed=90)
        m2, ctr2 = run_general(ccv, c2, (1, 1), (1, 1), (1, 1), 1)
        assert ctr2["simt"] == 1 and ctr2["tcgen05_f32"] == 0


@pytest.mark.parametrize("Cin,Cout,H,W", [(64, 64, 96, 96), (48, 192, 64, 80)])   # two pixel blocks per CTA; one
def test_fp32_on_cta_pairs_equals_single_ctas_bitwise(ccv, Cin, Cout, H, W):
    """The 3xTF32 route on CTA pairs: same passes, same accumulators, same bits as on single CTAs, within the FP32
    tolerance of the oracle."""
    c = _case(1, Cin, Cout, 2, H, W, (3, 3, 3), si.F32, 2, seed=43)
    ref, ref_nc = oracle.forward_general(c["x"], c["cache"], c["w"], c["b"])
    outs = []
    for flags in (ccv.FLAG_F32_TENSOR, ccv.FLAG_F32_TENSOR | ccv.FLAG_NO_PAIR):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK and layer.counters()["tcgen05_f32"] == 1
        assert np.array_equal(bits(nc), ref_nc)
        outs.append(o)
        layer.close()
    check(as_f64(outs[0]), ref, "f32")
    assert torch.equal(outs[0], outs[1])


# ---------------------------------------------------------------------------- optional SiLU epilogue
def _silu64(v):
    return v / (1.0 + np.exp(-v))


@pytest.mark.parametrize("route", ["f32_fma", "bf16_fma", "bf16_tc", "bf16_tc_two_kernels", "bf16_fused", "f32_tc", "bf16_1x1"])
def test_silu_epilogue(ccv, route):
    """out = silu(conv + b) in FP32 before the one output rounding, on every route; the oracle's FP64 output through
    the same function is the reference.  (Not part of the paper's operator: a fused activation for decoder blocks.)"""
    f32 = route.startswith("f32")
    k = (1, 1, 1) if route == "bf16_1x1" else (3, 3, 3)
    shape = (1, 16, 24, 2, 12, 16) if route == "f32_fma" else (1, 64, 96, 4, 160, 192) if route == "bf16_tc" else (1, 64, 96, 2, 40, 48)
    c = _case(*shape, k, si.F32 if f32 else si.BF16, k[0] - 1, seed=44)
    flags = {"f32_fma": 0, "bf16_fma": ccv.FLAG_FORCE_SIMT, "bf16_tc": 0, "bf16_tc_two_kernels": ccv.FLAG_TWO_KERNELS,
             "bf16_fused": ccv.FLAG_FUSED, "f32_tc": ccv.FLAG_F32_TENSOR, "bf16_1x1": 0}[route]
    ref, ref_nc = oracle.forward_general(c["x"], c["cache"], c["w"], c["b"])
    ref = _silu64(ref)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags | ccv.FLAG_EPI_SILU)
    out, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK
    _check_activated(as_f64(out), ref, f32)
    if nc is not None:
        assert np.array_equal(bits(nc), ref_nc)
    layer.close()


def _check_activated(got, ref, f32):
    """SiLU shrinks the RMS of the output (0.64 against 1.05) but not its largest values, so the BF16 tolerance
    "max <= 2e-2 x RMS" no longer covers the rounding of an output in [4, 8) (half a step there is 0.0156 = 2.4e-2 x
    RMS).  The bound is therefore per element: one BF16 rounding (2^-8 relative, a half step with margin) plus the
    accumulation error, and the usual mean bound."""
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    assert np.isfinite(got).all()
    if f32:
        assert err.max() <= 1e-4 * rms
    else:
        assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-3 * rms), float((err / (2.0 ** -8 * np.abs(ref) + 1e-3 * rms)).max())
        assert err.mean() <= 2e-3 * rms


def test_silu_then_residual_on_rings(ccv):
    """Ring epilogue order: activation first, then the residual, each with its own BF16 rounding."""
    c = _case(1, 64, 64, 2, 40, 48, (3, 3, 3), si.BF16, 2, seed=45)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=ccv.FLAG_EPI_SILU)
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    rin = ccv.FrameRing(1, 64, 4, 40, 48)
    rin.load(0, cache)
    rin.load(2, x)
    plain = torch.empty((1, 64, 2, 40, 48), dtype=torch.bfloat16, device="cuda")
    both = torch.empty_like(plain)
    layer.forward_ring(rin, 2, 2, 2, out=plain)
    layer.forward_ring(rin, 2, 2, 2, out=both, res=rin, res_slot=2)
    torch.cuda.synchronize()
    ref, _ = oracle.forward_general(c["x"], c["cache"], c["w"], c["b"])
    _check_activated(as_f64(plain), _silu64(ref), False)
    assert torch.equal(both, (plain.float() + x.float()).to(torch.bfloat16))
    layer.close()
