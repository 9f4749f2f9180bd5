"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
the same seeded inputs, element by element.  Tolerances, relative to
RMS(oracle out): FP32 max <= 1e-4; BF16 (FP32 accumulate) max <= 2e-2 and
mean <= 2e-3; the cache update is bit-exact."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from _util import as_f64, bits, check, metrics, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

GUARD = 64  # elements of guard band on each side of out / new_cache


@pytest.fixture(scope="module")
def ccv():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as m
    torch.cuda.set_device(0)
    return m


def _guarded(shape, dtype):
    """A poison-filled buffer with guard bands; returns (whole buffer, view of the payload)."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), float("nan"), dtype=dtype, device="cuda:0")
    return buf, buf[GUARD:GUARD + n].view(shape)


def _guards_intact(buf):
    return bool(torch.isnan(buf[:GUARD]).all() and torch.isnan(buf[-GUARD:]).all())


def run_case(ccv, c, flags=0, out_dtype=None, kind=None):
    """One forward call with poison-filled, guarded outputs; full comparison with the oracle."""
    ref, ref_nc = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, out_dtype=out_dtype)
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    N, Cin, T, H, W = c["x"].shape
    tc = c["k"][0] - 1
    odt = torch.float32 if (c["dtype"] == si.F32 or out_dtype == ccv.F32) else torch.bfloat16
    obuf, out = _guarded(ref.shape, odt)
    nbuf, nc = (_guarded((N, Cin, tc, H, W), x.dtype) if tc else (None, None))
    layer(x, cache, out=out, new_cache=nc)
    torch.cuda.synchronize()
    st, detail = layer.device_status()
    assert st == ccv.OK, (ccv.status_string(st), hex(detail))
    assert _guards_intact(obuf) and (nbuf is None or _guards_intact(nbuf)), "guard band overwritten"
    if kind is None:
        kind = "f32" if c["dtype"] == si.F32 else ("bf16_f32out" if out_dtype == ccv.F32 else "bf16")
    m = check(as_f64(out), ref, kind)                       # NaN poison left behind fails the non-finite check
    if tc:
        assert np.array_equal(bits(nc), ref_nc), "cache update is not bit-exact"
    ctr = layer.counters()
    assert ctr["calls"] == ctr["ok"] == 1 and ctr["unsupported"] == ctr["invalid"] == ctr["cuda_error"] == 0
    layer.close()
    return m, ctr


# ---------------------------------------------------------------------------- FP32
def test_cfg1_fp32(ccv):
    """Configuration 1 on both FP32 routes: the tensor cores by 3xTF32 (the default: K = 432 is long enough for the
    FMA kernel's serial walk to lose) and the plain FMA kernel, each within the FP32 tolerance, cache bit-exact."""
    m, ctr = run_case(ccv, si.conv_case(**si.CONFIGS["cfg1_f32_16"]))
    assert ctr["tcgen05_f32"] == 1 and ctr["tcgen05_bf16"] == 0 and ctr["simt"] == 0 and m["cos"] > 0.9999999
    m, ctr = run_case(ccv, si.conv_case(**si.CONFIGS["cfg1_f32_16"]), flags=ccv.FLAG_FORCE_SIMT)
    assert ctr["simt"] == 1 and m["cos"] > 0.9999999


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache", [
    (2, 3, 5, 3, 7, 9, (3, 3, 3), "random"),
    (1, 16, 16, 1, 5, 13, (3, 3, 3), None),
    (1, 7, 9, 2, 4, 6, (1, 1, 1), None),
    (1, 4, 4, 4, 3, 5, (3, 1, 1), "zeros"),
    (1, 5, 3, 2, 6, 7, (1, 3, 3), None),
    (1, 6, 10, 3, 8, 8, (2, 3, 3), "random"),
])
def test_fp32_shapes(ccv, N, Cin, Cout, T, H, W, k, cache):
    run_case(ccv, si.conv_case(N, Cin, Cout, T, H, W, k=k, dtype=si.F32, cache=cache, seed=3))


# ---------------------------------------------------------------------------- BF16, plain FMA route
@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache", [
    (1, 16, 16, 2, 8, 8, (3, 3, 3), "random"),
    (2, 24, 40, 1, 5, 11, (3, 3, 3), None),
    (1, 32, 8, 3, 6, 6, (1, 1, 1), None),
])
def test_bf16_fma_route(ccv, N, Cin, Cout, T, H, W, k, cache):
    m, ctr = run_case(ccv, si.conv_case(N, Cin, Cout, T, H, W, k=k, cache=cache, seed=4), flags=ccv.FLAG_FORCE_SIMT)
    assert ctr["simt"] == 1 and ctr["tcgen05_bf16"] == 0


# ---------------------------------------------------------------------------- BF16, tensor-core route
TC_CASES = [
    # N, Cin, Cout, T, H,  W,  k,         cache,    bias
    (1, 64, 64, 2, 16, 16, (3, 3, 3), "random", True),     # exactly one tile
    (1, 64, 64, 1, 1, 8, (3, 3, 3), "random", True),       # a single image row, T < kt-1
    (1, 16, 16, 3, 3, 24, (3, 3, 3), "zeros", True),       # Cin below one K block (zero-padded channels)
    (1, 48, 96, 2, 8, 72, (3, 3, 3), "random", False),     # Cin = 32 + 16, no bias
    (1, 96, 96, 4, 44, 80, (3, 3, 3), "random", True),     # 64-byte swizzle route, ragged tile rows
    (1, 96, 192, 5, 20, 24, (3, 3, 3), None, True),        # first chunk, T > kt-1
    (2, 192, 192, 2, 17, 40, (3, 3, 3), "random", True),   # batch 2, H = tile + 1
    (1, 192, 384, 1, 16, 16, (3, 3, 3), "random", True),   # two output-channel tiles
    (1, 64, 80, 2, 16, 32, (3, 3, 3), "random", True),     # Cout % 32 == 16: 16-channel epilogue chunks
    (1, 64, 100, 2, 9, 16, (3, 3, 3), "random", True),     # Cout not a multiple of 16
    (1, 64, 300, 1, 8, 8, (3, 3, 3), None, True),          # two padded output-channel tiles
    (1, 128, 64, 3, 24, 13, (3, 3, 3), "random", True),    # W % 8 != 0: scalar staging, direct-store epilogue
    (1, 64, 64, 2, 5, 7, (3, 3, 3), None, False),          # everything smaller than a tile, odd W
    (1, 192, 96, 2, 32, 48, (1, 1, 1), None, True),        # 1x1x1: per-pixel matmul, no cache (streaming kernel, NCTHW direct)
    (2, 96, 96, 3, 10, 16, (1, 1, 1), None, True),         # 1x1x1 with Cin % 64 != 0: general kernel, one tap
    (2, 128, 80, 3, 10, 24, (1, 1, 1), None, True),        # 1x1x1 streaming kernel: ragged last pixel tile, 16-channel chunks
    (1, 64, 64, 1, 5, 7, (1, 1, 1), None, False),          # 1x1x1 with T*H*W % 8 != 0: general kernel
    (1, 64, 64, 4, 12, 16, (3, 1, 1), "random", True),     # temporal-only kernel
    (1, 64, 64, 2, 18, 24, (1, 3, 3), None, True),         # spatial-only kernel
    (1, 64, 32, 3, 16, 16, (2, 3, 3), "random", True),     # even temporal extent: one cache frame
    (1, 32, 48, 2, 20, 40, (3, 5, 5), "random", True),     # 5x5 spatial: run-time tap loop
    (1, 64, 64, 2, 16, 24, (3, 3, 1), "random", True),     # kh != kw
]


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache,bias", TC_CASES)
def test_bf16_tensor_core_route(ccv, N, Cin, Cout, T, H, W, k, cache, bias):
    m, ctr = run_case(ccv, si.conv_case(N, Cin, Cout, T, H, W, k=k, cache=cache, bias=bias, seed=5))
    assert ctr["tcgen05_bf16"] + ctr["pointwise"] == 1 and ctr["simt"] == 0   # (1x1x1 layers may take the streaming kernel)


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache,bias", [TC_CASES[0], TC_CASES[4], TC_CASES[6], TC_CASES[11]])
def test_bf16_tensor_core_fp32_output(ccv, N, Cin, Cout, T, H, W, k, cache, bias):
    # FP32 output exposes the accumulation itself: FP32 accumulate over K is ~1e-5 x RMS
    run_case(ccv, si.conv_case(N, Cin, Cout, T, H, W, k=k, cache=cache, bias=bias, seed=6), out_dtype=ccv.F32)


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache,bias", [TC_CASES[0], TC_CASES[4], TC_CASES[7], TC_CASES[-2]])
def test_bf16_tensor_core_per_tap_loads(ccv, N, Cin, Cout, T, H, W, k, cache, bias):
    run_case(ccv, si.conv_case(N, Cin, Cout, T, H, W, k=k, cache=cache, bias=bias, seed=7), flags=ccv.FLAG_TC_PER_TAP_A)


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache", [
    (1, 64, 64, 3, 150, 160, (3, 3, 3), "random"),          # 10 tile rows -> 4 bands, ragged last band
    (2, 96, 96, 3, 100, 128, (3, 3, 3), None),
])
def test_bf16_tensor_core_banded_overlap(ccv, N, Cin, Cout, T, H, W, k, cache):
    """Banded schedule on side streams (staging of band k+1 overlaps the convolution of band k): same result,
    bit for bit, as the single-stream schedule."""
    c = si.conv_case(N, Cin, Cout, T, H, W, k=k, cache=cache, seed=13)
    m, ctr = run_case(ccv, c, flags=ccv.FLAG_OVERLAP)
    assert ctr["tcgen05_bf16"] == 1 and ctr["kernel_launches"] > 4          # several staging + convolution launches
    a = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=ccv.FLAG_OVERLAP)
    b = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cache_d = to_dev(c["x"]), to_dev(c["cache"])
    oa, na = a(x, cache_d)
    ob, nb = b(x, cache_d)
    torch.cuda.synchronize()
    assert torch.equal(oa, ob) and torch.equal(na, nb)
    a.close()
    b.close()


FUSED_CASES = [TC_CASES[i] for i in (0, 1, 2, 3, 4, 5, 6, 7, 9, 11, 17, 19, 20, 21)] + [
    (1, 192, 192, 4, 48, 80, (3, 3, 3), "random", True),     # 256-pixel tiles, several waves
    (1, 40, 24, 2, 33, 56, (3, 3, 3), None, True),           # Cin not a multiple of 32: channels beyond Cin arrive as zeros
]


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,k,cache,bias", FUSED_CASES)
def test_bf16_tensor_core_fused_route(ccv, N, Cin, Cout, T, H, W, k, cache, bias):
    """CCV3D_FLAG_FUSED: no staging copy - the kernel reads x and the cache through tensor maps and transposes in
    shared memory; the cache update is a separate copy kernel.  (W % 8 != 0 falls back to the staged route.)"""
    c = si.conv_case(N, Cin, Cout, T, H, W, k=k, cache=cache, bias=bias, seed=15)
    m, ctr = run_case(ccv, c, flags=ccv.FLAG_FUSED)
    assert ctr["tcgen05_bf16"] == 1 and ctr["simt"] == 0


def test_fused_route_equals_staged_route_bitwise(ccv):
    c = si.conv_case(1, 96, 192, 3, 40, 64, seed=16)
    a = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=ccv.FLAG_FUSED)
    b = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cache_d = to_dev(c["x"]), to_dev(c["cache"])
    oa, na = a(x, cache_d)
    ob, nb = b(x, cache_d)
    torch.cuda.synchronize()
    assert torch.equal(oa, ob) and torch.equal(na, nb)          # same K order per output element in both routes
    assert ccv.ccv3d_workspace_bytes(a.h, 1, 3, 40, 64) == (ccv.OK, 0)
    a.close()
    b.close()


@pytest.mark.parametrize("dtype,flags,T", [(si.F32, 0, 3), (si.BF16, 0, 4), (si.BF16, 0, 1), (si.BF16, 8, 4), (si.BF16, 1, 2)])
def test_short_cache_is_zero_history_in_front(ccv, dtype, flags, T):
    """ccv3d_forward_ex with one cache frame and a temporal kernel of 3 (the T_c = 1 calls of the paper's Table 1):
    the missing older frame does not exist, i.e. Eq. (1)-(3) with p_l = 1 - identical to a two-frame cache whose
    first frame is zero, which is what the oracle is given."""
    N, Cin, Cout, H, W = 1, 64, 48, 20, 24
    c = si.conv_case(N, Cin, Cout, T, H, W, dtype=dtype, seed=17)
    short = np.ascontiguousarray(c["cache"][:, :, 1:])                 # the newest history frame only
    padded = c["cache"].copy()
    padded[:, :, 0] = 0
    ref, ref_nc = oracle.forward(c["x"], padded, c["w"], c["b"])
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
    x, cd = to_dev(c["x"]), to_dev(short)
    odt = torch.float32 if dtype == si.F32 else torch.bfloat16
    obuf, out = _guarded(ref.shape, odt)
    nbuf, nc = _guarded((N, Cin, 2, H, W), x.dtype)
    s = ccv.ccv3d_forward_ex(layer.h, x.data_ptr(), cd.data_ptr(), 1, out.data_ptr(), nc.data_ptr(), N, T, H, W,
                             torch.cuda.current_stream().cuda_stream)
    assert s == ccv.OK, ccv.status_string(s)
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK and _guards_intact(obuf) and _guards_intact(nbuf)
    check(as_f64(out), ref, "f32" if dtype == si.F32 else "bf16")
    assert np.array_equal(bits(nc), ref_nc)
    # argument checks of the extended call
    assert ccv.ccv3d_forward_ex(layer.h, x.data_ptr(), cd.data_ptr(), 3, out.data_ptr(), nc.data_ptr(), N, T, H, W) \
        == ccv.ERR_INVALID_ARG
    assert ccv.ccv3d_forward_ex(layer.h, x.data_ptr(), None, 1, out.data_ptr(), nc.data_ptr(), N, T, H, W) \
        == ccv.ERR_INVALID_ARG
    layer.close()


def test_two_samples_on_the_cooperative_schedule(ccv):
    """N = 2 at a size that takes cooperative staging on CTA pairs: the batch is an outer loop of tiles and staging
    tasks with a cache per sample; against the oracle, cache bit-exact; two launches per call (the first two bands of rows go
    through the staging kernel, everything else is the cooperative kernel)."""
    c = si.conv_case(2, 64, 192, 4, 160, 256, seed=19)
    m, ctr = run_case(ccv, c)
    assert ctr["tcgen05_bf16"] == 1 and ctr["kernel_launches"] == 4      # weight pack, bias, head staging, cooperative kernel


def test_cooperative_staging_shared_memory_budget(ccv):
    """A layer whose rings leave room for a third stager slot AND qualify for the third activation slot (temporal-only
    taps, 80 output channels, two pixel blocks per CTA): both extras together must still fit the shared memory of a CTA
    (once they did not, and the launch failed).  Same bits as the two-kernel schedule."""
    c = si.conv_case(1, 128, 80, 5, 257, 888, k=(3, 1, 1), seed=25)
    a = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    b = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=ccv.FLAG_TWO_KERNELS)
    x, cache_d = to_dev(c["x"]), to_dev(c["cache"])
    oa, na = a(x, cache_d)
    ob, nb = b(x, cache_d)
    torch.cuda.synchronize()
    assert a.device_status()[0] == ccv.OK and torch.equal(oa, ob) and torch.equal(na, nb)
    assert np.array_equal(bits(na), np.concatenate([c["cache"], c["x"]], axis=2)[:, :, -2:])
    a.close()
    b.close()


def test_cooperative_staging_with_absent_history(ccv):
    """A first chunk of ONE frame on the cooperative schedule: Z = [absent, absent, x0], and the updated cache is
    [absent ; x0] - a frame of history that never existed, which the stager warps write as zeros (into the staged copy
    and into new_cache) without fetching anything.  Against the oracle, cache bit-exact."""
    c = si.conv_case(1, 64, 64, 1, 704, 640, cache=None, seed=23)
    m, ctr = run_case(ccv, c)
    assert ctr["tcgen05_bf16"] == 1 and ctr["kernel_launches"] == 4      # weight pack, bias, head staging, cooperative kernel


@pytest.mark.parametrize("Cin,Cout,W", [(64, 64, 160), (96, 48, 200), (96, 48, 192)])   # 64-channel blocks; 32-channel blocks with a ragged
                                                                                         # 128-pixel task, and with one whose second box lies beyond the row
def test_bf16_tensor_core_cooperative_staging(ccv, Cin, Cout, W):
    """Large enough for the default schedule to stage inside the convolution kernel (four stager warps per CTA, a
    band of 16 rows ahead of the tiles that read it; only the first two bands are staged by the staging kernel), and
    the same bits as the two-kernel schedule."""
    c = si.conv_case(1, Cin, Cout, 16, 125, W, seed=18)              # 8 tile rows (ragged last), more than eight waves of tiles
    m, ctr = run_case(ccv, c)
    assert ctr["tcgen05_bf16"] == 1 and ctr["kernel_launches"] == 4    # weight pack, bias, head staging, staging + convolution in one launch
    a = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    b = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=ccv.FLAG_TWO_KERNELS)
    x, cache_d = to_dev(c["x"]), to_dev(c["cache"])
    oa, na = a(x, cache_d)
    ob, nb = b(x, cache_d)
    oa2, na2 = a(x[:, :, :3].contiguous(), None)                       # first chunk, T < tile count threshold: two kernels
    torch.cuda.synchronize()
    assert torch.equal(oa, ob) and torch.equal(na, nb)
    assert b.counters()["kernel_launches"] == 4                        # weight pack, bias, staging, convolution
    assert a.device_status()[0] == ccv.OK and bool(torch.isfinite(oa2).all())
    a.close()
    b.close()


def test_cfg2_bf16_384(ccv):
    m, ctr = run_case(ccv, si.conv_case(**si.CONFIGS["cfg2_bf16_384"]))
    assert ctr["tcgen05_bf16"] == 1 and m["cos"] > 0.99998


# ---------------------------------------------------------------------------- exact cases
def test_delta_and_ones_kernels_are_exact_in_bf16(ccv):
    N, Cin, Cout, T, H, W = 1, 64, 64, 3, 20, 24
    c = si.conv_case(N, Cin, Cout, T, H, W, seed=8)
    # small integers: every product and partial sum is exact in FP32 and the result is exact in BF16
    rng = np.random.default_rng(0)
    xi = rng.integers(-3, 4, size=c["x"].shape).astype(np.float32)
    ci = rng.integers(-3, 4, size=c["cache"].shape).astype(np.float32)
    for kind in ("delta", "ones"):
        w = np.zeros((Cout, Cin, 3, 3, 3), np.float32)
        if kind == "delta":
            for co in range(Cout):
                w[co, (co * 7) % Cin, co % 3, (co // 3) % 3, (co // 9) % 3] = 1.0
        else:
            w[:, :2] = 1.0                                   # 54 ones per output channel: |sum| <= 162
        b = rng.integers(-2, 3, size=(Cout,)).astype(np.float32)
        cc = dict(c, x=si.to_bf16_bits(xi), cache=si.to_bf16_bits(ci), w=si.to_bf16_bits(w), b=si.to_bf16_bits(b))
        ref, _ = oracle.forward(cc["x"], cc["cache"], cc["w"], cc["b"])
        layer = ccv.CausalConv3d(to_dev(cc["w"]), to_dev(cc["b"]))
        out, _ = layer(to_dev(cc["x"]), to_dev(cc["cache"]))
        torch.cuda.synchronize()
        assert np.array_equal(as_f64(out), ref), kind
        layer.close()


def test_null_cache_equals_zero_cache_bitwise(ccv):
    c = si.conv_case(1, 96, 96, 3, 24, 32, cache="zeros", seed=9)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x = to_dev(c["x"])
    o0, n0 = layer(x, to_dev(c["cache"]))
    o1, n1 = layer(x, None)
    torch.cuda.synchronize()
    assert torch.equal(o0, o1) and torch.equal(n0, n1)
    x1 = x[:, :, :1].contiguous()                           # T < kt-1 with no history: a zero frame stays in front
    _, n2 = layer(x1, None)
    torch.cuda.synchronize()
    assert np.array_equal(bits(n2), oracle.cache_update(np.ascontiguousarray(c["x"][:, :, :1]), None, 3))
    layer.close()


@pytest.mark.parametrize("chunks", [[1] * 6, [4, 2], [2, 1, 3]])
def test_streaming_equivalence_on_gpu(ccv, chunks):
    """Chunked calls with the cache carried equal one whole-sequence call from an empty history: bit-identical on
    the GPU too (the K order of an output element does not depend on the chunking), and within tolerance of the
    oracle's whole-sequence run."""
    c = si.conv_case(1, 96, 64, 6, 20, 24, cache=None, seed=10)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x = to_dev(c["x"])
    whole, whole_nc = layer(x, None)
    cache, outs, pos = None, [], 0
    for n in chunks:
        o, cache = layer(x[:, :, pos:pos + n].contiguous(), cache)
        outs.append(o)
        pos += n
    torch.cuda.synchronize()
    assert torch.equal(torch.cat(outs, dim=2), whole) and torch.equal(cache, whole_nc)
    ref, ref_nc = oracle.forward(c["x"], None, c["w"], c["b"])
    check(as_f64(whole), ref, "bf16")
    assert np.array_equal(bits(cache), ref_nc)
    layer.close()


# ---------------------------------------------------------------------------- argument checks on a live handle
def test_forward_argument_errors_and_counters(ccv):
    c = si.conv_case(1, 64, 64, 2, 16, 16, seed=11)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    out = torch.empty((1, 64, 2, 16, 16), dtype=torch.bfloat16, device="cuda:0")
    nc = torch.empty_like(cache)
    h = layer.h
    f = lambda *a: ccv.ccv3d_forward(h, *a)
    assert f(x.data_ptr(), cache.data_ptr(), x.data_ptr(), nc.data_ptr(), 1, 2, 16, 16) == ccv.ERR_ALIAS       # out is x
    assert f(x.data_ptr(), cache.data_ptr(), out.data_ptr(), cache.data_ptr(), 1, 2, 16, 16) == ccv.ERR_ALIAS  # in-place cache
    assert f(x.data_ptr(), cache.data_ptr(), out.data_ptr(), out.data_ptr(), 1, 2, 16, 16) == ccv.ERR_ALIAS
    assert f(x.data_ptr() + 2, cache.data_ptr(), out.data_ptr(), nc.data_ptr(), 1, 2, 16, 16) == ccv.ERR_ALIGNMENT
    assert f(None, cache.data_ptr(), out.data_ptr(), nc.data_ptr(), 1, 2, 16, 16) == ccv.ERR_INVALID_ARG
    assert f(x.data_ptr(), cache.data_ptr(), out.data_ptr(), nc.data_ptr(), 1, 0, 16, 16) == ccv.ERR_INVALID_ARG
    assert f(x.data_ptr(), cache.data_ptr(), out.data_ptr(), nc.data_ptr(), 1, 2, 16, 16) == ccv.OK
    torch.cuda.synchronize()
    ctr = layer.counters()
    assert ctr["calls"] == 7 and ctr["ok"] == 1 and ctr["invalid"] == 6 and ctr["tcgen05_bf16"] == 1
    assert layer.device_status()[0] == ccv.OK
    s, ws = ccv.ccv3d_workspace_bytes(h, 1, 2, 16, 16)
    assert s == ccv.OK and ws == 4 * 64 * 16 * 16 * 2
    layer.close()


def test_bounded_wait_reports_a_timeout_and_the_handle_stays_usable(ccv):
    """A wait that can never be satisfied (a barrier nothing signals) gives up after its limit: the kernel
    returns, the status word says where, and the next call on the same handle works."""
    import time
    c = si.conv_case(1, 64, 64, 2, 16, 16, seed=14)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    stream = torch.cuda.current_stream().cuda_stream
    t0 = time.time()
    assert ccv.ccv3d_selftest_wait_timeout(layer.h, 20, stream) == ccv.OK
    torch.cuda.synchronize()
    assert time.time() - t0 < 5.0
    st, detail = layer.device_status()
    assert st == ccv.ERR_DEVICE_TIMEOUT and (detail & 0xFF) == 0x7F
    assert layer.device_status()[0] == ccv.OK                   # reading cleared the word
    assert layer.counters()["device_timeout"] == 1
    ref, ref_nc = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    out, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK
    check(as_f64(out), ref, "bf16")
    assert np.array_equal(bits(nc), ref_nc)
    layer.close()


def test_host_entry_point_matches_device_entry_point(ccv):
    c = si.conv_case(1, 64, 96, 3, 24, 40, seed=12)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    out_d, nc_d = layer(to_dev(c["x"]), to_dev(c["cache"]))
    torch.cuda.synchronize()
    out_h = np.empty((1, 96, 3, 24, 40), np.uint16)
    nc_h = np.empty_like(c["cache"])
    s = ccv.ccv3d_forward_host(layer.h, c["x"].ctypes.data, c["cache"].ctypes.data, out_h.ctypes.data,
                               nc_h.ctypes.data, 1, 3, 24, 40, torch.cuda.current_stream().cuda_stream)
    assert s == ccv.OK
    assert np.array_equal(out_h, bits(out_d)) and np.array_equal(nc_h, bits(nc_d))
    ref, ref_nc = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    check(si.to_f64(out_h), ref, "bf16")
    assert np.array_equal(nc_h, ref_nc)
    layer.close()


@pytest.mark.parametrize("N,Cin,Cout,T,H,W,cache", [(1, 64, 96, 5, 128, 160, "random"), (2, 96, 64, 3, 120, 136, None),
                                                       (1, 64, 64, 2, 160, 200, "random"),
                                                       (1, 64, 96, 3, 352, 640, "random"),     # frames of 43 MB: two bands of rows
                                                       (1, 128, 64, 2, 250, 648, None)])       # two bands of 125 rows (ragged tiles), first chunk
def test_pipelined_host_entry_point(ccv, N, Cin, Cout, T, H, W, cache):
    """Frames of a few MB: the host entry point uploads, convolves (on a frame ring, one frame per call) and
    downloads piece by piece on three streams - whole frames, or bands of rows of a frame (with their halo rows) when
    a frame is tens of MB.  Same bits as the device entry point on the whole tensor, cache update included; pageable
    host memory."""
    c = si.conv_case(N, Cin, Cout, T, H, W, cache=cache, seed=13)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    out_d, nc_d = layer(to_dev(c["x"]), to_dev(c["cache"]))
    torch.cuda.synchronize()
    out_h = np.full((N, Cout, T, H, W), 0x7FC0, np.uint16)
    nc_h = np.full((N, Cin, 2, H, W), 0x7FC0, np.uint16)
    for _ in range(2):                                             # second call: the rotating buffers and events are reused
        s = ccv.ccv3d_forward_host(layer.h, c["x"].ctypes.data, None if c["cache"] is None else c["cache"].ctypes.data,
                                   out_h.ctypes.data, nc_h.ctypes.data, N, T, H, W, torch.cuda.current_stream().cuda_stream)
        assert s == ccv.OK
        assert np.array_equal(out_h, bits(out_d)) and np.array_equal(nc_h, bits(nc_d))
    ctr = layer.counters()
    assert ctr["calls"] == ctr["ok"] == 3 and ctr["kernel_launches"] > 2 * T     # frame-by-frame launches: the pipelined path ran
    layer.close()


def test_host_stream_keeps_the_history_on_the_device(ccv):
    """ccv3d_forward_host_stream: chunks of 3, 1, 1 and 4 frames with nothing but x going up and out coming down give
    the bits of the whole-sequence causal run (and so of ccv3d_forward_host with the cache carried by the caller);
    reset starts over; another host call on the handle in between ends the stream; small frames are refused."""
    N, Cin, Cout, H, W = 1, 64, 96, 128, 160
    lens = [3, 1, 1, 4]
    c = si.conv_case(N, Cin, Cout, sum(lens), H, W, cache=None, seed=14)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    whole, _ = layer(to_dev(c["x"]), None)
    whole = bits(whole)
    st = torch.cuda.current_stream().cuda_stream

    def run(t0, T, reset):
        xc = np.ascontiguousarray(c["x"][:, :, t0:t0 + T])
        out = np.full((N, Cout, T, H, W), 0x7FC0, np.uint16)
        assert ccv.ccv3d_forward_host_stream(layer.h, xc.ctypes.data, out.ctypes.data, reset, N, T, H, W, st) == ccv.OK
        return out

    t0 = 0
    for i, T in enumerate(lens):
        assert np.array_equal(run(t0, T, i == 0), whole[:, :, t0:t0 + T]), f"chunk {i}"
        t0 += T
    # reset: the same first chunk again gives the first frames again (no history)
    assert np.array_equal(run(0, 3, True), whole[:, :, 0:3])
    assert np.array_equal(run(3, 2, False), whole[:, :, 3:5])
    # a non-streaming host call reuses the device buffers: the next stream call starts from no history
    nc = np.empty((N, Cin, 2, H, W), np.uint16)
    o5 = np.empty((N, Cout, 2, H, W), np.uint16)
    x5 = np.ascontiguousarray(c["x"][:, :, 5:7])
    assert ccv.ccv3d_forward_host(layer.h, x5.ctypes.data, None, o5.ctypes.data, nc.ctypes.data, N, 2, H, W, st) == ccv.OK
    first = run(0, 3, False)
    assert np.array_equal(first, whole[:, :, 0:3])
    ref, _ = oracle.forward(c["x"][:, :, :3], None, c["w"], c["b"])
    check(si.to_f64(first), ref, "bf16")
    assert layer.device_status()[0] == ccv.OK
    layer.close()
    small = si.conv_case(1, 64, 64, 2, 16, 16, cache=None, seed=15)
    l2 = ccv.CausalConv3d(to_dev(small["w"]), to_dev(small["b"]))
    o = np.empty((1, 64, 2, 16, 16), np.uint16)
    assert ccv.ccv3d_forward_host_stream(l2.h, small["x"].ctypes.data, o.ctypes.data, 1, 1, 2, 16, 16, st) == ccv.ERR_UNSUPPORTED
    l2.close()


def test_host_stream_in_bands_of_rows(ccv):
    """ccv3d_forward_host_stream with frames large enough for the host pipeline to cut them into bands of rows (three
    here): every band keeps its own history ring on the device between calls; chunks of 2, 1 and 3 frames give the bits of
    the whole-sequence run."""
    N, Cin, Cout, H, W = 1, 128, 64, 352, 640
    lens = [2, 1, 3]
    c = si.conv_case(N, Cin, Cout, sum(lens), H, W, cache=None, seed=24)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    whole, _ = layer(to_dev(c["x"]), None)
    whole = bits(whole)
    st = torch.cuda.current_stream().cuda_stream
    t0 = 0
    for i, T in enumerate(lens):
        xc = np.ascontiguousarray(c["x"][:, :, t0:t0 + T])
        out = np.full((N, Cout, T, H, W), 0x7FC0, np.uint16)
        assert ccv.ccv3d_forward_host_stream(layer.h, xc.ctypes.data, out.ctypes.data, i == 0, N, T, H, W, st) == ccv.OK
        assert np.array_equal(out, whole[:, :, t0:t0 + T]), f"chunk {i}"
        t0 += T
    assert layer.device_status()[0] == ccv.OK
    layer.close()


@pytest.mark.parametrize("shape,rt", [((2, 3, 2, 5, 6), 3), ((1, 4, 3, 6, 8), 4), ((1, 2, 2, 4, 12), 1)])
def test_chain_glue_kernels(ccv, shape, rt):
    """Residual add (exact sum, one RNE rounding) and nearest-neighbour upsampling (exact copies), scalar and
    vector code paths, against their definitions written out in numpy."""
    rng = np.random.default_rng(1)
    a = si.to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    b = si.to_bf16_bits(rng.standard_normal(shape).astype(np.float32))
    da, db = to_dev(a), to_dev(b)
    ybuf, y = _guarded(shape, torch.bfloat16)
    assert ccv.ccv3d_add_bf16(da.data_ptr(), db.data_ptr(), y.data_ptr(), da.numel()) == ccv.OK
    exp = si.to_bf16_bits((si.bf16_bits_to_f32(a) + si.bf16_bits_to_f32(b)).astype(np.float32))
    assert np.array_equal(bits(y), exp)
    N, C, T, H, W = shape
    ubuf, up = _guarded((N, C, T * rt, 2 * H, 2 * W), torch.bfloat16)
    assert ccv.ccv3d_upsample_bf16(da.data_ptr(), up.data_ptr(), N, C, T, H, W, rt) == ccv.OK
    torch.cuda.synchronize()
    assert _guards_intact(ybuf) and _guards_intact(ubuf), "glue kernel wrote outside its output"
    exp_up = np.repeat(np.repeat(np.repeat(a, rt, axis=2), 2, axis=3), 2, axis=4)
    assert np.array_equal(bits(up), exp_up)


# ---------------------------------------------------------------------------- CTA pairs (cta_group::2)
@pytest.mark.parametrize("Cin,Cout,T,H,W,k,flags", [
    (64, 192, 4, 160, 256, (3, 3, 3), 0),                      # cooperative staging on CTA pairs (640 pair tiles)
    (64, 192, 2, 90, 100, (3, 3, 3), 0),                       # two kernels; ragged: the second CTA's columns partly outside
    (96, 160, 2, 70, 72, (3, 3, 3), 16),                       # 32-channel blocks, forced two-kernel schedule
    (128, 384, 1, 96, 96, (3, 3, 3), 0),                       # two output-channel tiles of 192
    (96, 96, 4, 96, 128, (3, 3, 3), 0),                        # narrow output tile: two pixel blocks per CTA, 16x32-pixel tiles
])
def test_cta_pairs_match_the_oracle_and_the_single_cta_kernel(ccv, Cin, Cout, T, H, W, k, flags):
    """Layers with more than 128 output channels per tile run on pairs of CTAs (MMAs with M = 256 issued by the
    leader, each CTA holding half of every weight tile): within tolerance of the oracle, cache bit-exact, and bit
    for bit what the single-CTA kernel computes (the K order of an output element is the same)."""
    c = si.conv_case(1, Cin, Cout, T, H, W, k=k, seed=51)
    m, ctr = run_case(ccv, c, flags=flags)
    assert ctr["tcgen05_bf16"] == 1
    a = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
    b = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags | ccv.FLAG_NO_PAIR)
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    oa, na = a(x, cache)
    ob, nb = b(x, cache)
    torch.cuda.synchronize()
    assert a.device_status()[0] == ccv.OK and b.device_status()[0] == ccv.OK
    assert torch.equal(oa, ob) and (na is None or torch.equal(na, nb))
    a.close()
    b.close()


def test_two_handles_on_two_streams_concurrently(ccv):
    """Handles are independent: two layers issued alternately on two streams (cooperative-staging kernels, which are
    launched cooperatively so that each gets all its CTAs resident) give the results of running them one after the
    other."""
    cases = [si.conv_case(1, 64, 192, 4, 160, 256, seed=61), si.conv_case(1, 64, 64, 8, 125, 160, seed=62)]
    layers = [ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"])) for c in cases]
    xs = [(to_dev(c["x"]), to_dev(c["cache"])) for c in cases]
    want = [l(x, ch) for l, (x, ch) in zip(layers, xs)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    got = [None, None]
    for rep in range(3):
        for i in (0, 1):
            with torch.cuda.stream(streams[i]):
                got[i] = layers[i](xs[i][0], xs[i][1])
    torch.cuda.synchronize()
    for i in (0, 1):
        assert layers[i].device_status()[0] == ccv.OK
        assert torch.equal(got[i][0], want[i][0]) and torch.equal(got[i][1], want[i][1])
        layers[i].close()


def test_random_shapes_every_schedule_agrees(ccv):
    """Seeded random layers (channel counts, kernel shapes, chunk lengths, image sizes, cache lengths): whatever
    schedule the library picks by itself (CTA pairs, half-width tiles, cooperative staging, 1x1x1 streaming kernel)
    gives the bits of the plain two-kernel single-CTA route, run after run, with a clean device status."""
    import random
    rnd = random.Random(20261125)
    g = torch.Generator(device="cuda:0").manual_seed(11)
    ref_flags = ccv.FLAG_TWO_KERNELS | ccv.FLAG_NO_PAIR
    done = 0
    while done < 60:
        Cin, Cout = rnd.choice([32, 64, 96, 128, 192, 256, 384]), rnd.choice([32, 64, 96, 128, 192, 256, 384])
        k = rnd.choice([(3, 3, 3), (3, 3, 3), (1, 3, 3), (3, 1, 1), (1, 1, 1), (2, 3, 3)])
        T = rnd.randint(1, 5)
        big = rnd.random() < 0.25
        H = rnd.randint(64, 300) if big else rnd.randint(8, 90)
        W = 8 * (rnd.randint(20, 64) if big else rnd.randint(2, 24))
        if Cin * Cout * T * H * W * k[0] * k[1] * k[2] > 2e12:
            continue
        cf = rnd.randint(0, k[0] - 1)
        w = (torch.randn((Cout, Cin) + k, device="cuda:0", generator=g) / (Cin * k[0] * k[1] * k[2]) ** 0.5).to(torch.bfloat16)
        b = torch.randn((Cout,), device="cuda:0", generator=g).to(torch.bfloat16)
        x = torch.randn((1, Cin, T, H, W), device="cuda:0", generator=g).to(torch.bfloat16)
        cache = torch.randn((1, Cin, cf, H, W), device="cuda:0", generator=g).to(torch.bfloat16) if cf else None
        res = []
        for flags in (0, 0, ref_flags):
            layer = ccv.CausalConv3d(w, b, flags=flags)
            o, nc = layer(x, cache)
            torch.cuda.synchronize()
            assert layer.device_status()[0] == ccv.OK, (Cin, Cout, k, T, H, W, cf, flags)
            res.append((o, nc))
            layer.close()
        for o, nc in res[:2]:
            assert torch.equal(o, res[2][0]), (Cin, Cout, k, T, H, W, cf)
            assert nc is None or torch.equal(nc, res[2][1]), (Cin, Cout, k, T, H, W, cf)
        done += 1


@pytest.mark.parametrize("Cin,Cout,T,H,W", [(128, 128, 3, 60, 100), (64, 384, 2, 64, 96)])
def test_half_width_tail_through_ncthw(ccv, Cin, Cout, T, H, W):
    """Mid-size layers on CTA pairs whose last wave of tiles is at most half full (84 = 74 + 10 and 96 = 74 + 22 items)
    end the launch with half-width tiles: same bits as without (CCV3D_FLAG_NO_TAIL_SPLIT), within tolerance of the
    oracle, cache bit-exact."""
    c = si.conv_case(1, Cin, Cout, T, H, W, seed=41)
    ref, ref_nc = oracle.forward(c["x"], c["cache"], c["w"], c["b"])
    outs = []
    for flags in (0, ccv.FLAG_NO_TAIL_SPLIT):
        layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
        o, nc = layer(to_dev(c["x"]), to_dev(c["cache"]))
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        assert np.array_equal(bits(nc), ref_nc)
        outs.append(o)
        layer.close()
    assert torch.equal(outs[0], outs[1])
    check(as_f64(outs[0]), ref, "bf16")


def test_call_log_line():
    """CCV3D_LOG=1: one line per call on stderr with the entry point, the shape, the status and the route counters
    (read at create time, so the layer is made in a child process)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import torch, paper_2609_31938_b200 as ccv\n"
        "w = torch.randn(64, 64, 3, 3, 3, device='cuda').bfloat16()\n"
        "l = ccv.CausalConv3d(w)\n"
        "x = torch.randn(1, 64, 2, 16, 24, device='cuda').bfloat16()\n"
        "l(x, None); torch.cuda.synchronize()\n"
        "print(ccv.ccv3d_forward(l.h, None, None, None, None, 1, 2, 16, 24))\n")
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, CCV3D_LOG="1"), capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stderr.splitlines() if l.startswith("ccv3d ")]
    assert len(lines) == 2, r.stderr
    assert "ccv3d_forward_ex N=1 T=2 H=16 W=24 64->64 k=3x3x3: CCV3D_OK" in lines[0] and "tcgen05 1" in lines[0]
    assert "CCV3D_ERR_INVALID_ARG" in lines[1] and "calls 2" in lines[1]
