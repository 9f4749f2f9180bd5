"""The allocation-free entry point, ccv3d_forward_static, against the oracle and the ordinary entry point.

Some callers of this library cannot allocate device memory while they run a layer (a real-time loop that must
not block in the allocator, a host runtime that owns all device memory).  For them the library offers a
variant of the forward call whose staging copy lives in a fixed 32 MiB device array instead of an allocated
workspace.  These tests call it through the C ABI twice in a row - the second call finds the first call's bytes
in the shared array - and hold both results to the CPU oracle within the parity tolerances (BF16: max <= 2e-2 x
RMS, mean <= 2e-3 x RMS; FP32 output of a BF16 layer: max <= 2e-4 x RMS; cache update bit-exact) and, bit for bit,
to ccv3d_forward on a handle that runs the same two kernels (the order of accumulation per output element is the
same).  They cover both channel-block sizes, a width TMA cannot address, a chunk shorter than the history with no
cache, FP32 output and a 1x1x1 layer; that the second call changes the free device memory by nothing; and that a
shape whose staging copy exceeds the array is refused.  Collected last on purpose: a failure here stops nothing else.
"""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from _util import as_f64, bits, check, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

CASES = [  # Cin, Cout, T, H, W, k, out_f32
    (96, 64, 3, 40, 48, (3, 3, 3), False),     # 32-channel blocks
    (64, 96, 2, 24, 40, (3, 3, 3), False),     # 64-channel blocks
    (64, 64, 2, 20, 27, (3, 3, 3), False),     # W % 8 != 0: scalar staging loads, direct-store epilogue
    (64, 32, 1, 16, 24, (3, 3, 3), False),     # T < kt-1
    (64, 48, 2, 16, 32, (3, 3, 3), True),      # FP32 output
    (128, 64, 2, 16, 24, (1, 1, 1), False),    # 1x1x1: no history at all
]


def _static(ccv, layer, x, cache, out, nc, dims, stream):
    N, T, H, W = dims
    return ccv.ccv3d_forward_static(layer.h, x.data_ptr(), None if cache is None else cache.data_ptr(), out.data_ptr(),
                                    None if nc is None else nc.data_ptr(), N, T, H, W, stream)


@pytest.mark.parametrize("Cin,Cout,T,H,W,k,out_f32", CASES)
def test_static_scratch_entry_point_matches_oracle_and_forward(Cin, Cout, T, H, W, k, out_f32):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as ccv
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    N, tc = 1, k[0] - 1
    odt = ccv.F32 if out_f32 else None
    kind = "bf16_f32out" if out_f32 else "bf16"
    # two problems: with a cache, then different data as a first chunk (no cache), so that the two calls leave
    # different bytes behind in the shared array
    c1 = si.conv_case(N, Cin, Cout, T, H, W, k=k, seed=21)
    c2 = si.conv_case(N, Cin, Cout, T, H, W, k=k, seed=22, cache=None)
    layer = ccv.CausalConv3d(to_dev(c1["w"]), to_dev(c1["b"]), out_dtype=odt)
    plain = ccv.CausalConv3d(to_dev(c1["w"]), to_dev(c1["b"]), out_dtype=odt,
                             flags=ccv.FLAG_TWO_KERNELS | ccv.FLAG_NO_PAIR)
    free_before_second = None
    for i, c in enumerate((c1, c2)):
        x, cache = to_dev(c["x"]), to_dev(c["cache"])
        ref, ref_nc = oracle.forward(c["x"], c["cache"], c1["w"], c1["b"])
        fwd, fwd_nc = plain(x, cache)                          # the ordinary entry point, same two kernels
        out = torch.full_like(fwd, float("nan"))
        nc = torch.full_like(fwd_nc, float("nan")) if tc else None
        torch.cuda.synchronize()
        if i == 1:
            free_before_second = torch.cuda.mem_get_info()[0]
        s = _static(ccv, layer, x, cache, out, nc, (N, T, H, W), stream)
        assert s == ccv.OK, ccv.status_string(s)
        torch.cuda.synchronize()
        if i == 1:
            assert torch.cuda.mem_get_info()[0] == free_before_second, "the call changed the free device memory"
        assert layer.device_status()[0] == ccv.OK
        check(as_f64(out), ref, kind)                          # NaN poison left behind fails the non-finite check
        if k != (1, 1, 1):                                     # (ccv3d_forward serves 1x1x1 layers with another kernel)
            assert torch.equal(out, fwd), "differs from ccv3d_forward"
        if tc:
            assert np.array_equal(bits(nc), ref_nc), "cache update differs from the oracle's"
    ctr = layer.counters()
    assert ctr["calls"] == ctr["ok"] == 2 and ctr["tcgen05_bf16"] == 2
    layer.close()
    plain.close()


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as ccv
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    N, Cin, Cout, T = 1, 96, 64, 3
    c = si.conv_case(N, Cin, Cout, T, 8, 8, seed=23)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    # a staging copy larger than the fixed array is refused before anything is launched:
    # N (kt-1+T) cin_pad H W 2 bytes = 5 x 96 x 512 x 512 x 2 = 240 MiB
    big_h, big_w = 512, 512
    assert N * (2 + T) * 96 * big_h * big_w * 2 > 32 << 20
    launches = layer.counters()["kernel_launches"]
    xb = torch.zeros((N, Cin, T, big_h, big_w), dtype=torch.bfloat16, device="cuda:0")
    ob = torch.empty((N, Cout, T, big_h, big_w), dtype=torch.bfloat16, device="cuda:0")
    s = ccv.ccv3d_forward_static(layer.h, xb.data_ptr(), None, ob.data_ptr(), None, N, T, big_h, big_w, stream)
    assert s == ccv.ERR_UNSUPPORTED
    assert layer.counters()["kernel_launches"] == launches
    # FP32 layers have no tensor-core staging copy to replace
    cf = si.conv_case(1, 8, 8, 2, 8, 8, dtype=si.F32, seed=24)
    lf = ccv.CausalConv3d(to_dev(cf["w"]), to_dev(cf["b"]), flags=ccv.FLAG_FORCE_SIMT)
    xf = to_dev(cf["x"])
    of = torch.empty((1, 8, 2, 8, 8), dtype=torch.float32, device="cuda:0")
    assert ccv.ccv3d_forward_static(lf.h, xf.data_ptr(), None, of.data_ptr(), None, 1, 2, 8, 8, stream) == ccv.ERR_UNSUPPORTED
    layer.close()
    lf.close()
