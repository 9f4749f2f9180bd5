"""A workspace lent by the caller (ccv3d_set_workspace): one staging buffer for many layers, no allocation inside
ccv3d_forward, calls legal inside a stream capture.

The lowering's extra memory is what Section 7.2 of the paper names as its remaining overhead; here the only such
buffer is the channels-last staging copy, and a decoder of many layers needs one of the largest single need, not
one per layer."""
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


# eight layers of different shapes, dtypes and routes that stage: BF16 two-kernel and cooperative, FP32 as 3xTF32,
# a width TMA cannot address, a general geometry
LAYERS = [
    dict(Cin=64, Cout=64, T=2, H=24, W=40),
    dict(Cin=96, Cout=48, T=3, H=20, W=27),                       # W % 8 != 0
    dict(Cin=192, Cout=96, T=2, H=32, W=48),
    dict(Cin=32, Cout=200, T=1, H=18, W=32, cache=None),          # first chunk
    dict(Cin=64, Cout=64, T=4, H=160, W=256),                     # enough waves for cooperative staging
    dict(Cin=48, Cout=32, T=2, H=20, W=24, dtype="f32"),          # 3xTF32
    dict(Cin=64, Cout=32, T=3, H=21, W=24, stride=(1, 2, 2)),     # spatial stride 2
    dict(Cin=128, Cout=128, T=2, H=16, W=16, flags="NO_PAIR"),
]


def _make(ccv, spec, seed):
    dt = si.F32 if spec.get("dtype") == "f32" else si.BF16
    c = si.conv_case(1, spec["Cin"], spec["Cout"], spec["T"], spec["H"], spec["W"], dtype=dt, seed=seed,
                     cache=spec.get("cache", "random"))
    flags = ccv.FLAG_F32_TENSOR if dt == si.F32 else 0
    if spec.get("flags") == "NO_PAIR":
        flags |= ccv.FLAG_NO_PAIR
    stride = spec.get("stride", (1, 1, 1))
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags, stride=stride)
    return c, layer, stride


def test_eight_handles_share_one_workspace(ccv):
    cases = [_make(ccv, spec, 60 + i) for i, spec in enumerate(LAYERS)]
    needs = []
    for c, layer, _ in cases:
        N, _, T, H, W = c["x"].shape
        s, need = ccv.ccv3d_workspace_bytes(layer.h, N, T, H, W)
        assert s == ccv.OK and need > 0
        needs.append(need)
    ws = torch.empty(max(needs) + 256, dtype=torch.uint8, device="cuda:0")
    base = (ws.data_ptr() + 255) // 256 * 256
    # results with each handle's own workspace first (the existing path), then all on the shared one
    own = [layer(to_dev(c["x"]), to_dev(c["cache"])) for c, layer, _ in cases]
    torch.cuda.synchronize()
    for c, layer, _ in cases:
        assert ccv.ccv3d_set_workspace(layer.h, base, max(needs)) == ccv.OK
    for rep in range(2):                                      # in turn, twice: every call finds another layer's bytes
        for (c, layer, stride), (o_own, nc_own) in zip(cases, own):
            x, cache = to_dev(c["x"]), to_dev(c["cache"])
            out = torch.full_like(o_own, float("nan"))
            nc = torch.full_like(nc_own, float("nan"))
            layer(x, cache, out=out, new_cache=nc)
            torch.cuda.synchronize()
            assert layer.device_status()[0] == ccv.OK
            assert torch.equal(out, o_own) and torch.equal(nc, nc_own)
            if rep == 0:
                ref, ref_nc = oracle.forward_general(c["x"], c["cache"], c["w"], c["b"], stride=stride[1:])
                check(as_f64(out), ref, "f32" if c["dtype"] == si.F32 else "bf16")
                assert np.array_equal(bits(nc), ref_nc)
    # a workspace that is too small is an error before anything is launched, not an allocation
    c, layer, _ = cases[4]
    launches = layer.counters()["kernel_launches"]
    assert ccv.ccv3d_set_workspace(layer.h, base, needs[4] - 256) == ccv.OK
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    with pytest.raises(ccv.Ccv3dError) as e:
        layer(x, cache)
    assert e.value.status == ccv.ERR_NOMEM and layer.counters()["kernel_launches"] == launches
    assert ccv.ccv3d_set_workspace(layer.h, base + 16, needs[4]) == ccv.ERR_ALIGNMENT
    # and taking it back returns the handle to its own workspace
    assert ccv.ccv3d_set_workspace(layer.h, None, 0) == ccv.OK
    o2, _ = layer(x, cache)
    torch.cuda.synchronize()
    assert torch.equal(o2, own[4][0])
    for _, layer, _ in cases:
        layer.close()
    del ws


@pytest.mark.parametrize("flags_name", ["default", "TWO_KERNELS"])
def test_forward_on_a_lent_workspace_is_legal_inside_stream_capture(ccv, flags_name):
    """With a lent workspace ccv3d_forward enqueues kernels (and one memset of the band counters) and nothing else:
    a capture of two calls replays to the same bits as the eager calls."""
    flags = ccv.FLAG_TWO_KERNELS if flags_name == "TWO_KERNELS" else 0
    c = si.conv_case(1, 64, 64, 4, 160, 256, seed=71)          # large enough for cooperative staging by default
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]), flags=flags)
    x, cache = to_dev(c["x"]), to_dev(c["cache"])
    ref, ref_nc = layer(x, cache)
    ref2, _ = layer(x, ref_nc)
    torch.cuda.synchronize()
    s, need = ccv.ccv3d_workspace_bytes(layer.h, 1, 4, 160, 256)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda:0")
    assert ccv.ccv3d_set_workspace(layer.h, (ws.data_ptr() + 255) // 256 * 256, need) == ccv.OK
    out, nc = torch.empty_like(ref), torch.empty_like(ref_nc)
    out2, nc2 = torch.empty_like(ref), torch.empty_like(ref_nc)
    layer(x, cache, out=out, new_cache=nc)                     # warm-up outside the capture (kernel attributes, tensor maps)
    torch.cuda.synchronize()
    out.zero_(); nc.zero_()
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        g.capture_begin()
        layer(x, cache, out=out, new_cache=nc)
        layer(x, nc, out=out2, new_cache=nc2)
        g.capture_end()
    torch.cuda.synchronize()
    for _ in range(2):
        out.zero_(); out2.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        assert torch.equal(out, ref) and torch.equal(nc, ref_nc) and torch.equal(out2, ref2)
    layer.close()
