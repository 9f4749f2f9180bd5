"""The allocation-free entry point, ccv3d_forward_static, against the ordinary one.

Some callers of this library cannot allocate device memory while they run a layer (a real-time loop that must
not block in the allocator, a host runtime that owns all device memory).  For them the library offers a
variant of the forward call whose staging copy lives in a fixed 32 MiB device array instead of an allocated
workspace.  This test calls it through the C ABI twice in a row - the second call finds the first call's bytes
in the shared array - and checks both results against ccv3d_forward on the same inputs, within the parity
tolerances (BF16: max <= 2e-2 x RMS, mean <= 2e-3 x RMS; cache update bit-exact).  It also checks that a shape
whose staging copy exceeds the array is refused.  Collected last on purpose: a failure here stops nothing else.
"""
import numpy as np
import pytest

import synth_inputs as si
from _util import as_f64, bits, check, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_forward():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as ccv
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    N, Cin, Cout, T, H, W = 1, 96, 64, 3, 40, 48
    c = si.conv_case(N, Cin, Cout, T, H, W, seed=21)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    s, need = ccv.ccv3d_workspace_bytes(layer.h, N, T, H, W)
    assert s == ccv.OK and 0 < need <= 32 << 20

    x1, cache1 = to_dev(c["x"]), to_dev(c["cache"])
    ref1, ref_nc1 = layer(x1, cache1)                         # the ordinary entry point
    # second problem: different data, first chunk (no cache), so the two calls leave different bytes behind
    c2 = si.conv_case(N, Cin, Cout, T, H, W, seed=22, cache=None)
    x2 = to_dev(c2["x"])
    ref2, ref_nc2 = layer(x2, None)
    torch.cuda.synchronize()

    for (x, cache, ref, ref_nc) in ((x1, cache1, ref1, ref_nc1), (x2, None, ref2, ref_nc2)):
        out = torch.full_like(ref, float("nan"))
        nc = torch.full_like(ref_nc, float("nan"))
        s = ccv.ccv3d_forward_static(layer.h, x.data_ptr(), None if cache is None else cache.data_ptr(),
                                     out.data_ptr(), nc.data_ptr(), N, T, H, W, stream)
        assert s == ccv.OK, ccv.status_string(s)
        torch.cuda.synchronize()
        assert layer.device_status()[0] == ccv.OK
        check(as_f64(out), as_f64(ref), "bf16")
        assert np.array_equal(bits(nc), bits(ref_nc)), "cache update differs"

    # a staging copy larger than the fixed array is refused before anything is launched
    big_h, big_w = 512, 512
    s, need = ccv.ccv3d_workspace_bytes(layer.h, N, T, big_h, big_w)
    assert need > 32 << 20
    launches = layer.counters()["kernel_launches"]
    xb = torch.zeros((N, Cin, T, big_h, big_w), dtype=torch.bfloat16, device="cuda:0")
    ob = torch.empty((N, Cout, T, big_h, big_w), dtype=torch.bfloat16, device="cuda:0")
    s = ccv.ccv3d_forward_static(layer.h, xb.data_ptr(), None, ob.data_ptr(), None, N, T, big_h, big_w, stream)
    assert s == ccv.ERR_UNSUPPORTED
    assert layer.counters()["kernel_launches"] == launches
    layer.close()
