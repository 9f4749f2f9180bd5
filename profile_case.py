"""Run a few forward calls of one layer shape on cuda:0 - a small, self-ending program to put under a profiler.

    python profile_case.py --cin 192 --cout 192 --t 4 --h 176 --w 320 [--k 3 3 3] [--calls 3] [--ring]
                           [--stride 1 2 2] [--dilation 1 2 2]

Inputs are the seeded synthetic tensors of the benchmark (normal activations, fan-in-scaled weights).
"""
import argparse
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def main():
    import torch
    import synth_inputs as si
    import paper_2609_31938_b200 as ccv
    ap = argparse.ArgumentParser()
    ap.add_argument("--cin", type=int, default=192)
    ap.add_argument("--cout", type=int, default=192)
    ap.add_argument("--t", type=int, default=4)
    ap.add_argument("--h", type=int, default=176)
    ap.add_argument("--w", type=int, default=320)
    ap.add_argument("--k", type=int, nargs=3, default=[3, 3, 3])
    ap.add_argument("--calls", type=int, default=3)
    ap.add_argument("--no-cache", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="CCV3D_FLAG_* bits (16 = two-kernel schedule, 8 = fused route)")
    ap.add_argument("--ring", action="store_true", help="resident activations: input and output in frame rings")
    ap.add_argument("--f32", action="store_true", help="FP32 layer (tensor cores by 3xTF32 when the call is large enough)")
    ap.add_argument("--stride", type=int, nargs=3, default=[1, 1, 1], help="(s_t, s_h, s_w)")
    ap.add_argument("--dilation", type=int, nargs=3, default=[1, 1, 1], help="(d_t, d_h, d_w); size-preserving padding")
    a = ap.parse_args()
    c = si.conv_case(1, a.cin, a.cout, a.t, a.h, a.w, k=tuple(a.k), cache=None if a.no_cache else "random",
                     dtype=si.F32 if a.f32 else si.BF16)
    if a.f32:
        up = lambda v: None if v is None else torch.from_numpy(v).cuda()
    else:
        up = lambda v: None if v is None else torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16)
    layer = ccv.CausalConv3d(up(c["w"]), up(c["b"]), flags=a.flags, stride=tuple(a.stride), dilation=tuple(a.dilation))
    x, cache = up(c["x"]), up(c["cache"])
    if cache is not None and a.dilation[0] > 1:        # the history is d_t (kt-1) frames long
        cache = torch.cat([cache] * a.dilation[0], dim=2).contiguous()
    _, To, Ho, Wo, _ = ccv.ccv3d_out_dims(layer.h, a.t, a.h, a.w)
    out = torch.empty((1, a.cout, To, Ho, Wo), dtype=torch.float32 if a.f32 else torch.bfloat16, device="cuda")
    nc = torch.empty_like(cache) if cache is not None else None
    if a.ring:
        tc = a.k[0] - 1
        rin = ccv.FrameRing(1, a.cin, a.t + tc, a.h, a.w)
        rout = ccv.FrameRing(1, a.cout, a.t, a.h, a.w)
        if cache is not None:
            rin.load(0, cache)
        rin.load(tc, x)
        slot = tc
        for _ in range(a.calls):
            layer.forward_ring(rin, slot, tc if cache is not None else 0, a.t, out_ring=rout)
            slot = (slot + a.t) % rin.F
    else:
        for _ in range(a.calls):
            layer(x, cache, out=out, new_cache=nc)
    torch.cuda.synchronize()
    st, detail = layer.device_status()
    assert st == ccv.OK, (ccv.status_string(st), hex(detail))
    print("ok", layer.counters())


if __name__ == "__main__":
    main()
