"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times: the outputs are too
many for the CPU oracle to compute whole, so it evaluates sampled output elements one dot product at a time
(random samples plus the corners and seams of the kernel's 16 x 16-pixel tiles); the cache update is compared
whole, bit for bit."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from _util import bits, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _sample_indices(shape, n_random, seed):
    N, C, T, H, W = shape
    rng = np.random.default_rng(seed)
    idx = [rng.integers(0, int(np.prod(shape)), size=n_random, dtype=np.int64)]
    hs = sorted({0, 1, 15, 16, 17, H // 2, H - 17, H - 16, H - 1} & set(range(H)))
    ws = sorted({0, 1, 7, 8, 15, 16, 17, W // 2, W - 9, W - 8, W - 1} & set(range(W)))
    cs = sorted({0, 1, 31, 32, C // 2, C - 1} & set(range(C)))
    g = np.stack(np.meshgrid(np.arange(N), cs, np.arange(T), hs, ws, indexing="ij"), axis=-1).reshape(-1, 5)
    idx.append(np.ravel_multi_index(g.T, shape).astype(np.int64))
    return np.unique(np.concatenate(idx))


@pytest.mark.parametrize("name,cache", [
    ("cfg3_bf16_192", "random"),
    ("cfg3_bf16_192", None),              # the first-chunk form of configuration 3
    ("cfg4a_bf16_96", "random"),
    ("cfg4b_bf16_192_96", "random"),
    ("cfg4c_bf16_pw_192_96", None),
])
def test_full_size_sampled(name, cache):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as ccv
    torch.cuda.set_device(0)
    cfg = dict(si.CONFIGS[name])
    c = si.conv_case(cache=cache, **cfg)
    kt = c["k"][0]
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cch = to_dev(c["x"]), to_dev(c["cache"])
    out, nc = layer(x, cch)
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK
    ctr = layer.counters()
    assert ctr["ok"] == 1 and (ctr["pointwise"] if c["k"] == (1, 1, 1) else ctr["tcgen05_bf16"]) == 1

    idx = _sample_indices(tuple(out.shape), 3000, seed=1)
    got = out.view(-1)[torch.from_numpy(idx).cuda()].float().cpu().numpy().astype(np.float64)
    ref = oracle.points(c["x"], c["cache"], c["w"], c["b"], idx)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    assert np.isfinite(got).all()
    assert err.max() <= 2e-2 * rms, (err.max() / rms, idx[np.argmax(err)])
    assert err.mean() <= 2e-3 * rms, err.mean() / rms
    # nothing left unwritten anywhere (the output buffer came from torch.empty): finite everywhere, and its
    # overall RMS is that of the sampled oracle values
    assert bool(torch.isfinite(out).all())
    assert abs(float(out.float().pow(2).mean().sqrt()) / rms - 1.0) < 0.05
    if kt > 1:
        assert np.array_equal(bits(nc), oracle.cache_update(c["x"], c["cache"], kt)), "cache update is not bit-exact"
    layer.close()
    del out, nc, x, cch
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["cfg3_bf16_192", "cfg4a_bf16_96"])
def test_full_size_on_frame_rings_sampled(name):
    """The resident-activation path at the benchmark's full sizes, in the launch configuration bench.py's
    `resident` leg times: input and history in a frame ring, output into a frame ring.  Sampled outputs against
    the oracle, and the whole output bit for bit against the NCTHW entry point."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as ccv
    torch.cuda.set_device(0)
    cfg = dict(si.CONFIGS[name])
    c = si.conv_case(cache="random", **cfg)
    kt = c["k"][0]
    N, Cin, T, H, W = c["x"].shape
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cch = to_dev(c["x"]), to_dev(c["cache"])
    rin = ccv.FrameRing(N, Cin, T + kt - 1, H, W)
    rout = ccv.FrameRing(N, cfg["Cout"], T, H, W)
    rout.buf.fill_(float("nan"))
    rin.load(T, cch)                       # slots T, T+1 hold the history; x wraps around to slots 0 .. T-1
    rin.load((T + kt - 1) % rin.F, x)
    layer.forward_ring(rin, (T + kt - 1) % rin.F, kt - 1, T, out_ring=rout, out_slot=0)
    out = rout.store(0, T)
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK
    idx = _sample_indices(tuple(out.shape), 3000, seed=2)
    got = out.view(-1)[torch.from_numpy(idx).cuda()].float().cpu().numpy().astype(np.float64)
    ref = oracle.points(c["x"], c["cache"], c["w"], c["b"], idx)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    assert np.isfinite(got).all() and bool(torch.isfinite(out).all())
    assert err.max() <= 2e-2 * rms and err.mean() <= 2e-3 * rms, (err.max() / rms, err.mean() / rms)
    del rin, rout
    torch.cuda.empty_cache()
    abi, _ = layer(x, cch)
    torch.cuda.synchronize()
    assert torch.equal(out, abi)
    layer.close()
    del out, abi, x, cch
    torch.cuda.empty_cache()


def test_more_than_2_31_elements():
    """Maximum sizes: x and out hold 2.26e9 elements each (offsets beyond 32 bits in the staging pass, the TMA
    coordinates of the convolution and its stores), x, out, caches and the staged copy take 19 GB of the device.
    Sampled outputs - random over the whole range plus the last channel's last frame, whose offsets are the
    largest - against the oracle; the cache update whole, bit for bit."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2609_31938_b200 as ccv
    torch.cuda.set_device(0)
    N, Cin, Cout, T, H, W, k = 1, 64, 64, 5, 2304, 3072, (3, 3, 3)
    assert N * Cin * T * H * W > 2 ** 31 and N * Cout * T * H * W > 2 ** 31
    c = si.conv_case(N, Cin, Cout, T, H, W, k=k, dtype=si.BF16, cache="random", seed=0)
    layer = ccv.CausalConv3d(to_dev(c["w"]), to_dev(c["b"]))
    x, cch = to_dev(c["x"]), to_dev(c["cache"])
    out, nc = layer(x, cch)
    torch.cuda.synchronize()
    assert layer.device_status()[0] == ccv.OK and layer.counters()["tcgen05_bf16"] == 1
    shape = tuple(out.shape)
    rng = np.random.default_rng(3)
    tail = np.ravel_multi_index(np.stack(np.meshgrid([0], [Cout - 1], [T - 1], [0, 1, H // 2, H - 2, H - 1],
                                                     [0, 1, W // 2, W - 9, W - 1], indexing="ij"), -1).reshape(-1, 5).T, shape)
    idx = np.unique(np.concatenate([rng.integers(0, int(np.prod(shape)), size=4000, dtype=np.int64), tail.astype(np.int64)]))
    assert idx.max() > 2 ** 31
    got = out.view(-1)[torch.from_numpy(idx).cuda()].float().cpu().numpy().astype(np.float64)
    ref = oracle.points(c["x"], c["cache"], c["w"], c["b"], idx)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    assert np.isfinite(got).all()
    assert err.max() <= 2e-2 * rms and err.mean() <= 2e-3 * rms, (err.max() / rms, err.mean() / rms, idx[np.argmax(err)])
    for t in range(T):                      # nothing left unwritten (frame by frame: no 9 GB temporary)
        assert bool(torch.isfinite(out[:, :, t]).all())
    assert np.array_equal(bits(nc), oracle.cache_update(c["x"], c["cache"], k[0])), "cache update is not bit-exact"
    layer.close()
    del out, nc, x, cch
    torch.cuda.empty_cache()
