"""Pins for the oracle of the paper's full supported contract (spatial stride, padding, dilation per temporal tap;
temporal dilation; unit temporal stride - Eq. (1)-(2) as printed): hand-worked values, bit-for-bit reduction to the
already pinned unit-stride oracle, a structurally different numpy routine, the fp64 library conv3d on the explicitly
concatenated and padded input, Eq. (4)'s intervals, and the streaming/causality invariants with temporal dilation."""
import json
import os
import zlib

import numpy as np
import pytest

import oracle
import synth_inputs as si

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_examples_general.json")


def _case(rng, N, Cin, Cout, T, H, W, k, cf, bias=True):
    mk = lambda *s: rng.standard_normal(s).astype(np.float32)
    x, w = mk(N, Cin, T, H, W), mk(Cout, Cin, *k)
    cache = mk(N, Cin, cf, H, W) if cf else None
    return x, cache, w, (mk(Cout) if bias else None)


def test_hand_examples_general():
    g = json.load(open(GOLD))
    for c in g["cases"]:
        for dtype in (np.float32, np.uint16):                     # every value is exact in bf16 too
            conv = (lambda a: si.to_bf16_bits(np.asarray(a, np.float32))) if dtype == np.uint16 else \
                   (lambda a: np.asarray(a, np.float32))
            x = conv(c["x"]).reshape(1, 1, c["T"], 1, c["W"])
            w = conv(c["w"]).reshape(1, 1, *c["k"])
            cache = None if c["cache"] is None else conv(c["cache"]).reshape(1, 1, -1, 1, c["W"])
            st = c.get("stride_t", 1)
            out, nc = oracle.forward_general(x, cache, w, conv(c["b"]), stride=c["stride"], pad=c["pad"], dil=c["dil"],
                                             dil_t=c["dil_t"], stride_t=st)
            assert out.ravel().tolist() == c["out"], c["name"]
            if c["new_cache"] is not None:
                assert si.to_f64(nc).ravel().tolist() == c["new_cache"], c["name"]
            bf, bnc = oracle.brute_force_general(x, cache, w, conv(c["b"]), stride=c["stride"], pad=c["pad"],
                                                 dil=c["dil"], dil_t=c["dil_t"], stride_t=st)
            assert bf.ravel().tolist() == c["out"], c["name"]


@pytest.mark.parametrize("seed", range(6))
def test_reduces_to_the_unit_stride_oracle_bit_for_bit(seed):
    rng = np.random.default_rng(seed)
    k = [(3, 3, 3), (1, 1, 1), (2, 3, 1), (3, 1, 5), (1, 3, 3), (3, 5, 3)][seed]
    cf = (k[0] - 1) if seed % 2 == 0 else 0
    x, cache, w, b = _case(rng, 1 + seed % 2, 3, 4, 1 + seed % 3, 5, 6, k, cf)
    a, nca = oracle.forward(x, cache, w, b)
    g, ncg = oracle.forward_general(x, cache, w, b)
    assert np.array_equal(a, g)
    assert (nca is None and ncg is None) or np.array_equal(nca, ncg)


GEOMS = [  # k, stride, pad, dil, dil_t
    ((3, 3, 3), (2, 2), (1, 1), (1, 1), 1),
    ((3, 3, 3), (1, 1), (2, 2), (2, 2), 1),
    ((3, 3, 3), (1, 1), (0, 0), (1, 1), 1),
    ((3, 3, 3), (1, 1), (1, 1), (1, 1), 2),
    ((2, 3, 3), (2, 1), (0, 2), (1, 2), 3),
    ((3, 1, 1), (1, 1), (0, 0), (1, 1), 2),
    ((1, 3, 3), (3, 2), (1, 0), (1, 1), 1),
    ((3, 5, 3), (2, 2), (3, 1), (1, 2), 2),
]


@pytest.mark.parametrize("k,stride,pad,dil,dil_t", GEOMS)
@pytest.mark.parametrize("cache_mode", ["full", "short", "none"])
@pytest.mark.parametrize("stride_t", [1, 2, 3])
def test_general_against_numpy_routine_and_library_conv3d(k, stride, pad, dil, dil_t, cache_mode, stride_t):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(zlib.crc32(repr((k, stride, pad, dil, dil_t, cache_mode, stride_t)).encode()))
    tc = dil_t * (k[0] - 1)
    cf = {"full": tc, "short": tc // 2, "none": 0}[cache_mode]
    x, cache, w, b = _case(rng, 2, 3, 4, 3 + stride_t, 9, 8, k, cf)
    out, nc = oracle.forward_general(x, cache, w, b, stride=stride, pad=pad, dil=dil, dil_t=dil_t, stride_t=stride_t)
    bf, bnc = oracle.brute_force_general(x, cache, w, b, stride=stride, pad=pad, dil=dil, dil_t=dil_t, stride_t=stride_t)
    scale = np.abs(out).max() + 1.0
    assert out.shape == bf.shape and np.abs(out - bf).max() <= 1e-12 * scale
    if tc:
        assert np.array_equal(nc.astype(np.float64), bnc)
    # the textbook routine this reduces to: the library's conv3d in fp64 on [zeros ; cache ; x] with temporal
    # padding 0, temporal stride 1, dilation (d_t, d_h, d_w)
    parts = [np.zeros((2, 3, tc - cf, 9, 8))] + ([cache.astype(np.float64)] if cf else []) + [x.astype(np.float64)]
    Z = torch.from_numpy(np.concatenate(parts, axis=2))
    ref = torch.nn.functional.conv3d(Z, torch.from_numpy(w.astype(np.float64)), torch.from_numpy(b.astype(np.float64)),
                                     stride=(stride_t, *stride), padding=(0, *pad), dilation=(dil_t, *dil)).numpy()
    assert ref.shape == out.shape and np.abs(out - ref).max() <= 1e-12 * scale


def test_interval_route_with_temporal_dilation_equals_the_definition():
    """Eq. (2)'s sum over temporal taps taken tap by tap over Eq. (4)'s intervals, with d_t in the tap offset: per tap one strided, dilated
    2-D correlation of the source interval, added into the output interval."""
    rng = np.random.default_rng(5)
    k, stride, pad, dil, dil_t = (3, 3, 3), (2, 1), (1, 2), (1, 2), 2
    tc = dil_t * (k[0] - 1)
    for cf in (0, 1, tc):
        x, cache, w, b = _case(rng, 1, 2, 3, 4, 7, 6, k, cf)
        out, _ = oracle.forward_general(x, cache, w, b, stride=stride, pad=pad, dil=dil, dil_t=dil_t)
        Z = np.concatenate(([cache.astype(np.float64)] if cf else []) + [x.astype(np.float64)], axis=2)
        T_o, taps = oracle.tap_intervals(k[0], cf, 4, dil_t)
        assert T_o == 4
        acc = np.zeros_like(out)
        for (kk, o_l, o_h, z_l, z_h) in taps:
            if o_l >= o_h:
                continue
            wk = np.zeros_like(w)
            wk[:, :, 0] = w[:, :, kk]                               # a kt = 1 layer holding W_k
            r, _ = oracle.forward_general(Z[:, :, z_l:z_h].astype(np.float32), None, wk[:, :, :1], None,
                                          stride=stride, pad=pad, dil=dil)
            acc[:, :, o_l:o_h] += r
        acc += b.astype(np.float64)[None, :, None, None, None]
        assert np.abs(acc - out).max() <= 1e-12 * (np.abs(out).max() + 1)


@pytest.mark.parametrize("chunks", [[1, 1, 1, 1, 1, 1], [4, 2], [2, 3, 1]])
def test_streaming_equivalence_with_temporal_dilation(chunks):
    rng = np.random.default_rng(7)
    k, dil_t = (3, 3, 3), 2
    x, _, w, b = _case(rng, 1, 3, 2, sum(chunks), 5, 4, k, 0)
    whole, whole_nc = oracle.forward_general(x, None, w, b, stride=(2, 1), pad=(1, 1), dil_t=dil_t)
    cache, outs, pos = None, [], 0
    for n in chunks:
        o, cache = oracle.forward_general(x[:, :, pos:pos + n], cache, w, b, stride=(2, 1), pad=(1, 1), dil_t=dil_t)
        outs.append(o)
        pos += n
    assert np.array_equal(np.concatenate(outs, axis=2), whole) and np.array_equal(cache, whole_nc)


@pytest.mark.parametrize("chunks", [[2, 2, 2, 2], [4, 4], [6, 2]])
def test_streaming_equivalence_with_temporal_stride(chunks):
    """Chunks whose lengths are multiples of s_t keep the phase of the strided output frames, so chunked calls
    with the cache carried equal the whole-sequence run bit for bit."""
    rng = np.random.default_rng(9)
    x, _, w, b = _case(rng, 1, 3, 2, sum(chunks), 5, 4, (3, 3, 3), 0)
    whole, whole_nc = oracle.forward_general(x, None, w, b, stride_t=2)
    assert whole.shape[2] == sum(chunks) // 2
    cache, outs, pos = None, [], 0
    for n in chunks:
        o, cache = oracle.forward_general(x[:, :, pos:pos + n], cache, w, b, stride_t=2)
        outs.append(o)
        pos += n
    assert np.array_equal(np.concatenate(outs, axis=2), whole) and np.array_equal(cache, whole_nc)


def test_causality_with_temporal_dilation():
    rng = np.random.default_rng(8)
    x, cache, w, b = _case(rng, 1, 2, 2, 5, 4, 4, (3, 3, 3), 4)
    a, _ = oracle.forward_general(x, cache, w, b, dil_t=2)
    x2 = x.copy()
    x2[:, :, 3:] += 1.0
    c, _ = oracle.forward_general(x2, cache, w, b, dil_t=2)
    assert np.array_equal(a[:, :, :3], c[:, :, :3]) and not np.array_equal(a[:, :, 3:], c[:, :, 3:])
