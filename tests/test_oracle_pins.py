"""Pins for the CPU oracle: everything here runs without a GPU and compares the
oracle with something other than itself - hand-worked values, a structurally
different brute-force routine, Eq. (2) read frame by frame with a library 2-D correlation, the
fp64 library conv3d on the explicitly concatenated input, and the invariants
the operator must satisfy (causality, streaming equivalence, linearity,
1x1x1 = per-pixel matmul, delta kernel, NULL cache = zero cache)."""
import json
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")


def _rand_case(rng, N, Cin, Cout, T, H, W, k, cache=True, bias=True, dtype=np.float32):
    kt = k[0]
    mk = lambda *s: rng.standard_normal(s).astype(np.float32)
    x, w = mk(N, Cin, T, H, W), mk(Cout, Cin, *k)
    c = mk(N, Cin, kt - 1, H, W) if (cache and kt > 1) else None
    b = mk(Cout) if bias else None
    if dtype == np.uint16:
        x, w = si.to_bf16_bits(x), si.to_bf16_bits(w)
        c = None if c is None else si.to_bf16_bits(c)
        b = None if b is None else si.to_bf16_bits(b)
    return x, c, w, b


# ------------------------------------------------------------------ hand-worked values
def test_hand_examples():
    g = json.load(open(GOLD))
    for c in g["cases"]:
        kt, kh, kw = c["k"]
        for dtype in (np.float32, np.uint16):       # all values are exact in bf16 too
            conv = (lambda a: si.to_bf16_bits(np.asarray(a, np.float32))) if dtype == np.uint16 else \
                   (lambda a: np.asarray(a, np.float32))
            x = conv(c["x"]).reshape(1, c["Cin"], c["T"], c["H"], c["W"])
            w = conv(c["w"]).reshape(c["Cout"], c["Cin"], kt, kh, kw)
            b = conv(c["b"])
            cache = None if c["cache"] is None else conv(c["cache"]).reshape(1, c["Cin"], kt - 1, c["H"], c["W"])
            out, nc = oracle.forward(x, cache, w, b)
            assert out.ravel().tolist() == c["out"], c["name"]
            if c["new_cache"] is not None:
                assert si.to_f64(nc).ravel().tolist() == c["new_cache"], c["name"]
            pts = oracle.points(x, cache, w, b, np.arange(out.size))
            assert pts.tolist() == c["out"], c["name"]


def test_interval_algebra_matches_worked_cases_and_brute_force():
    g = json.load(open(GOLD))["intervals"]
    for c in g["cases"]:
        T_o, taps = oracle.tap_intervals(3, c["cache_frames"], c["T"])
        assert T_o == c["T"]
        assert [[k, ol, oh] for (k, ol, oh, _, _) in taps] == c["taps"]
    # Eq. (4) against direct enumeration of Eq. (1) for a range of kernels, dilations, caches
    for kt in (1, 2, 3):
        for dil in (1, 2):
            for nC in range(0, dil * (kt - 1) + 1):
                for T in range(1, 6):
                    T_o, taps = oracle.tap_intervals(kt, nC, T, dil)
                    p_l = dil * (kt - 1) - nC
                    for (k, ol, oh, zl, zh) in taps:
                        valid = [o for o in range(T_o) if 0 <= o + k * dil - p_l < nC + T]
                        assert valid == list(range(ol, max(ol, oh)))
                        assert zh - zl == oh - ol


# ------------------------------------------------------------------ independent routines
@pytest.mark.parametrize("seed", range(12))
def test_brute_force_and_points_agree(seed):
    rng = np.random.default_rng(seed)
    N, Cin, Cout = rng.integers(1, 3), rng.integers(1, 6), rng.integers(1, 6)
    T, H, W = rng.integers(1, 5), rng.integers(1, 7), rng.integers(1, 7)
    k = tuple(int(v) for v in rng.choice([1, 3], size=3))
    dtype = np.uint16 if seed % 2 else np.float32
    x, c, w, b = _rand_case(rng, N, Cin, Cout, T, H, W, k, cache=bool(seed % 3), bias=bool(seed % 4), dtype=dtype)
    out, nc = oracle.forward(x, c, w, b)
    ref, ref_nc = oracle.brute_force(x, c, w, b)
    scale = np.abs(si.to_f64(w)).sum() * np.abs(si.to_f64(x)).max() + 1.0
    assert np.max(np.abs(out - ref)) <= 1e-12 * scale
    if k[0] > 1:
        assert np.array_equal(si.to_f64(nc), ref_nc)
    pts = oracle.points(x, c, w, b, np.arange(out.size))
    assert np.array_equal(pts.reshape(out.shape), out)      # same order of summation -> identical


@pytest.mark.parametrize("cache_frames", [2, 1, 0])
@pytest.mark.parametrize("T", [1, 2, 4])
def test_eq2_frame_by_frame_with_library_conv2d(cache_frames, T):
    """Eq. (2) as a statement about single frames: output frame t is the bias plus, for every temporal tap k, the
    2-D correlation (the library's, fp64) of Z frame q_k(t) = t + k - p_l of Eq. (1) with W[:, :, k]; a tap whose
    source time falls outside Z contributes nothing.  Z = [C ; X], p_l = (kt-1) - |C|.  No intervals, no batching:
    a different route to the same numbers than the oracle's loops, and the temporal index is written here from
    Eq. (1), not taken from the oracle."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(100 + T)
    x, c, w, b = _rand_case(rng, 2, 3, 4, T, 5, 6, (3, 3, 3), cache=True)
    kt = 3
    p_l = (kt - 1) - cache_frames
    Z = x if cache_frames == 0 else np.concatenate([c[:, :, kt - 1 - cache_frames:], x], axis=2)
    # the oracle's interface takes a full-length cache: absent older frames are zeros in front
    c_full = None if cache_frames == 0 else c.copy()
    if cache_frames == 1:
        c_full[:, :, 0] = 0
    out, _ = oracle.forward(x, c_full, w, b)
    Zt, wt = torch.from_numpy(Z.astype(np.float64)), torch.from_numpy(w.astype(np.float64))
    ref = np.zeros_like(out)
    for t in range(T):
        acc = torch.from_numpy(b.astype(np.float64))[None, :, None, None].expand(2, 4, 5, 6).clone()
        for k in range(kt):
            q = t + k - p_l
            if 0 <= q < Z.shape[2]:
                acc = acc + torch.nn.functional.conv2d(Zt[:, :, q], wt[:, :, k], padding=1)
        ref[:, :, t] = acc.numpy()
    assert np.max(np.abs(out - ref)) <= 1e-12 * (np.abs(out).max() + 1)


@pytest.mark.parametrize("k", [(3, 3, 3), (1, 1, 1), (3, 1, 1), (1, 3, 3)])
def test_library_conv3d_fp64(k):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(7)
    x, c, w, b = _rand_case(rng, 2, 5, 7, 3, 9, 11, k)
    out, _ = oracle.forward(x, c, w, b)
    z = np.concatenate([c, x], axis=2) if c is not None else x
    ref = torch.nn.functional.conv3d(torch.from_numpy(z.astype(np.float64)), torch.from_numpy(w.astype(np.float64)),
                                     torch.from_numpy(b.astype(np.float64)), stride=1,
                                     padding=(0, (k[1] - 1) // 2, (k[2] - 1) // 2)).numpy()
    assert ref.shape == out.shape
    assert np.max(np.abs(out - ref)) <= 1e-12 * (np.abs(ref).max() + 1)


# ------------------------------------------------------------------ invariants
def test_causality():
    rng = np.random.default_rng(1)
    x, c, w, b = _rand_case(rng, 1, 4, 3, 5, 6, 6, (3, 3, 3))
    out, _ = oracle.forward(x, c, w, b)
    for t in range(4):
        x2 = x.copy()
        x2[:, :, t + 1:] += rng.standard_normal(x2[:, :, t + 1:].shape).astype(np.float32)
        out2, _ = oracle.forward(x2, c, w, b)
        assert np.array_equal(out2[:, :, :t + 1], out[:, :, :t + 1])
        assert not np.array_equal(out2[:, :, t + 1:], out[:, :, t + 1:])


@pytest.mark.parametrize("chunks", [[1] * 7, [4, 3], [2, 1, 4], [7], [1, 2, 1, 3]])
@pytest.mark.parametrize("dtype", [np.float32, np.uint16])
def test_streaming_equivalence(chunks, dtype):
    rng = np.random.default_rng(2)
    x, _, w, b = _rand_case(rng, 2, 3, 4, 7, 5, 4, (3, 3, 3), cache=False, dtype=dtype)
    whole, whole_nc = oracle.forward(x, None, w, b)
    cache, outs, pos = None, [], 0
    for n in chunks:
        o, cache = oracle.forward(np.ascontiguousarray(x[:, :, pos:pos + n]), cache, w, b)
        outs.append(o)
        pos += n
    assert np.array_equal(np.concatenate(outs, axis=2), whole)      # bit-identical
    assert np.array_equal(cache, whole_nc)
    assert np.array_equal(cache, x[:, :, -2:])                      # the last kt-1 input frames
    assert np.array_equal(oracle.cache_update(x, None, 3), x[:, :, -2:])
    c1 = oracle.cache_update(np.ascontiguousarray(x[:, :, :1]), None, 3)
    assert np.array_equal(oracle.cache_update(np.ascontiguousarray(x[:, :, 1:2]), c1, 3), x[:, :, :2])


def test_linearity_in_x_and_w():
    rng = np.random.default_rng(3)
    x1, c1, w, b = _rand_case(rng, 1, 3, 3, 3, 5, 5, (3, 3, 3), dtype=np.float32)
    x2, c2, w2, _ = _rand_case(rng, 1, 3, 3, 3, 5, 5, (3, 3, 3), dtype=np.float32)
    a, be = np.float32(2.0), np.float32(-0.5)            # exact scalings keep the inputs representable
    bd = b.astype(np.float64)[None, :, None, None, None]
    o1, _ = oracle.forward(x1, c1, w, b)
    o2, _ = oracle.forward(x2, c2, w, b)
    o12, _ = oracle.forward(a * x1 + be * x2, a * c1 + be * c2, w, b)
    # fp32 rounding of the input combination is the only inexact step: recompute it in fp64 via linearity of the oracle's widened inputs
    xs, cs = (a * x1 + be * x2), (a * c1 + be * c2)
    resid = (xs.astype(np.float64) - (2.0 * x1.astype(np.float64) - 0.5 * x2.astype(np.float64)))
    assert np.abs(resid).max() < 1e-6
    tol = 1e-6 * np.abs(w).sum() + 1e-12
    assert np.max(np.abs((o12 - bd) - (2.0 * (o1 - bd) - 0.5 * (o2 - bd)))) <= tol
    ow, _ = oracle.forward(x1, c1, w2, b)
    ows, _ = oracle.forward(x1, c1, (a * w + be * w2), b)
    assert np.max(np.abs((ows - bd) - (2.0 * (o1 - bd) - 0.5 * (ow - bd)))) <= 1e-5 * np.abs(x1).sum() / x1.size * w.size


def test_pointwise_kernel_is_per_pixel_matmul():
    rng = np.random.default_rng(4)
    x, _, w, b = _rand_case(rng, 2, 6, 5, 3, 4, 7, (1, 1, 1), cache=False)
    out, nc = oracle.forward(x, None, w, b)
    assert nc is None
    W2 = w.reshape(5, 6).astype(np.float64)
    for n in range(2):
        X2 = x[n].reshape(6, -1).astype(np.float64)
        ref = (W2 @ X2 + b.astype(np.float64)[:, None]).reshape(5, 3, 4, 7)
        assert np.max(np.abs(out[n] - ref)) <= 1e-12 * (np.abs(ref).max() + 1)


def test_delta_kernel_is_shifted_input_plus_bias():
    rng = np.random.default_rng(5)
    Cin, Cout, T, H, W = 3, 4, 3, 5, 6
    x, c, _, b = _rand_case(rng, 1, Cin, Cout, T, H, W, (3, 3, 3))
    z = np.concatenate([c, x], axis=2).astype(np.float64)
    for (ci0, co0, dt, dh, dw) in [(0, 0, 0, 0, 0), (2, 3, 2, 1, 1), (1, 2, 1, 2, 0), (2, 1, 0, 0, 2)]:
        w = np.zeros((Cout, Cin, 3, 3, 3), np.float32)
        w[co0, ci0, dt, dh, dw] = 1.0
        out, _ = oracle.forward(x, c, w, b)
        zp = np.zeros((T + 2, H + 2, W + 2))
        zp[:, 1:H + 1, 1:W + 1] = z[0, ci0]
        exp = zp[dt:dt + T, dh:dh + H, dw:dw + W] + float(b[co0])
        assert np.array_equal(out[0, co0], exp)
        others = [co for co in range(Cout) if co != co0]
        assert np.array_equal(out[0, others], np.broadcast_to(b[others].astype(np.float64)[:, None, None, None],
                                                             (Cout - 1, T, H, W)))


def test_null_cache_equals_zero_cache():
    rng = np.random.default_rng(6)
    for dtype in (np.float32, np.uint16):
        x, _, w, b = _rand_case(rng, 2, 3, 3, 2, 4, 5, (3, 3, 3), cache=False, dtype=dtype)
        zc = np.zeros((2, 3, 2, 4, 5), dtype=x.dtype)
        o1, n1 = oracle.forward(x, None, w, b)
        o2, n2 = oracle.forward(x, zc, w, b)
        assert np.array_equal(o1, o2) and np.array_equal(n1, n2)
    # T < kt-1 with no history: the new cache keeps a zero frame in front
    x1 = np.ascontiguousarray(x[:, :, :1])
    _, n3 = oracle.forward(x1, None, w, b)
    assert np.array_equal(n3[:, :, 0], np.zeros_like(n3[:, :, 0])) and np.array_equal(n3[:, :, 1], x1[:, :, 0])


def test_bf16_inputs_are_widened_exactly():
    rng = np.random.default_rng(8)
    x, c, w, b = _rand_case(rng, 1, 3, 2, 2, 4, 4, (3, 3, 3), dtype=np.uint16)
    o16, n16 = oracle.forward(x, c, w, b)
    f = si.bf16_bits_to_f32
    o32, n32 = oracle.forward(f(x), f(c), f(w), f(b))
    assert np.array_equal(o16, o32)
    assert np.array_equal(f(n16), n32)
