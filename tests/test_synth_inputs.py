"""The seeded input generator: determinism, distribution moments, bf16 rounding."""
import math

import numpy as np

import synth_inputs as si


def test_deterministic_and_sliceable():
    a = si.normal((3, 1000), 1.0, si.F32, seed=0, tid=1)
    b = si.normal((3, 1000), 1.0, si.F32, seed=0, tid=1)
    c = si.normal((3000,), 1.0, si.F32, seed=0, tid=1)
    assert np.array_equal(a, b) and np.array_equal(a.ravel(), c)
    assert not np.array_equal(a, si.normal((3, 1000), 1.0, si.F32, seed=1, tid=1))
    assert not np.array_equal(a, si.normal((3, 1000), 1.0, si.F32, seed=0, tid=2))


def test_moments():
    n = 400000
    u = si.uniform((n,), -1.0, 1.0, si.F32, 0, si.TID_X).astype(np.float64)
    assert abs(u.mean()) < 5e-3 and abs(u.var() - 1 / 3) < 5e-3 and u.min() >= -1 and u.max() <= 1
    g = si.to_f64(si.normal((n,), 2.0, si.BF16, 0, si.TID_W))
    assert abs(g.mean()) < 2e-2 and abs(g.std() - 2.0) < 2e-2
    assert abs(np.mean(g ** 4) / g.var() ** 2 - 3.0) < 0.1


def test_bf16_rounding_is_nearest_even():
    vals = np.array([1.0, 1.00390625, 1.01171875, 1.0 + 2 ** -9, -3.1415927, 65280.0], np.float32)
    bits = si.to_bf16_bits(vals)
    back = si.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.015625 and back[3] == 1.0
    assert abs(back[4] + 3.1415927) <= 2 ** -7 and back[5] == 65280.0


def test_config_case_shapes_and_scaling():
    c = si.conv_case(1, 16, 16, 2, 16, 16, dtype=si.F32, x_dist="uniform")
    assert c["x"].shape == (1, 16, 2, 16, 16) and c["cache"].shape == (1, 16, 2, 16, 16)
    assert c["w"].shape == (16, 16, 3, 3, 3) and c["b"].shape == (16,)
    assert abs(c["w"].astype(np.float64).std() - 1 / math.sqrt(16 * 27)) < 2e-3
    assert si.conv_flops(1, 192, 192, 4, 352, 640, (3, 3, 3)) == 2.0 * 192 * 192 * 27 * 4 * 352 * 640
