"""Pins for the oracle's specified elementary functions against double-precision libm."""
import numpy as np

import oracle


def ulp_err(approx, true64):
    t32 = true64.astype(np.float32)
    ulp = np.maximum(np.spacing(np.abs(t32)).astype(np.float64), 2.0 ** -149)
    return np.abs(approx.astype(np.float64) - true64) / ulp


def test_sin_cos_accuracy():
    rng = np.random.default_rng(0)
    for lo, hi in [(-0.25, 0.25), (-np.pi, np.pi), (-13, 13), (-1000, 1000), (-1e4, 1e4)]:
        x = rng.uniform(lo, hi, 200_000).astype(np.float32)
        x64 = x.astype(np.float64)
        assert ulp_err(oracle.map_f32("sin", x), np.sin(x64)).max() <= 2.0
        assert ulp_err(oracle.map_f32("cos", x), np.cos(x64)).max() <= 2.0
    # absolute accuracy over the full stated domain |x| < 1e6
    x = rng.uniform(-1e6, 1e6, 200_000).astype(np.float32)
    assert np.abs(oracle.map_f32("sin", x) - np.sin(x.astype(np.float64))).max() < 1e-6


def test_sincos_exact_identities():
    s, c = oracle.sincos_s(0.0)
    assert s == 0.0 and c == 1.0
    rng = np.random.default_rng(1)
    x = rng.uniform(-20, 20, 50_000).astype(np.float32)
    assert np.array_equal(oracle.map_f32("sin", -x).view(np.uint32), (-oracle.map_f32("sin", x)).view(np.uint32))
    assert np.array_equal(oracle.map_f32("cos", -x).view(np.uint32), oracle.map_f32("cos", x).view(np.uint32))
    # every quadrant: sin and cos swap roles and signs as the angle passes multiples of pi/2
    for q in range(-6, 7):
        xq = np.float32(q * np.pi / 2 + 0.3)
        s, c = oracle.sincos_s(xq)
        assert abs(float(s) - np.sin(float(xq))) < 3e-7 and abs(float(c) - np.cos(float(xq))) < 3e-7
    # sin_s / cos_s are the two halves of sincos_s
    for v in (0.1, 1.7, -2.9, 5.5):
        s, c = oracle.sincos_s(v)
        assert oracle.sin_s(v) == s and oracle.cos_s(v) == c


def test_exp_accuracy_and_clamp():
    rng = np.random.default_rng(2)
    for lo, hi in [(-1, 1), (0, 18), (-87, 88)]:
        y = rng.uniform(lo, hi, 200_000).astype(np.float32)
        assert ulp_err(oracle.map_f32("exp", y), np.exp(y.astype(np.float64))).max() <= 1.5
    assert oracle.exp_s(0.0) == 1.0
    assert oracle.exp_s(1000.0) == oracle.exp_s(88.0)
    assert oracle.exp_s(-1000.0) == oracle.exp_s(-87.0)
    assert np.isfinite(oracle.exp_s(88.0)) and oracle.exp_s(-87.0) > 0


def test_tanh_accuracy_and_symmetry():
    rng = np.random.default_rng(3)
    for lo, hi in [(-0.01, 0.01), (-1, 1), (-5, 5), (-12, 12)]:
        x = rng.uniform(lo, hi, 200_000).astype(np.float32)
        err = np.abs(oracle.map_f32("tanh", x).astype(np.float64) - np.tanh(x.astype(np.float64)))
        assert err.max() <= 2e-7
    x = rng.uniform(-12, 12, 50_000).astype(np.float32)
    assert np.array_equal(oracle.map_f32("tanh", -x).view(np.uint32), (-oracle.map_f32("tanh", x)).view(np.uint32))
    assert oracle.tanh_s(0.0) == 0.0
    assert oracle.tanh_s(9.5) == 1.0 and oracle.tanh_s(-9.5) == -1.0
    assert oracle.tanh_s(9.0) < 1.0 + 1e-12 and oracle.tanh_s(100.0) == 1.0
    # monotone where it matters for a policy: larger pre-activation never gives a smaller output
    xs = np.sort(rng.uniform(-4, 4, 20_000).astype(np.float32))
    assert np.all(np.diff(oracle.map_f32("tanh", xs).astype(np.float64)) >= -2.5e-7)
