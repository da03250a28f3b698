"""Pins for the oracle's synthetic S-float simulator."""
import math

import numpy as np

import oracle


def test_zero_state_and_constant_state():
    for S in (4, 64, 512):
        out, done = oracle.synth_step(np.zeros(S, np.float32), 1)
        assert done == 0 and np.all(out == np.float32(0.001))
        out, _ = oracle.synth_step(np.zeros(S, np.float32), 0)
        assert np.all(out == -np.float32(0.001))
        c = np.float32(0.37)
        out, _ = oracle.synth_step(np.full(S, c, np.float32), 1)
        want = float(c) + 0.01 * math.sin(2 * float(c)) + 0.001
        assert np.all(out == out[0]) and abs(float(out[0]) - want) < 2e-7


def test_small_case_against_double_and_jacobi_order():
    rng = np.random.default_rng(0)
    for S in (4, 8, 64):
        x = rng.uniform(-1.5, 1.5, S).astype(np.float32)
        for act in (0, 1):
            out, _ = oracle.synth_step(x, act)
            x64 = x.astype(np.float64)
            want = x64 + 0.01 * np.sin(x64 + np.roll(x64, -1)) + 0.001 * (2 * act - 1)   # all pre-step values
            assert np.abs(out.astype(np.float64) - want).max() < 3e-7
    # a Gauss-Seidel sweep (using already-updated neighbours) would differ by ~1e-5 here
    x = np.array([1.0, -1.0, 0.5, -0.5], np.float32)
    out, _ = oracle.synth_step(x, 1)
    gs_last = 0.01 * math.sin(-0.5 + float(out[0])) - 0.01 * math.sin(-0.5 + 1.0)
    assert abs(gs_last) > 5e-6
    assert abs(float(out[3]) - (-0.5 + 0.01 * math.sin(0.5) + 0.001)) < 2e-7


def test_rotation_equivariance_bitwise():
    rng = np.random.default_rng(1)
    x = rng.uniform(-1, 1, 64).astype(np.float32)
    base, _ = oracle.synth_step(x, 1)
    for shift in (1, 5, 32):
        rolled, _ = oracle.synth_step(np.roll(x, shift), 1)
        assert np.array_equal(rolled.view(np.uint32), np.roll(base, shift).view(np.uint32))


def test_pairwise_reduction_order():
    t = np.float32(2.0 ** -24)
    # adjacent pairs first: (t+t) + (1+0) = 1 + 2^-23 exactly; a strided or sequential order gives 1
    assert oracle.pairwise_sum([t, t, 1.0, 0.0]) == np.float32(1.0 + 2.0 ** -23)
    assert oracle.pairwise_sum([1.0, t, t, 0.0]) == np.float32(1.0)          # (1+t) rounds to 1, (t+0) is lost
    # depth 3: blocks of four are reduced before they meet
    assert oracle.pairwise_sum([t, t, t, t, 1.0, 0.0, 0.0, 0.0]) == np.float32(1.0 + 2.0 ** -22)
    assert oracle.pairwise_sum([t, 1.0, t, 0, t, 0, t, 0]) == np.float32(1.0 + 2.0 ** -23)
    rng = np.random.default_rng(2)
    q = rng.uniform(0, 9, 4096).astype(np.float32)
    assert abs(float(oracle.pairwise_sum(q)) - q.astype(np.float64).sum()) < 4096 * 9 * 2.0 ** -24 * 12


def test_done_threshold_is_mean_square_above_four():
    for S in (4, 64):
        for v, want in ((2.1, 1), (1.9, 0), (-2.1, 1)):
            out, done = oracle.synth_step(np.full(S, v, np.float32), 1)
            assert done == want
        # exactly 4.0 is not done (strict >): constant state whose update lands on +-2 is hard to hit,
        # so check the rule from the outputs themselves
        x = np.full(S, 2.0, np.float32)
        out, done = oracle.synth_step(x, 0)
        assert done == int(np.mean(out.astype(np.float64) ** 2) > 4.0)


def test_done_and_reset_in_rollout():
    sim = oracle.OracleSim(oracle.SYNTH, 8, state_dim=64, seed=1)
    sim.state[:] = 2.1
    out = sim.rollout(3)
    assert np.all(out["done"][0] == 1) and np.all(out["rew"] == 1.0)
    assert np.all(sim.reset_count == 1)
    for e in range(8):
        assert np.array_equal(out["obs"][1, e], oracle.draw_state(oracle.SYNTH, 64, 1, e, 1))
    assert np.all(out["done"][1:] == 0) and np.all(np.abs(out["obs"][1]) <= 1.0) and np.all(np.abs(out["obs"][2]) <= 1.012)
