"""Pins for the oracle's Acrobot: independent mass-matrix solve, closed forms at rest, energy
conservation, RK4 against a tight adaptive integrator, wrap / clip / goal / time limit."""
import math

import numpy as np
from scipy.integrate import solve_ivp

import oracle

G = 9.8


def dsdt_linear_solve(y, tau):
    """Two-link pendulum (masses 1, lengths 1, centres 0.5, inertias 1) as M(q) qdd = tau - C - G."""
    th1, th2, w1, w2 = [float(v) for v in y]
    c2, s2 = math.cos(th2), math.sin(th2)
    M = np.array([[0.25 + (1 + 0.25 + c2) + 2.0, 0.25 + 0.5 * c2 + 1.0], [0.25 + 0.5 * c2 + 1.0, 1.25]])
    h = 0.5 * s2
    Cv = np.array([-h * w2 * w2 - 2 * h * w1 * w2, h * w1 * w1])
    Gv = np.array([1.5 * G * math.sin(th1) + 0.5 * G * math.sin(th1 + th2), 0.5 * G * math.sin(th1 + th2)])
    qdd = np.linalg.solve(M, np.array([0.0, tau]) - Cv - Gv)
    return np.array([w1, w2, qdd[0], qdd[1]])


def energy(y):
    th1, th2, w1, w2 = [float(v) for v in y]
    d1 = 3.5 + math.cos(th2)
    d2 = 1.25 + 0.5 * math.cos(th2)
    return 0.5 * d1 * w1 * w1 + d2 * w1 * w2 + 0.625 * w2 * w2 - 14.7 * math.cos(th1) - 4.9 * math.cos(th1 + th2)


def test_rest_state_closed_form_and_fixed_point():
    f = oracle.acrobot_dsdt([0, 0, 0, 0], 1.0)
    dd2 = 1.0 / (1.25 - 1.75 ** 2 / 4.5)
    dd1 = -1.75 * dd2 / 4.5
    assert f[0] == 0 and f[1] == 0 and abs(f[3] - dd2) < 3e-7 and abs(f[2] - dd1) < 3e-7
    assert np.all(oracle.acrobot_dsdt([0, 0, 0, 0], 0.0) == 0)
    nxt, goal = oracle.acrobot_step([0, 0, 0, 0], 1)                  # action 1 = zero torque
    assert goal == 0 and np.array_equal(nxt.view(np.uint32), np.zeros(4, dtype=np.uint32))


def test_derivative_matches_independent_solve():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        y = (rng.uniform(-1, 1, 4) * np.array([math.pi, math.pi, 6, 12])).astype(np.float32)
        a = float(rng.integers(-1, 2))
        f = oracle.acrobot_dsdt(y, a).astype(np.float64)
        ref = dsdt_linear_solve(y, a)
        assert np.all(np.abs(f - ref) <= 3e-6 * np.maximum(1.0, np.abs(ref)) + 3e-5 * (np.abs(ref) > 50))


def test_action_encoding_and_clamp():
    y = [0.3, -0.2, 0.1, 0.05]
    outs = [oracle.acrobot_step(y, a)[0] for a in (0, 1, 2)]
    # torque -1, 0, +1: the response of omega2 is monotone in the torque
    assert outs[0][3] < outs[1][3] < outs[2][3]
    assert np.array_equal(oracle.acrobot_step(y, -5)[0], outs[0]) and np.array_equal(oracle.acrobot_step(y, 9)[0], outs[2])


def test_rk4_step_against_adaptive_integrator():
    rng = np.random.default_rng(1)
    worst = 0.0
    for _ in range(200):
        y = rng.uniform(-0.1, 0.1, 4).astype(np.float32)
        act = int(rng.integers(0, 3))
        nxt, _ = oracle.acrobot_step(y, act)
        sol = solve_ivp(lambda t, s: dsdt_linear_solve(s, act - 1.0), (0, 0.2), y.astype(np.float64), rtol=1e-11, atol=1e-13)
        worst = max(worst, np.abs(nxt.astype(np.float64) - sol.y[:, -1]).max())
    # one classical RK4 step of 0.2 s from the reset distribution has a local error of ~4e-4
    # against the exact flow; wrong stage weights, stage times or step size miss by 4e-3 or more
    assert worst < 1e-3


def test_rk4_step_against_butcher_tableau_in_double():
    """The classical fourth-order tableau applied, in float64, to the independent derivative."""
    A = np.array([[0, 0, 0, 0], [0.5, 0, 0, 0], [0, 0.5, 0, 0], [0, 0, 1.0, 0]])
    b = np.array([1, 2, 2, 1]) / 6.0
    rng = np.random.default_rng(4)
    for _ in range(300):
        y = (rng.uniform(-1, 1, 4) * np.array([1.0, 1.0, 2.0, 2.0])).astype(np.float32)
        act = int(rng.integers(0, 3))
        y64 = y.astype(np.float64)
        ks = []
        for i in range(4):
            ks.append(dsdt_linear_solve(y64 + 0.2 * sum(A[i, j] * ks[j] for j in range(i)), act - 1.0))
        want = y64 + 0.2 * sum(b[i] * ks[i] for i in range(4))
        nxt, _ = oracle.acrobot_step(y, act)
        assert np.abs(nxt.astype(np.float64) - want).max() < 5e-6


def test_energy_conservation_zero_torque():
    rng = np.random.default_rng(2)
    for _ in range(20):
        y = rng.uniform(-0.1, 0.1, 4).astype(np.float32)
        e0 = energy(y)
        worst = 0.0
        for _ in range(500):
            y, _ = oracle.acrobot_step(y, 1)
            worst = max(worst, abs(energy(y) - e0))
        assert worst <= 1e-3 * abs(e0)


def test_wrap_clip_goal():
    PI = float(np.float32(math.pi))
    # theta1 just below pi with positive omega1 crosses and wraps to near -pi
    nxt, _ = oracle.acrobot_step([3.1, 0.0, 2.0, 0.0], 1)
    assert -PI <= nxt[0] <= PI and nxt[0] < 0
    nxt, _ = oracle.acrobot_step([0.0, -3.1, 0.0, -3.0], 1)
    assert -PI <= nxt[1] <= PI and nxt[1] > 0
    # velocity clips: 4 pi and 9 pi
    nxt, _ = oracle.acrobot_step([1.5, 0.0, 12.56, 28.2], 2)
    assert abs(nxt[2]) <= np.float32(4 * math.pi) and abs(nxt[3]) <= np.float32(9 * math.pi)
    nxt, _ = oracle.acrobot_step([0.0, 0.0, 40.0, -60.0], 1)
    assert nxt[2] == np.float32(4 * math.pi) and nxt[3] == -np.float32(9 * math.pi)
    # goal: tip above one link length; hanging down is not the goal, pointing up is
    _, goal = oracle.acrobot_step([math.pi, 0.0, 0.0, 0.0], 1)
    assert goal == 1
    _, goal = oracle.acrobot_step([0.2, 0.1, 0.0, 0.0], 1)
    assert goal == 0


def test_time_limit_and_reward_through_rollout():
    sim = oracle.OracleSim(oracle.ACROBOT, 64, seed=3)
    out = sim.rollout(1001)
    done = out["done"].astype(bool)
    rew = out["rew"]
    assert set(np.unique(out["act"])) == {0, 1, 2}
    for e in range(sim.n):
        idx = np.flatnonzero(done[:, e])
        lengths = np.diff(np.concatenate([[-1], idx]))
        assert lengths.max() <= 500                     # the 500th step of an episode is its last
        for t, ln in zip(idx, lengths):
            if ln == 500 and rew[t, e] == -1.0:
                continue                                # ended by the time limit
            assert rew[t, e] == 0.0                     # ended at the goal
        live = ~done[:, e]
        assert np.all(rew[live, e] == -1.0)
    # most random-torque episodes run into the limit
    first_done = np.array([np.flatnonzero(done[:, e])[0] for e in range(sim.n)])
    assert np.mean(first_done == 499) > 0.9


def test_six_value_observation():
    rng = np.random.default_rng(9)
    for _ in range(200):
        s = (rng.uniform(-1, 1, 4) * np.array([math.pi, math.pi, 12, 28])).astype(np.float32)
        o = oracle.acrobot_observation(s).astype(np.float64)
        want = [math.cos(float(s[0])), math.sin(float(s[0])), math.cos(float(s[1])), math.sin(float(s[1])), float(s[2]), float(s[3])]
        assert np.abs(o - want).max() < 3e-7
    assert np.array_equal(oracle.acrobot_observation([0, 0, 1.5, -2.5]), np.array([1, 0, 1, 0, 1.5, -2.5], np.float32))
