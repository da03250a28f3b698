"""Pins for the oracle's CartPole step: closed forms, an independent mass-matrix solve,
symmetry, the energy balance, thresholds and episode statistics."""
import math

import numpy as np

import oracle

G, MC, MP, L, FMAG, TAU = 9.8, 1.0, 0.1, 0.5, 10.0, 0.02


def accel_by_linear_solve(state, act):
    """Lagrangian form of the cart with a uniform pole of half-length L (float64):
         (mc+mp) xdd + mp L cos(th) thdd = F + mp L thd^2 sin(th)
         mp L cos(th) xdd + (4/3) mp L^2 thdd = mp g L sin(th)
    solved as a 2x2 system; nothing here follows the oracle's operation order."""
    x, xd, th, thd = [float(v) for v in state]
    F = FMAG if act else -FMAG
    M = np.array([[MC + MP, MP * L * math.cos(th)], [MP * L * math.cos(th), 4.0 / 3.0 * MP * L * L]])
    rhs = np.array([F + MP * L * thd * thd * math.sin(th), MP * G * L * math.sin(th)])
    xdd, thdd = np.linalg.solve(M, rhs)
    return xdd, thdd


def test_closed_form_at_rest():
    for act, sign in ((1, 1.0), (0, -1.0)):
        temp, thacc, xacc = oracle.cartpole_accel([0, 0, 0, 0], act)
        t = sign * 10.0 / 1.1
        th = -t / (0.5 * (4.0 / 3.0 - 0.1 / 1.1))
        xa = t - 0.05 * th / 1.1
        assert abs(temp - t) < 1e-6 and abs(thacc - th) < 2e-6 and abs(xacc - xa) < 1e-6
        nxt, done = oracle.cartpole_step([0, 0, 0, 0], act)
        assert done == 0
        assert nxt[0] == 0.0 and nxt[2] == 0.0                        # positions use the OLD velocities
        assert abs(nxt[1] - TAU * xa) < 2e-7 and abs(nxt[3] - TAU * th) < 2e-7


def test_accelerations_match_independent_solve():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        s = np.array([rng.uniform(-2.4, 2.4), rng.uniform(-3, 3), rng.uniform(-0.3, 0.3), rng.uniform(-3, 3)], dtype=np.float32)
        act = int(rng.integers(0, 2))
        _, thacc, xacc = oracle.cartpole_accel(s, act)
        xdd, thdd = accel_by_linear_solve(s, act)
        assert abs(float(xacc) - xdd) <= 2e-6 * max(1.0, abs(xdd))
        assert abs(float(thacc) - thdd) <= 2e-6 * max(1.0, abs(thdd))


def test_euler_update_uses_old_velocities_and_tau():
    rng = np.random.default_rng(1)
    for _ in range(500):
        s = rng.uniform(-1, 1, 4).astype(np.float32) * np.array([2, 2, 0.2, 2], dtype=np.float32)
        act = int(rng.integers(0, 2))
        nxt, _ = oracle.cartpole_step(s, act)
        xdd, thdd = accel_by_linear_solve(s, act)
        want = [s[0] + TAU * float(s[1]), s[1] + TAU * xdd, s[2] + TAU * float(s[3]), s[3] + TAU * thdd]
        assert np.allclose(nxt.astype(np.float64), want, rtol=1e-6, atol=2e-7)


def test_mirror_symmetry_is_bitwise():
    rng = np.random.default_rng(2)
    for _ in range(2000):
        s = rng.uniform(-1, 1, 4).astype(np.float32) * np.array([2.4, 3, 0.25, 3], dtype=np.float32)
        act = int(rng.integers(0, 2))
        a, da = oracle.cartpole_step(s, act)
        b, db = oracle.cartpole_step(-s, 1 - act)
        assert np.array_equal(a.view(np.uint32), (-b).view(np.uint32)) and da == db


def test_energy_balance():
    """dE/dt = F * xdot for the exact accelerations (E = kinetic + potential of cart and rod)."""
    rng = np.random.default_rng(3)
    for _ in range(500):
        s = np.array([0.0, rng.uniform(-2, 2), rng.uniform(-0.3, 0.3), rng.uniform(-2, 2)], dtype=np.float32)
        act = int(rng.integers(0, 2))
        _, thacc, xacc = [float(v) for v in oracle.cartpole_accel(s, act)]
        x, xd, th, thd = [float(v) for v in s]
        F = FMAG if act else -FMAG
        # E = 1/2 (mc+mp) xd^2 + mp L xd thd cos th + 2/3 mp L^2 thd^2 + mp g L cos th
        dE = ((MC + MP) * xd * xacc + MP * L * (xacc * thd * math.cos(th) + xd * thacc * math.cos(th) - xd * thd * thd * math.sin(th))
              + 4.0 / 3.0 * MP * L * L * thd * thacc - MP * G * L * math.sin(th) * thd)
        assert abs(dE - F * xd) < 2e-5 * max(1.0, abs(F * xd))


def test_thresholds_strict_and_on_new_state():
    x_th = np.float32(2.4)
    th_th = np.float32(12 * 2 * math.pi / 360)
    up = lambda v: np.nextafter(np.float32(v), np.float32(np.inf))
    # zero velocities: the new position equals the old one exactly
    for x, want in [(x_th, 0), (up(x_th), 1), (-x_th, 0), (-up(x_th), 1)]:
        _, done = oracle.cartpole_step([x, 0, 0, 0], 1)
        assert done == want
    for th, want in [(th_th, 0), (up(th_th), 1), (-th_th, 0), (-up(th_th), 1)]:
        _, done = oracle.cartpole_step([0, 0, th, 0], 0)
        assert done == want
    # the test looks at the NEW state: a state inside the limit that steps across it is done
    nxt, done = oracle.cartpole_step([2.39, 1.0, 0.0, 0.0], 1)
    assert nxt[0] > x_th and done == 1
    # and a state beyond the limit that steps back inside is not
    nxt, done = oracle.cartpole_step([2.41, -1.0, 0.0, 0.0], 1)
    assert nxt[0] < x_th and done == 0
    assert abs(float(th_th) - 0.20943951) < 1e-7


def test_random_policy_episode_statistics():
    sim = oracle.OracleSim(oracle.CARTPOLE, 2048, seed=5)
    out = sim.rollout(400)
    assert np.all(out["rew"] == 1.0)
    assert set(np.unique(out["act"])) == {0, 1}
    done = out["done"].astype(bool)
    lengths = []
    for e in range(sim.n):
        idx = np.flatnonzero(done[:, e])
        lengths += np.diff(np.concatenate([[-1], idx])).tolist()
    lengths = np.array(lengths)
    assert 21.0 < lengths.mean() < 23.5          # random-policy CartPole: about 22 steps per episode
    assert lengths.min() >= 7
    # every recorded observation is a live state
    assert np.all(np.abs(out["obs"][:, :, 0]) <= 2.4) and np.all(np.abs(out["obs"][:, :, 2]) <= 0.2095)
