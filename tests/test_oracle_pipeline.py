"""Pins for the oracle's per-step sequencing and bookkeeping (properties that hold for any run)."""
import numpy as np
import pytest

import oracle
from paper_2207_07736_b200 import inputs

KINDS = [(oracle.CARTPOLE, 4, 300), (oracle.ACROBOT, 4, 600), (oracle.SYNTH, 8, 40)]


@pytest.mark.parametrize("kind,S,T", KINDS)
def test_split_rollout_invariance(kind, S, T):
    a = oracle.OracleSim(kind, 32, S, seed=4)
    b = oracle.OracleSim(kind, 32, S, seed=4)
    ra = a.rollout(T)
    r1, r2 = b.rollout(T // 3), b.rollout(T - T // 3)
    for k in ("obs", "act", "rew", "done"):
        assert np.array_equal(ra[k], np.concatenate([r1[k], r2[k]]))
    assert np.array_equal(a.state, b.state) and np.array_equal(a.ep_len, b.ep_len) and np.array_equal(a.reset_count, b.reset_count)
    assert a.t == b.t == T


@pytest.mark.parametrize("kind,S,T", KINDS)
def test_env_subset_invariance(kind, S, T):
    full = oracle.OracleSim(kind, 64, S, seed=11)
    ids = np.array([3, 17, 40, 63], dtype=np.uint32)
    sub = oracle.OracleSim(kind, state_dim=S, seed=11, env_ids=ids)
    rf, rs = full.rollout(T), sub.rollout(T)
    for k in ("obs", "act", "rew", "done"):
        assert np.array_equal(rf[k][:, ids], rs[k])


def test_bookkeeping_identities():
    for kind, S, T in KINDS:
        sim = oracle.OracleSim(kind, 48, S, seed=2)
        if kind == oracle.SYNTH:
            sim.state[::2] = 2.05           # force some terminations
        out = sim.rollout(T, want=("obs", "act", "rew", "done", "next_obs"))
        done = out["done"].astype(bool)
        assert np.array_equal(sim.reset_count, done.sum(0).astype(np.uint32))
        for e in range(sim.n):
            idx = np.flatnonzero(done[:, e])
            last = idx[-1] if idx.size else -1
            assert sim.ep_len[e] == T - 1 - last               # steps since the last reset
            # the observation after a reset is draw #(number of resets so far)
            for r, t in enumerate(idx, start=1):
                assert np.array_equal(out["next_obs"][t, e], oracle.draw_state(kind, S, 2, e, r))
        # obs[t+1] is the post-step, post-reset state of step t; the final one is the handle's state
        assert np.array_equal(out["obs"][1:], out["next_obs"][:-1])
        assert np.array_equal(out["next_obs"][-1], sim.state)
        # obs[0] is draw #0 unless overwritten
        if kind != oracle.SYNTH:
            for e in range(sim.n):
                assert np.array_equal(out["obs"][0, e], oracle.draw_state(kind, S, 2, e, 0))


def test_given_actions_path_matches_policy_path():
    for kind, S, T in KINDS:
        a = oracle.OracleSim(kind, 16, S, seed=6)
        ra = a.rollout(T)
        b = oracle.OracleSim(kind, 16, S, seed=6)
        rb = b.rollout(T, actions=ra["act"])
        for k in ("obs", "act", "rew", "done"):
            assert np.array_equal(ra[k], rb[k])
        c = oracle.OracleSim(kind, 16, S, seed=6)
        for t in range(5):
            nxt, rew, done = c.step(ra["act"][t])
            assert np.array_equal(nxt, ra["obs"][t + 1]) and np.array_equal(done, ra["done"][t]) and np.array_equal(rew, ra["rew"][t])


def test_seed_selects_the_stream():
    a = oracle.OracleSim(oracle.CARTPOLE, 8, seed=0).rollout(20)
    b = oracle.OracleSim(oracle.CARTPOLE, 8, seed=1).rollout(20)
    c = oracle.OracleSim(oracle.CARTPOLE, 8, seed=1 << 32).rollout(20)
    assert not np.array_equal(a["obs"], b["obs"]) and not np.array_equal(a["obs"], c["obs"]) and not np.array_equal(b["act"], c["act"])


def test_workload_table_shapes():
    w = inputs.WORKLOADS
    assert w["cfg2"].n_envs == 65536 and w["cfg2"].T == 1000 and w["cfg2"].k_sweep == (1, 10, 100, 1000)
    for S in (4, 64, 512, 4096):
        c = w["cfg5_S%d" % S]
        assert c.n_envs * S * 4 == 4 << 30 and not c.trajectory
    assert inputs.mlp_params(1).shape == (4610,) and np.all(inputs.mlp_params(1)[256:320] == 0)


def test_compute_factor_is_iterated_dynamics_with_the_action_held():
    """Compute factor C (the paper's simulator-complexity knob): one recorded step = C dynamics
    iterations under one action.  Where no episode ends, that equals C plain steps with the action repeated."""
    for kind, S, T, C in [(oracle.CARTPOLE, 4, 3, 2), (oracle.ACROBOT, 4, 30, 3), (oracle.SYNTH, 16, 12, 4)]:
        n = 24
        fat = oracle.OracleSim(kind, n, S, seed=8, compute_factor=C)
        rf = fat.rollout(T)
        assert not rf["done"].any()
        plain = oracle.OracleSim(kind, n, S, seed=8)
        rp = plain.rollout(T * C, actions=np.repeat(rf["act"], C, axis=0))
        assert not rp["done"].any()
        assert np.array_equal(rf["obs"], rp["obs"][::C])
        assert np.array_equal(fat.state, plain.state)
        assert np.all(fat.ep_len == T) and np.all(plain.ep_len == T * C)      # ep_len counts recorded steps
        assert fat.t == T
    # C = 1 is the plain simulator
    a = oracle.OracleSim(oracle.CARTPOLE, 16, seed=3, compute_factor=1).rollout(60)
    b = oracle.OracleSim(oracle.CARTPOLE, 16, seed=3).rollout(60)
    assert all(np.array_equal(a[k], b[k]) for k in ("obs", "act", "rew", "done"))
    # the done test looks at the state after the last iteration; episodes get shorter in recorded steps
    fat = oracle.OracleSim(oracle.CARTPOLE, 256, seed=1, compute_factor=4)
    out = fat.rollout(100)
    first = np.array([np.flatnonzero(out["done"][:, e])[0] for e in range(256)])
    assert 1 <= first.min() and first.mean() < 8
    assert np.array_equal(fat.reset_count, out["done"].sum(0).astype(np.uint32))


def test_episode_returns():
    sim = oracle.OracleSim(oracle.CARTPOLE, 40, seed=3)
    out = sim.rollout(120)
    ret, carry = oracle.episode_returns(out["rew"], out["done"])
    done = out["done"].astype(bool)
    for e in range(40):
        steps = 0
        for t in range(120):
            steps += 1
            assert ret[t, e] == steps              # CartPole pays 1 per step: the return is the step count of the episode
            if done[t, e]:
                steps = 0
        assert carry[e] == steps == sim.ep_len[e]
    # split in two calls with the carry
    r1, c1 = oracle.episode_returns(out["rew"][:50], out["done"][:50])
    r2, c2 = oracle.episode_returns(out["rew"][50:], out["done"][50:], c1)
    assert np.array_equal(np.concatenate([r1, r2]), ret) and np.array_equal(c2, carry)
    # Acrobot: -1 per step, 0 on the goal step
    ac = oracle.OracleSim(oracle.ACROBOT, 16, seed=1)
    o = ac.rollout(600)
    r, _ = oracle.episode_returns(o["rew"], o["done"])
    assert r[498, 0] == -499.0 and r.min() >= -500.0
