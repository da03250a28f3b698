"""Pins for the oracle's MLP policy and categorical sampling."""
import numpy as np

import oracle
from paper_2207_07736_b200 import inputs


def unpack(p):
    W1, b1 = p[:256].reshape(64, 4), p[256:320]
    W2, b2 = p[320:4416].reshape(64, 64), p[4416:4480]
    W3, b3 = p[4480:4608].reshape(2, 64), p[4608:4610]
    return W1, b1, W2, b2, W3, b3


def logits64(p, obs):
    W1, b1, W2, b2, W3, b3 = [a.astype(np.float64) for a in unpack(p)]
    h1 = np.tanh(W1 @ np.asarray(obs, np.float64) + b1)
    h2 = np.tanh(W2 @ h1 + b2)
    return W3 @ h2 + b3


def test_logits_against_float64_matmul():
    rng = np.random.default_rng(0)
    for seed, bias_std in ((1, 0.0), (2, 0.5)):
        p = inputs.mlp_params(seed, bias_std)
        for _ in range(300):
            obs = (rng.uniform(-1, 1, 4) * np.array([2.4, 3.0, 0.21, 3.0])).astype(np.float32)
            got = oracle.mlp_logits(p, obs).astype(np.float64)
            assert np.abs(got - logits64(p, obs)).max() < 1e-5


def test_one_hot_weights_give_hand_computable_logits():
    p = np.zeros(inputs.MLP_PARAM_COUNT, np.float32)
    W1, b1, W2, b2, W3, b3 = unpack(p)           # views into p
    W1[5, 2] = 1.0        # h1[5] = tanh(obs[2])
    W2[9, 5] = 2.0        # h2[9] = tanh(2 h1[5])
    W3[1, 9] = 3.0        # logit1 = 3 h2[9] + b3[1]
    b3[:] = (0.25, -0.5)
    b1[7] = 0.3           # h1[7] = tanh(0.3), feeds nothing
    obs = np.array([9.0, -9.0, 0.4, 9.0], np.float32)
    got = oracle.mlp_logits(p, obs)
    assert got[0] == np.float32(0.25)
    assert abs(float(got[1]) - (3 * np.tanh(2 * np.tanh(0.4)) - 0.5)) < 2e-6
    # transposed weight indexing would read W1[2,5] / W2[5,9] / W3[.., wrong row] = 0
    W3[1, 9] = 0.0
    W3[0, 9] = 3.0
    got = oracle.mlp_logits(p, obs)
    assert got[1] == np.float32(-0.5) and abs(float(got[0]) - (3 * np.tanh(2 * np.tanh(0.4)) + 0.25)) < 2e-6


def test_sampling_rule():
    # equal logits: action 0 iff u < 1/2 iff the top bit of the word is 0
    for w, want in [(0, 0), (0x7FFFFFFF, 0), (0x80000000, 1), (0xFFFFFFFF, 1)]:
        assert oracle.sample_action([0.0, 0.0], w) == want
        assert oracle.sample_action([3.5, 3.5], w) == want
    # p0 = 0.75: threshold at u = 0.75
    l = [float(np.log(3.0)), 0.0]
    assert oracle.sample_action(l, int(0.74 * 2 ** 32)) == 0
    assert oracle.sample_action(l, int(0.76 * 2 ** 32)) == 1
    # a dominant logit always wins
    assert oracle.sample_action([50.0, -50.0], 0xFFFFFFFF) == 0
    assert oracle.sample_action([-200.0, 0.0], 0x100) == 1          # smallest non-zero u already exceeds exp(-87)
    assert oracle.sample_action([-200.0, 0.0], 0) == 0              # u = 0 always picks the first action


def test_sampling_frequencies_match_softmax():
    rng = np.random.default_rng(1)
    words = rng.integers(0, 2 ** 32, 20000, dtype=np.uint64)
    for l in ([0.3, -0.4], [-1.0, 1.5], [2.0, 2.1]):
        p0 = np.exp(l[0]) / (np.exp(l[0]) + np.exp(l[1]))
        a = np.array([oracle.sample_action(l, int(w)) for w in words])
        assert abs((a == 0).mean() - p0) < 4 * np.sqrt(p0 * (1 - p0) / words.size)


def test_zero_parameters_reproduce_the_random_policy_bit_for_bit():
    z = np.zeros(inputs.MLP_PARAM_COUNT, np.float32)
    a = oracle.OracleSim(oracle.CARTPOLE, 128, seed=9)
    b = oracle.OracleSim(oracle.CARTPOLE, 128, seed=9)
    ra, rb = a.rollout(150), b.rollout(150, policy_params=z)
    for k in ("obs", "act", "rew", "done"):
        assert np.array_equal(ra[k], rb[k])


def test_policy_changes_the_action_distribution():
    p = inputs.mlp_params(1)
    sim = oracle.OracleSim(oracle.CARTPOLE, 256, seed=0)
    out = sim.rollout(64, policy_params=p)
    # empirical action frequency vs the mean softmax probability of the recorded observations
    p0 = []
    for t in range(0, 64, 8):
        for e in range(0, 256, 8):
            l = logits64(p, out["obs"][t, e])
            p0.append(1 / (1 + np.exp(l[1] - l[0])))
    freq0 = (out["act"][::8, ::8] == 0).mean()
    assert abs(freq0 - np.mean(p0)) < 0.08
