"""Tensor-mode MLP policy (tolerance mode): the layers run as FP16 tensor-core contractions with fp32
accumulation and tanh is the packed half-precision hardware approximation, so actions are not bit-reproducible.  What is unique is compared
exactly, the rest is checked for validity:
  * logits against the oracle's exact logits, within the bound derived from the weights;
  * a rollout must be an exact CartPole trajectory under the actions it records (oracle stepping with those
    actions reproduces every observation, reward, done flag, the final state and the counters bit for bit);
  * every recorded action must be the oracle's action for the recorded observation, except where the
    uniform draw lies within the probability error bound of the decision threshold.
"""
import numpy as np
import pytest

import oracle
from paper_2207_07736_b200 import binding, inputs
from gpu_common import assert_same_bits, to_np, torch_cuda
from tensor_bound import logit_error_bound

pytestmark = pytest.mark.gpu

def exact_logits(p, obs):
    return np.stack([oracle.mlp_logits(p, o) for o in obs])


@pytest.mark.parametrize("seed,bias", [(1, 0.0), (7, 0.3)])
def test_tensor_logits_within_the_derived_bound(seed, bias):
    torch = torch_cuda()
    rng = np.random.default_rng(seed)
    obs = (rng.uniform(-1, 1, (1000, 4)) * np.array([2.4, 3, 0.21, 3])).astype(np.float32)     # 7 full CTAs and a tail
    p = inputs.mlp_params(seed, bias)
    sim = binding.Sim(oracle.CARTPOLE, 8, policy_mode=binding.SIM_POLICY_TENSOR)
    got = to_np(sim.policy_logits(torch.from_numpy(obs).cuda(), torch.from_numpy(p).cuda())).astype(np.float64)
    assert sim.device_status() == 0
    want = exact_logits(p, obs).astype(np.float64)
    err, bound = np.abs(got - want), logit_error_bound(p, obs)
    assert (err <= bound).all(), (err.max(), bound[np.unravel_index(err.argmax(), err.shape)])
    assert np.sqrt((err ** 2).mean()) <= 2e-3          # typical error is far below the worst case
    assert err.max() > 0                               # and it is the tolerance path that ran
    # exact mode through the same entry point is still bit-identical
    exact = binding.Sim(oracle.CARTPOLE, 8)
    assert_same_bits(to_np(exact.policy_logits(torch.from_numpy(obs).cuda(), torch.from_numpy(p).cuda())), exact_logits(p, obs), "exact logits")


def check_tensor_rollout(sim, out, p, seed, env_ids, T, what, cols=None):
    """Validity of a tensor-mode rollout on the envs with global indices `env_ids`, found in the output
    columns `cols` (default: the same numbers)."""
    sel = np.asarray(env_ids if cols is None else cols, dtype=np.int64)
    g = {k: to_np(out[k])[:, sel] for k in ("obs", "act", "rew", "done")}
    assert set(np.unique(g["act"]).tolist()) <= {0, 1}
    # 1. exact physics under the recorded actions
    orc = oracle.OracleSim(oracle.CARTPOLE, seed=seed, env_ids=env_ids)
    ref = orc.rollout(T, actions=g["act"])
    for k in ("obs", "rew", "done"):
        assert_same_bits(g[k], ref[k], "%s %s under the recorded actions" % (what, k))
    assert_same_bits(to_np(sim.state())[sel], orc.state, what + " final state")
    ep, rc, t = sim.counters()
    assert_same_bits(to_np(ep)[sel].astype(np.uint32), orc.ep_len, what + " ep_len")
    assert_same_bits(to_np(rc)[sel].astype(np.uint32), orc.reset_count, what + " reset_count")
    assert t == T
    # 2. recorded actions against the oracle's decision on the recorded observations
    flat_obs = g["obs"].reshape(-1, 4)
    lg = exact_logits(p, flat_obs).astype(np.float64)
    bound = logit_error_bound(p, flat_obs)
    p0 = 1.0 / (1.0 + np.exp(lg[:, 1] - lg[:, 0]))
    delta = 0.25 * (bound[:, 0] + bound[:, 1]) + 1e-6          # |d p0| <= |d (l0 - l1)| / 4
    differ = 0
    for idx in range(flat_obs.shape[0]):
        t_, c = divmod(idx, len(env_ids))
        w = oracle.action_word(seed, int(env_ids[c]), t_)
        want = oracle.sample_action(lg[idx].astype(np.float32), w)
        if int(g["act"][t_, c]) != want:
            differ += 1
            assert abs(oracle.uniform01(w) - p0[idx]) <= delta[idx], (what, t_, c, oracle.uniform01(w), p0[idx], delta[idx])
    assert differ <= 0.01 * flat_obs.shape[0], (what, differ)
    return differ


@pytest.mark.parametrize("K,bias", [(1, 0.0), (7, 0.5), (64, 0.0)])
def test_tensor_rollout_is_a_valid_trajectory(K, bias):
    torch = torch_cuda()
    n, T, seed = 300, 64, 4                     # two full CTAs and a ragged one
    p = inputs.mlp_params(1, bias)
    sim = binding.Sim(oracle.CARTPOLE, n, 4, seed, policy_mode=binding.SIM_POLICY_TENSOR)
    out = sim.rollout(T, K, torch.from_numpy(p).cuda())
    torch.cuda.synchronize()
    assert sim.device_status() == 0
    check_tensor_rollout(sim, out, p, seed, np.arange(n, dtype=np.uint32), T, "tensor K%d" % K)
    frac0 = float((out["act"] == 0).float().mean())
    assert 0.05 < frac0 < 0.95
    assert int(out["done"].sum()) > 0           # resets happened inside the window


def test_tensor_rollout_is_repeatable_and_close_to_exact_mode():
    torch = torch_cuda()
    n, T, seed = 1000, 40, 11
    p = torch.from_numpy(inputs.mlp_params(3, 0.2)).cuda()
    a = binding.Sim(oracle.CARTPOLE, n, 4, seed, policy_mode=binding.SIM_POLICY_TENSOR).rollout(T, 40, p)
    b = binding.Sim(oracle.CARTPOLE, n, 4, seed, policy_mode=binding.SIM_POLICY_TENSOR).rollout(T, 8, p)
    for k in ("obs", "act", "rew", "done"):
        assert torch.equal(a[k], b[k]), k       # same device, same inputs: same bits, whatever K
    e = binding.Sim(oracle.CARTPOLE, n, 4, seed).rollout(T, 40, p)
    assert torch.equal(a["obs"][0], e["obs"][0])
    same_first = float((a["act"][0] == e["act"][0]).float().mean())
    assert same_first > 0.99                    # first step: same observations, nearly always the same action


def test_tensor_mode_with_offset_compute_factor_and_mode_switch():
    torch = torch_cuda()
    n, T, seed, off = 200, 24, 5, 1000
    p = inputs.mlp_params(2, 0.1)
    dp = torch.from_numpy(p).cuda()
    sim = binding.Sim(oracle.CARTPOLE, n, 4, seed, env_offset=off, policy_mode=binding.SIM_POLICY_TENSOR)
    out = sim.rollout(T, 5, dp)
    torch.cuda.synchronize()
    # env ids are global: oracle envs off..off+n-1 are columns 0..n-1 of the outputs
    ids = np.arange(off, off + n, dtype=np.uint32)
    check_tensor_rollout(sim, out, p, seed, ids, T, "offset", cols=np.arange(n))
    orc = oracle.OracleSim(oracle.CARTPOLE, seed=seed, env_ids=ids)
    orc.rollout(T, actions=to_np(out["act"]))
    # back to exact mode on the same handle: bit-exact against the oracle from the current state
    binding.sim_set_policy_mode(sim.h, binding.SIM_POLICY_EXACT)
    out2 = sim.rollout(10, 10, dp)
    ref2 = orc.rollout(10, policy_params=p)
    for k in ("obs", "act", "rew", "done"):
        assert_same_bits(to_np(out2[k]), ref2[k], "exact after tensor " + k)
    assert sim.device_status() == 0


def test_tensor_mode_argument_errors():
    torch_cuda()
    acro = binding.Sim(oracle.ACROBOT, 16)
    assert binding.lib().sim_set_policy_mode(acro.h, binding.SIM_POLICY_TENSOR) == binding.SIM_EINVAL
    cp = binding.Sim(oracle.CARTPOLE, 16)
    assert binding.lib().sim_set_policy_mode(cp.h, 3) == binding.SIM_EINVAL
    assert binding.lib().sim_set_policy_mode(None, 0) == binding.SIM_EINVAL
    assert cp.device_status() == 0              # never selected: no status word, reads as clean


def test_cfg3_full_size_in_tensor_mode():
    """The largest CartPole + MLP workload in the launch configuration the bench times (one launch of 500
    steps over 2^20 envs): a sample of envs (first, last, random) is checked for validity by the oracle."""
    torch = torch_cuda()
    w = inputs.WORKLOADS["cfg3"]
    ids = inputs.sample_env_ids(23, w.n_envs, 12)
    p = inputs.mlp_params(w.mlp_seed)
    sim = binding.Sim(w.env_kind, w.n_envs, w.state_dim, w.seed, policy_mode=binding.SIM_POLICY_TENSOR)
    out = sim.rollout(w.T, max(w.k_sweep), torch.from_numpy(p).cuda())
    torch.cuda.synchronize()
    assert sim.device_status() == 0
    sel = torch.from_numpy(ids.astype(np.int64)).cuda()
    sample = {k: out[k][:, sel] for k in ("obs", "act", "rew", "done")}

    class View:                                  # the handle's state and counters restricted to the sample
        def state(self_):
            return sim.state()[sel]

        def counters(self_):
            ep, rc, t = sim.counters()
            return ep[sel], rc[sel], t

    check_tensor_rollout(View(), sample, p, w.seed, ids, w.T, "cfg3 tensor", cols=np.arange(len(ids)))
    # properties that hold at any size
    ep, rc, t = sim.counters()
    assert torch.equal(out["done"].sum(0, dtype=torch.int32), rc)
    assert float(out["obs"][:, :, 0].abs().max()) <= float(np.float32(2.4)) and float(out["obs"][:, :, 2].abs().max()) <= 0.2095
    # the tolerance-mode policy behaves like the exact one: action frequencies agree closely
    exact = binding.Sim(w.env_kind, w.n_envs, w.state_dim, w.seed)
    ref = exact.rollout(20, 20, torch.from_numpy(p).cuda(), want=("act",))
    f_t = float((out["act"][:20] == 0).float().mean()); f_e = float((ref["act"] == 0).float().mean())
    assert abs(f_t - f_e) < 2e-3, (f_t, f_e)


@pytest.mark.parametrize("n", [1, 129, 257])
def test_tensor_rollout_tiny_and_ragged_batches(n):
    """One env (a CTA whose second group only shadows), one env past a tile, one env past a CTA."""
    torch = torch_cuda()
    T, seed = 30, 8
    p = inputs.mlp_params(5, 0.2)
    sim = binding.Sim(oracle.CARTPOLE, n, 4, seed, policy_mode=binding.SIM_POLICY_TENSOR)
    out = sim.rollout(T, 4, torch.from_numpy(p).cuda())           # 8 launches, the last one of 2 steps
    torch.cuda.synchronize()
    assert sim.device_status() == 0 and sim.launches == 1 + 8
    check_tensor_rollout(sim, out, p, seed, np.arange(n, dtype=np.uint32), T, "tiny n%d" % n)


def test_tensor_mode_leaves_buffers_alone_and_handles_null_outputs():
    torch = torch_cuda()
    n, T, seed = 200, 12, 2
    p = torch.from_numpy(inputs.mlp_params(1)).cuda()
    a = binding.Sim(oracle.CARTPOLE, n, 4, seed, policy_mode=binding.SIM_POLICY_TENSOR)
    full = a.rollout(T, T, p)
    b = binding.Sim(oracle.CARTPOLE, n, 4, seed, policy_mode=binding.SIM_POLICY_TENSOR)
    guard = torch.full((T * n + 64,), 7, dtype=torch.uint8, device="cuda")
    binding.sim_rollout(b.h, T, 5, p, None, None, None, guard[32:32 + T * n])       # only the done flags
    torch.cuda.synchronize()
    assert bool((guard[:32] == 7).all()) and bool((guard[32 + T * n:] == 7).all())
    assert torch.equal(guard[32:32 + T * n].view(T, n), full["done"])
    assert torch.equal(a.state(), b.state())


def test_bounded_wait_gives_up_cleanly():
    """The tensor-mode kernels never spin without a limit: with the contractions left out (self-check launch)
    every wait runs out, the status bit is raised, no thread reports success, tensor memory is freed, and the
    context stays usable for an ordinary tensor-mode rollout afterwards."""
    torch = torch_cuda()
    sim = binding.Sim(oracle.CARTPOLE, 300, 4, 4, policy_mode=binding.SIM_POLICY_TENSOR)
    status, completed = binding.sim_selfcheck_tensor_wait(sim.h)
    assert status == binding.SIM_STATUS_TENSOR_WAIT and completed == 0
    assert sim.device_status() == 0                       # the self-check has a status word of its own
    p = inputs.mlp_params(1)
    out = sim.rollout(16, 16, torch.from_numpy(p).cuda())
    torch.cuda.synchronize()
    assert sim.device_status() == 0
    check_tensor_rollout(sim, out, p, 4, np.arange(300, dtype=np.uint32), 16, "after self-check")
