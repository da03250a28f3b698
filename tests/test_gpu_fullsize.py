"""Parity at the full workload sizes, in the launch configuration the bench times: the whole batch
runs on the GPU, a sample of envs (first, last, random) is recomputed one by one by the oracle."""
import numpy as np
import pytest

import oracle
from paper_2207_07736_b200 import binding, inputs
from gpu_common import assert_same_bits, to_np, torch_cuda

pytestmark = pytest.mark.gpu


def sampled_check(name, K, n_sample, want=("obs", "act", "rew", "done")):
    torch = torch_cuda()
    w = inputs.WORKLOADS[name]
    ids = inputs.sample_env_ids(17, w.n_envs, n_sample)
    params = None if w.mlp_seed is None else inputs.mlp_params(w.mlp_seed)
    sim = binding.Sim(w.env_kind, w.n_envs, w.state_dim, w.seed)
    d_params = None if params is None else torch.from_numpy(params).cuda()
    out = sim.rollout(w.T, K, d_params, want=want if w.trajectory else ())
    torch.cuda.synchronize()
    assert sim.launches == 1 + -(-w.T // K)
    orc = oracle.OracleSim(w.env_kind, state_dim=w.state_dim, seed=w.seed, env_ids=ids)
    ref = orc.rollout(w.T, policy_params=params, want=want if w.trajectory else ())
    sel = torch.from_numpy(ids.astype(np.int64)).cuda()
    for k in ("obs", "act", "rew", "done"):
        if out.get(k) is not None:
            assert_same_bits(to_np(out[k][:, sel]), ref[k], "%s K=%d %s" % (name, K, k))
    st = sim.state()[sel]
    ep, rc, t = sim.counters()
    assert_same_bits(to_np(st), orc.state, name + " final state")
    assert_same_bits(to_np(ep[sel]).astype(np.uint32), orc.ep_len, name + " ep_len")
    assert_same_bits(to_np(rc[sel]).astype(np.uint32), orc.reset_count, name + " reset_count")
    # properties that hold at any size
    if out.get("done") is not None:
        assert torch.equal(out["done"].sum(0, dtype=torch.int32), rc)
    return out


@pytest.mark.parametrize("K", [1000, 10])
def test_cfg2_cartpole_full(K):
    out = sampled_check("cfg2", K, 96)
    assert float(out["rew"].min()) == 1.0 and float(out["rew"].max()) == 1.0
    assert float(out["obs"][:, :, 0].abs().max()) <= float(np.float32(2.4)) and float(out["obs"][:, :, 2].abs().max()) <= 0.2095


def test_cfg3_mlp_full():
    sampled_check("cfg3", 500, 24)


def test_cfg4_acrobot_full():
    out = sampled_check("cfg4", 500, 48)
    assert int(out["done"][499].sum()) > 250000          # almost every env meets the 500-step limit together


@pytest.mark.parametrize("S,K,ns", [(4, 256, 4000), (64, 64, 500), (512, 16, 64), (4096, 256, 10), (4096, 1, 10)])
def test_cfg5_synth_full(S, K, ns):
    sampled_check("cfg5_S%d" % S, K, ns)


@pytest.mark.parametrize("kind", [oracle.CARTPOLE, oracle.ACROBOT])
def test_very_large_ragged_batch(kind):
    """Fifty million envs with a ragged tail: 64-bit trajectory indexing and the last partial warp."""
    torch = torch_cuda()
    n, T = 50_000_017, 9
    sim = binding.Sim(kind, n, 4, 7)
    out = sim.rollout(T, 9, want=("obs", "done"))
    torch.cuda.synchronize()
    ids = np.concatenate([inputs.sample_env_ids(1, n, 40), np.arange(n - 70, n, dtype=np.uint32)])
    ids = np.unique(ids)
    orc = oracle.OracleSim(kind, state_dim=4, seed=7, env_ids=ids)
    ref = orc.rollout(T, want=("obs", "done"))
    sel = torch.from_numpy(ids.astype(np.int64)).cuda()
    assert_same_bits(to_np(out["obs"][:, sel]), ref["obs"], "obs")
    assert_same_bits(to_np(out["done"][:, sel]), ref["done"], "done")
    assert_same_bits(to_np(sim.state()[sel]), orc.state, "state")
