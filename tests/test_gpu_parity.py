"""GPU-vs-oracle parity through the C ABI, bit for bit (actions, flags, counters, fp32 states),
at sizes the oracle finishes in seconds: several CTAs, a ragged tail, K that does not divide T,
launches that start at every phase of the 4-step action block."""
import numpy as np
import pytest

import oracle
from paper_2207_07736_b200 import binding, inputs
from gpu_common import assert_same_bits, compare_rollout, to_np, torch_cuda

pytestmark = pytest.mark.gpu


def run_pair(kind, n, T, K, S=4, seed=0, params=None, pre=None):
    torch = torch_cuda()
    sim = binding.Sim(kind, n, S, seed)
    orc = oracle.OracleSim(kind, n, S, seed)
    if pre is not None:
        pre(sim, orc, torch)
    d_params = None if params is None else torch.from_numpy(params).cuda()
    out = sim.rollout(T, K, d_params)
    torch.cuda.synchronize()
    ref = orc.rollout(T, policy_params=params)
    compare_rollout(out, sim, ref, orc, what="kind%d n%d T%d K%d S%d" % (kind, n, T, K, S))
    return sim, out


def test_cfg1_cartpole_small_exact():
    w = inputs.WORKLOADS["cfg1"]
    sim, out = run_pair(w.env_kind, w.n_envs, w.T, 1, seed=w.seed)
    assert sim.launches == 1 + w.T                       # one reset kernel + one launch per step
    assert float(out["rew"].min()) == 1.0 and int(out["done"].sum()) > 0


@pytest.mark.parametrize("K", [1, 3, 7, 10, 64, 157, 1000])
def test_cartpole_any_k_ragged(K):
    sim, _ = run_pair(oracle.CARTPOLE, 1000, 157, K, seed=3)
    assert sim.launches == 1 + -(-157 // min(K, 157))


@pytest.mark.parametrize("K", [1, 50, 500, 1100])
def test_acrobot_any_k(K):
    n, T = (64, 120) if K == 1 else (300, 1100)          # 1100 steps cross the 500-step limit twice
    sim, out = run_pair(oracle.ACROBOT, n, T, K, seed=5)
    if T > 500:
        assert int(out["done"][499].sum()) > n // 2


def test_acrobot_wrap_and_clip_states():
    def pre(sim, orc, torch):
        rng = np.random.default_rng(0)
        st = (rng.uniform(-1, 1, (sim.n, 4)) * np.array([3.14, 3.14, 12.5, 28.0])).astype(np.float32)
        orc.state[:] = st
        sim.set_state(torch.from_numpy(st).cuda())
    run_pair(oracle.ACROBOT, 257, 30, 30, seed=1, pre=pre)


@pytest.mark.parametrize("S", [4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096])
def test_synth_all_shapes(S):
    n = 37 if S <= 512 else 5

    def pre(sim, orc, torch):
        st = orc.state.copy()
        st[::3] = 2.02                                   # every third env terminates on the first step
        st[1::7] *= 2.2                                  # some drift over the threshold later
        orc.state[:] = st
        sim.set_state(torch.from_numpy(st).cuda())
    for K in (1, 5, 22):
        sim, out = run_pair(oracle.SYNTH, n, 22, K, S=S, seed=2, pre=pre)
        assert int(out["done"][0].sum()) >= n // 3


def test_synth_larger_batch_spans_many_ctas():
    run_pair(oracle.SYNTH, 3001, 9, 4, S=4, seed=8)
    run_pair(oracle.SYNTH, 1025, 9, 9, S=64, seed=8)
    run_pair(oracle.SYNTH, 70, 6, 3, S=4096, seed=8)


@pytest.mark.parametrize("bias_std", [0.0, 0.5])
@pytest.mark.parametrize("K", [1, 9, 60])
def test_mlp_policy(K, bias_std):
    p = inputs.mlp_params(1, bias_std)
    sim, out = run_pair(oracle.CARTPOLE, 300, 60, K, seed=4, params=p)
    frac0 = float((out["act"] == 0).float().mean())
    assert 0.05 < frac0 < 0.95


def test_mlp_zero_params_equal_random_policy():
    torch = torch_cuda()
    z = torch.zeros(inputs.MLP_PARAM_COUNT, dtype=torch.float32, device="cuda")
    a = binding.Sim(oracle.CARTPOLE, 500, 4, 9)
    b = binding.Sim(oracle.CARTPOLE, 500, 4, 9)
    ra, rb = a.rollout(80, 80), b.rollout(80, 16, z)
    for k in ("obs", "act", "rew", "done"):
        assert torch.equal(ra[k], rb[k])


def test_policy_logits_entry_point():
    torch = torch_cuda()
    rng = np.random.default_rng(0)
    obs = (rng.uniform(-1, 1, (1000, 4)) * np.array([2.4, 3, 0.21, 3])).astype(np.float32)
    sim = binding.Sim(oracle.CARTPOLE, 8)
    for seed, bias in ((1, 0.0), (7, 0.3)):
        p = inputs.mlp_params(seed, bias)
        got = to_np(sim.policy_logits(torch.from_numpy(obs).cuda(), torch.from_numpy(p).cuda()))
        want = np.stack([oracle.mlp_logits(p, o) for o in obs])
        assert np.abs(got - want).max() <= 1e-5          # the stated tolerance
        assert_same_bits(got, want, "logits")            # and in fact identical


@pytest.mark.parametrize("kind,S,nact", [(oracle.CARTPOLE, 4, 2), (oracle.ACROBOT, 4, 3), (oracle.SYNTH, 64, 2), (oracle.SYNTH, 2048, 2)])
def test_step_with_given_actions(kind, S, nact):
    torch = torch_cuda()
    n, T = 203, 40
    sim = binding.Sim(kind, n, S, 6)
    orc = oracle.OracleSim(kind, n, S, 6)
    acts = inputs.forced_actions(1, T, n, nact)
    acts[3, :5] = [-3, 7, 100, -128, 2]                   # out-of-range bytes follow the documented rule
    for t in range(T):
        nxt, rew, done = sim.step(torch.from_numpy(acts[t]).cuda())
        o_nxt, o_rew, o_done = orc.step(acts[t])
        assert_same_bits(to_np(nxt), o_nxt, "next_obs t=%d" % t)
        assert_same_bits(to_np(rew), o_rew, "rew")
        assert_same_bits(to_np(done), o_done, "done")
    ep, rc, tt = sim.counters()
    assert tt == T and np.array_equal(to_np(rc).astype(np.uint32), orc.reset_count)


def test_env_offset_shards_reproduce_the_global_population():
    torch = torch_cuda()
    full = oracle.OracleSim(oracle.CARTPOLE, 96, seed=12)
    ref = full.rollout(50)
    for off in (0, 32, 64):
        sim = binding.Sim(oracle.CARTPOLE, 32, 4, 12, env_offset=off)
        out = sim.rollout(50, 25)
        for k in ("obs", "act", "done"):
            assert_same_bits(to_np(out[k]), ref[k][:, off:off + 32], "shard %d %s" % (off, k))


def test_checkpoint_resume_and_split_rollout():
    torch = torch_cuda()
    a = binding.Sim(oracle.ACROBOT, 130, 4, 2)
    whole = a.rollout(90, 30)
    b = binding.Sim(oracle.ACROBOT, 130, 4, 2)
    first = b.rollout(41, 41)
    st, (ep, rc, t) = b.state(), b.counters()
    c = binding.Sim(oracle.ACROBOT, 130, 4, 2)
    c.set_state(st)
    c.set_counters(ep, rc, t)
    second = c.rollout(49, 7)
    for k in ("obs", "act", "rew", "done"):
        assert torch.equal(whole[k], torch.cat([first[k], second[k]]))
    assert torch.equal(a.state(), c.state())


@pytest.mark.parametrize("kind,S", [(oracle.CARTPOLE, 4), (oracle.ACROBOT, 4), (oracle.SYNTH, 64)])
def test_large_step_index_and_counter_restore(kind, S):
    """The action counter uses (t >> 2) truncated to 32 bits; a handle restored at a huge t, at every
    phase of the 4-step block, must keep matching the oracle."""
    torch = torch_cuda()
    for t0 in ((1 << 34) + 1, (1 << 32) - 3, 7):
        sim = binding.Sim(kind, 130, S, 13)
        orc = oracle.OracleSim(kind, 130, S, 13)
        ep, rc, _ = sim.counters()
        sim.set_counters(ep, rc, t0)
        orc.t = t0
        out = sim.rollout(21, 5)
        torch.cuda.synchronize()
        ref = orc.rollout(21)
        compare_rollout(out, sim, ref, orc, what="t0=%d" % t0)


@pytest.mark.parametrize("C", [2, 5])
def test_compute_factor_all_envs(C):
    """The paper's compute-factor knob: C dynamics iterations per recorded step, on every kernel."""
    torch = torch_cuda()
    cases = [(oracle.CARTPOLE, 4, 300, 90, 30, None), (oracle.CARTPOLE, 4, 200, 40, 8, inputs.mlp_params(1, 0.2)),
             (oracle.ACROBOT, 4, 257, 120, 50, None), (oracle.SYNTH, 4, 500, 20, 7, None), (oracle.SYNTH, 64, 77, 20, 20, None),
             (oracle.SYNTH, 512, 40, 12, 5, None), (oracle.SYNTH, 4096, 6, 9, 4, None)]
    for kind, S, n, T, K, params in cases:
        sim = binding.Sim(kind, n, S, 17, compute_factor=C)
        orc = oracle.OracleSim(kind, n, S, 17, compute_factor=C)
        if kind == oracle.SYNTH:
            st = orc.state.copy()
            st[::4] = 2.0                                   # some envs cross the threshold within a few iterations
            orc.state[:] = st
            sim.set_state(torch.from_numpy(st).cuda())
        d_params = None if params is None else torch.from_numpy(params).cuda()
        out = sim.rollout(T, K, d_params)
        torch.cuda.synchronize()
        ref = orc.rollout(T, policy_params=params)
        compare_rollout(out, sim, ref, orc, what="C=%d kind=%d S=%d" % (C, kind, S))
        # given-action steps use the same factor
        acts = inputs.forced_actions(2, 3, n, 3 if kind == oracle.ACROBOT else 2)
        for t in range(3):
            nxt, rew, done = sim.step(torch.from_numpy(acts[t]).cuda())
            o_nxt, o_rew, o_done = orc.step(acts[t])
            assert_same_bits(to_np(nxt), o_nxt, "C step next_obs")
            assert_same_bits(to_np(done), o_done, "C step done")
    L = binding.lib()
    sim = binding.Sim(oracle.CARTPOLE, 8)
    assert L.sim_set_compute_factor(sim.h, 0) == binding.SIM_EINVAL and L.sim_set_compute_factor(sim.h, 65537) == binding.SIM_EINVAL
    assert L.sim_set_compute_factor(None, 2) == binding.SIM_EINVAL


def test_null_outputs_and_reset():
    torch = torch_cuda()
    sim = binding.Sim(oracle.CARTPOLE, 777, 4, 1)
    orc = oracle.OracleSim(oracle.CARTPOLE, 777, 4, 1)
    sim.rollout(33, 33, want=())
    orc.rollout(33, want=())
    compare_rollout({}, sim, {}, orc, what="null outputs")
    only_done = sim.rollout(10, 10, want=("done",))
    assert only_done["obs"] is None and only_done["done"].shape == (10, 777)
    sim.reset()
    orc.reset()
    compare_rollout({}, sim, {}, orc, what="after reset")


def test_rollout_host_matches_device_rollout():
    torch = torch_cuda()
    n, T = 513, 37
    p = inputs.mlp_params(3, 0.1)
    for params in (None, p):
        a = binding.Sim(oracle.CARTPOLE, n, 4, 5)
        dev = a.rollout(T, 8, None if params is None else torch.from_numpy(params).cuda())
        b = binding.Sim(oracle.CARTPOLE, n, 4, 5)
        h = {"obs": torch.empty((T, n, 4), dtype=torch.float32).pin_memory(), "act": torch.empty((T, n), dtype=torch.int8).pin_memory(),
             "rew": torch.empty((T, n), dtype=torch.float32).pin_memory(), "done": torch.empty((T, n), dtype=torch.uint8).pin_memory()}
        binding.sim_rollout_host(b.h, T, 8, params, h["obs"], h["act"], h["rew"], h["done"])
        for k in h:
            assert torch.equal(dev[k].cpu(), h[k]), k
        assert torch.equal(a.state(), b.state())


def test_fused_cartpole_division_is_ieee_on_this_device():
    torch_cuda()
    sim = binding.Sim(oracle.CARTPOLE, 8)
    # every possible denominator x 2048 numerators (1.7e9 quotients) and every reciprocal
    assert binding.sim_selfcheck_division(sim.h, 2048) == 0


def test_cartpole_window_path_edge_cases():
    """States the straight-line window cannot promise anything about: angles far outside 12 degrees
    (general sin/cos), huge velocities (numerator outside the guarded range, infinities), states that
    terminate at once and repeatedly, exact zeros.  All must replay through the plain path and match."""
    def pre(sim, orc, torch):
        rng = np.random.default_rng(5)
        st = orc.state.copy()
        st[0::7] = (rng.uniform(-1, 1, st[0::7].shape) * np.array([2.3, 2.0, 3.0, 2.0])).astype(np.float32)   # |theta| up to 3 rad
        st[1::7, 3] = 1e18                       # theta_dot^2 overflows
        st[2::7, 2] = 0.2094                     # one step from the limit
        st[3::7] = 0.0                           # exact zeros: numerator of the division is +-10/1.1 * 1, fine; theta = 0
        st[4::7, 1] = 1e-30                      # tiny velocities
        st[5::7, 0] = 2.3999
        st[5::7, 1] = 3.0
        orc.state[:] = st
        sim.set_state(torch.from_numpy(st).cuda())
    for K in (1, 8, 16, 40):
        run_pair(oracle.CARTPOLE, 515, 40, K, seed=21, pre=pre)


def test_outputs_stay_inside_their_buffers():
    """Canary words around every output buffer (no memory checker runs on these kernels): ragged env counts, every
    kernel, K that does not divide T; nothing outside [T,N,...] may be written."""
    torch = torch_cuda()
    PAD = 4096
    cases = [(oracle.CARTPOLE, 4, 1003, 37, 8, None), (oracle.CARTPOLE, 4, 65, 19, 19, inputs.mlp_params(2)),
             (oracle.ACROBOT, 4, 197, 23, 7, None), (oracle.ACROBOT, 4, 130, 5, 2, None),
             (oracle.SYNTH, 4, 999, 9, 4, None), (oracle.SYNTH, 64, 33, 9, 9, None), (oracle.SYNTH, 2048, 3, 5, 2, None)]
    for kind, S, n, T, K, params in cases:
        sizes = {"obs": T * n * S * 4, "act": T * n, "rew": T * n * 4, "done": T * n}
        bufs, views = {}, {}
        for name, nbytes in sizes.items():
            padded = (nbytes + 15) // 16 * 16
            b = torch.full((PAD + padded + PAD,), 0xA5, dtype=torch.uint8, device="cuda")
            bufs[name] = (b, nbytes)
            views[name] = b[PAD:PAD + nbytes]
        sim = binding.Sim(kind, n, S, 4)
        d_params = None if params is None else torch.from_numpy(params).cuda()
        binding.sim_rollout(sim.h, T, K, d_params, views["obs"], views["act"], views["rew"], views["done"])
        state_before = sim.state().clone()
        torch.cuda.synchronize()
        for name, (b, nbytes) in bufs.items():
            assert bool((b[:PAD] == 0xA5).all()) and bool((b[PAD + nbytes:] == 0xA5).all()), (kind, S, name)
        done = views["done"].view(T, n)
        assert int(done.max()) <= 1
        # and the handle's own buffers: a second handle created right after must not be disturbed by the first
        other = binding.Sim(kind, n, S, 4)
        ref = other.rollout(T, K, d_params)
        assert torch.equal(ref["done"], done) and torch.equal(other.state(), state_before)


def test_acrobot_six_value_observation():
    torch = torch_cuda()
    sim = binding.Sim(oracle.ACROBOT, 300, 4, 3)
    out = sim.rollout(40, 40)
    states = out["obs"].reshape(-1, 4).contiguous()
    obs6 = torch.empty((states.shape[0], 6), dtype=torch.float32, device="cuda")
    binding.sim_acrobot_observation(sim.h, states, states.shape[0], obs6)
    got = to_np(obs6)
    st = to_np(states)
    for i in range(0, st.shape[0], 97):
        assert_same_bits(got[i], oracle.acrobot_observation(st[i]), "obs6 row %d" % i)
    assert float((obs6[:, 0] ** 2 + obs6[:, 1] ** 2 - 1).abs().max()) < 1e-6


def test_random_shapes_against_the_oracle():
    """Forty seeded random (env kind, S, N, T, K, C, seed, policy) combinations, including N = 1, K > T and
    rollouts split in two calls."""
    torch = torch_cuda()
    rng = np.random.default_rng(2024)
    p_mlp = inputs.mlp_params(5, 0.3)
    for case in range(40):
        kind = int(rng.integers(0, 3))
        S = int(2 ** rng.integers(2, 13)) if kind == oracle.SYNTH else 4
        n = 1 if case % 10 == 0 else int(rng.integers(1, 700 if S <= 256 else 12))
        T = int(rng.integers(1, 60))
        K = int(rng.integers(1, T + 4))
        C = int(rng.choice([1, 1, 2, 3]))
        seed = int(rng.integers(0, 2 ** 63))
        params = p_mlp if (kind == oracle.CARTPOLE and case % 3 == 0) else None
        sim = binding.Sim(kind, n, S, seed, compute_factor=C)
        orc = oracle.OracleSim(kind, n, S, seed, compute_factor=C)
        d_params = None if params is None else torch.from_numpy(params).cuda()
        T1 = int(rng.integers(0, T + 1))
        outs = []
        if T1 > 0:
            outs.append(sim.rollout(T1, K, d_params))
        if T - T1 > 0:
            outs.append(sim.rollout(T - T1, max(1, K - 1), d_params))
        torch.cuda.synchronize()
        ref = orc.rollout(T, policy_params=params)
        out = {k: torch.cat([o[k] for o in outs]) for k in ("obs", "act", "rew", "done")}
        compare_rollout(out, sim, ref, orc, what="case %d kind %d S %d n %d T %d K %d C %d" % (case, kind, S, n, T, K, C))


@pytest.mark.parametrize("K", [1, 5, 8, 13, 64, 300])
def test_bit_sliced_action_stream(K):
    """The optional one-bit-per-step action stream: windows aligned to bytes of action bits, launches starting
    at every offset inside a 128-step block, block boundaries inside a launch, the generic kernel (C > 1)."""
    torch = torch_cuda()
    for t0, C in ((0, 1), (121, 1), ((1 << 34) + 3, 1), (6, 2)):
        sim = binding.Sim(oracle.CARTPOLE, 333, 4, 19, compute_factor=C, action_stream=binding.SIM_ACTIONS_BITS)
        orc = oracle.OracleSim(oracle.CARTPOLE, 333, 4, 19, compute_factor=C, action_stream=1)
        ep, rc, _ = sim.counters()
        sim.set_counters(ep, rc, t0)
        orc.t = t0
        out = sim.rollout(300, K)
        torch.cuda.synchronize()
        ref = orc.rollout(300)
        compare_rollout(out, sim, ref, orc, what="bits K=%d t0=%d C=%d" % (K, t0, C))
    L = binding.lib()
    acro = binding.Sim(oracle.ACROBOT, 8)
    assert L.sim_set_action_stream(acro.h, binding.SIM_ACTIONS_BITS) == binding.SIM_EINVAL
    assert L.sim_set_action_stream(acro.h, 7) == binding.SIM_EINVAL and L.sim_set_action_stream(None, 0) == binding.SIM_EINVAL
    # the MLP policy is unaffected by the stream mode
    p = torch.from_numpy(inputs.mlp_params(1)).cuda()
    a = binding.Sim(oracle.CARTPOLE, 100, 4, 2, action_stream=binding.SIM_ACTIONS_BITS).rollout(20, 20, p)
    b = binding.Sim(oracle.CARTPOLE, 100, 4, 2).rollout(20, 20, p)
    assert torch.equal(a["act"], b["act"]) and torch.equal(a["obs"], b["obs"])


def test_episode_returns_entry_point():
    torch = torch_cuda()
    for kind in (oracle.CARTPOLE, oracle.ACROBOT):
        sim = binding.Sim(kind, 777, 4, 3)
        out = sim.rollout(530, 530)
        ret = torch.empty_like(out["rew"])
        carry = torch.zeros(777, dtype=torch.float32, device="cuda")
        binding.sim_episode_returns(sim.h, out["rew"][:200], out["done"][:200], 200, 777, carry, ret[:200])
        binding.sim_episode_returns(sim.h, out["rew"][200:], out["done"][200:], 330, 777, carry, ret[200:])
        want, wc = oracle.episode_returns(to_np(out["rew"]), to_np(out["done"]))
        assert_same_bits(to_np(ret), want, "returns")
        assert_same_bits(to_np(carry), wc, "carry")


def test_argument_errors_with_live_handle():
    torch = torch_cuda()
    sim = binding.Sim(oracle.ACROBOT, 16)
    L = binding.lib()
    assert L.sim_rollout(sim.h, 0, 1, None, None, None, None, None) == binding.SIM_EINVAL
    assert L.sim_rollout(sim.h, 5, 0, None, None, None, None, None) == binding.SIM_EINVAL
    p = torch.zeros(4610, device="cuda")
    assert L.sim_rollout(sim.h, 5, 1, p.data_ptr(), None, None, None, None) == binding.SIM_EINVAL   # MLP is CartPole-only
    assert L.sim_step(sim.h, None, None, None, None) == binding.SIM_EINVAL
    assert L.sim_set_env_offset(sim.h, (1 << 32) - 8) == binding.SIM_EINVAL
    ep, rc, t = sim.counters()
    assert t == 0                                         # nothing above advanced the handle


def test_rollout_records_into_a_cuda_graph_captured_by_the_caller():
    """The calls only enqueue kernels on the handle's stream, so a caller can capture reset + a one-step-per-launch
    rollout in a CUDA graph and replay it: every replay writes the oracle's trajectory again."""
    torch = torch_cuda()
    w = inputs.WORKLOADS["cfg1"]
    sim = binding.Sim(w.env_kind, w.n_envs, w.state_dim, w.seed)
    out = sim.alloc_outputs(w.T)
    st = torch.cuda.Stream()
    sim.use_stream(st)
    with torch.cuda.stream(st):
        sim.rollout(3, 1, None, out=sim.alloc_outputs(3))          # module loading and the first launches happen outside the capture
    st.synchronize()
    launches0 = sim.launches
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        sim.reset()
        sim.rollout(w.T, 1, None, out=out)
    assert sim.launches - launches0 == 1 + w.T                     # one graph node per launch
    orc = oracle.OracleSim(w.env_kind, w.n_envs, w.state_dim, seed=w.seed)
    ref = orc.rollout(w.T)
    for replay in range(2):
        for t in out.values():
            t.fill_(99)
        with torch.cuda.stream(st):
            g.replay()
        st.synchronize()
        for k in ("obs", "act", "rew", "done"):
            assert_same_bits(to_np(out[k]), ref[k], "graph replay %d %s" % (replay, k))
        assert_same_bits(to_np(sim.state()), orc.state, "state after replay")


def test_calls_with_another_device_current_are_refused():
    """A handle belongs to the device it was created on; with another device current every call that would touch
    its buffers returns SIM_ESTATE and enqueues nothing (needs two GPUs; skipped on a single-GPU machine)."""
    torch = torch_cuda()
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two CUDA devices")
    sim = binding.Sim(oracle.CARTPOLE, 64, 4, 0, device="cuda:0")
    L = binding.lib()
    with torch.cuda.device(1):
        assert L.sim_reset(sim.h) == binding.SIM_ESTATE
        assert L.sim_rollout(sim.h, 4, 4, None, None, None, None, None) == binding.SIM_ESTATE
        buf = torch.zeros(64 * 4, dtype=torch.float32, device="cuda:0")
        assert L.sim_get_state(sim.h, buf.data_ptr()) == binding.SIM_ESTATE
    with torch.cuda.device(0):
        assert L.sim_reset(sim.h) == binding.SIM_OK
