"""The entry point for callers that cannot allocate device memory (a loop that must not stall on
cudaMalloc, a process whose memory belongs to another allocator): `sim_rollout_noalloc` keeps its
per-env working memory in a fixed array inside the library.  Its outputs must equal those of the
ordinary path (sim_create + sim_rollout) bit for bit -- the tolerance every parity test here uses --
on two calls in a row, the second with a different problem so that anything left in the shared
array by the first call would show."""
import numpy as np
import pytest

import oracle
from paper_2207_07736_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _outputs(torch, T, n, S):
    return (torch.empty((T, n, S), dtype=torch.float32, device="cuda"), torch.empty((T, n), dtype=torch.int8, device="cuda"),
            torch.empty((T, n), dtype=torch.float32, device="cuda"), torch.empty((T, n), dtype=torch.uint8, device="cuda"))


def _check_case(torch, kind, n, S, seed, T, K, params):
    stream = torch.cuda.current_stream().cuda_stream
    d_params = None if params is None else torch.from_numpy(params).cuda()
    obs, act, rew, done = _outputs(torch, T, n, S)
    for t in (obs, act, rew, done):
        t.fill_(77)                                     # stale contents must be overwritten
    binding.sim_rollout_noalloc(kind, n, S, seed, T, K, d_params, obs, act, rew, done, stream)
    torch.cuda.synchronize()
    ref = binding.Sim(kind, n, S, seed)
    want = ref.rollout(T, K, d_params)
    torch.cuda.synchronize()
    assert torch.equal(obs, want["obs"]) and torch.equal(act, want["act"])
    assert torch.equal(rew, want["rew"]) and torch.equal(done, want["done"])
    assert int(done.sum()) > 0 or kind == binding.SIM_SYNTH


def test_noalloc_rollout_matches_the_allocating_path_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    # first call: CartPole, random policy, a ragged env count
    _check_case(torch, binding.SIM_CARTPOLE, 4099, 4, 3, 80, 16, None)
    # second call right after it: more envs than before and fewer, other env kinds, other seeds
    _check_case(torch, binding.SIM_ACROBOT, 5000, 4, 11, 520, 130, None)
    _check_case(torch, binding.SIM_CARTPOLE, 700, 4, 5, 40, 40, inputs.mlp_params(1))
    _check_case(torch, binding.SIM_SYNTH, 300, 512, 9, 12, 5, None)
    # and the first problem again: same bits as before
    _check_case(torch, binding.SIM_CARTPOLE, 4099, 4, 3, 80, 16, None)


def test_noalloc_matches_the_oracle_directly():
    """Not only transitively through the allocating path: one case against the CPU oracle itself, an Acrobot launch
    long enough for the launch planner to pick the packed two-env kernel."""
    import torch
    n, T, K, seed = 777, 48, 12, 21
    obs, act, rew, done = _outputs(torch, T, n, 4)
    binding.sim_rollout_noalloc(binding.SIM_ACROBOT, n, 4, seed, T, K, None, obs, act, rew, done, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    ref = oracle.OracleSim(oracle.ACROBOT, n, 4, seed=seed).rollout(T)
    for name, got in (("obs", obs), ("act", act), ("rew", rew), ("done", done)):
        assert np.array_equal(got.cpu().numpy().view(np.uint8), ref[name].view(np.uint8)), name


def test_noalloc_calls_after_the_first_allocate_nothing():
    """The first call on a device looks up the array's address (the driver may load the library's device image then);
    every later call must leave the device's free memory and torch's allocator untouched."""
    import torch
    n, T = 3000, 16
    obs, act, rew, done = _outputs(torch, T, n, 4)
    stream = torch.cuda.current_stream().cuda_stream
    cases = ((binding.SIM_CARTPOLE, 4, 4), (binding.SIM_ACROBOT, 4, 8), (binding.SIM_CARTPOLE, 4, 16))
    for kind, S, k in cases:                                        # warm-up: address lookup, and each kernel launched once
        binding.sim_rollout_noalloc(kind, n, S, 1, T, k, None, obs, act, rew, done, stream)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for seed in (2, 3):
        for kind, S, k in cases:
            binding.sim_rollout_noalloc(kind, n, S, seed, T, k, None, obs, act, rew, done, stream)
            torch.cuda.synchronize()
            free1, _ = torch.cuda.mem_get_info()
            assert free1 == free0, (kind, free0, free1)
            assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


def test_noalloc_rejects_what_does_not_fit():
    import torch
    L = binding.lib()
    cap = binding.SIM_NOALLOC_SCRATCH_BYTES
    too_many = cap // 24 + 64                               # four-float envs: 16 B state + 8 B counters each
    assert L.sim_rollout_noalloc(binding.SIM_CARTPOLE, too_many, 4, 0, 4, 4, None, None, None, None, None, None) == binding.SIM_ECAPACITY
    assert L.sim_rollout_noalloc(binding.SIM_SYNTH, 1024, 4096, 0, 4, 4, None, None, None, None, None, None) == binding.SIM_ECAPACITY
    assert b"scratch" in L.sim_strerror(binding.SIM_ECAPACITY)
    assert L.sim_rollout_noalloc(7, 16, 4, 0, 4, 4, None, None, None, None, None, None) == binding.SIM_EINVAL
    assert L.sim_rollout_noalloc(binding.SIM_ACROBOT, 16, 8, 0, 4, 4, None, None, None, None, None, None) == binding.SIM_EINVAL
    assert L.sim_rollout_noalloc(binding.SIM_CARTPOLE, 16, 4, 0, 0, 4, None, None, None, None, None, None) == binding.SIM_EINVAL
    # the largest count that fits runs: 16 n + 2 * 256-aligned(4 n) <= 8 MiB holds up to n = 349504
    fits = 349504
    assert L.sim_rollout_noalloc(binding.SIM_CARTPOLE, fits + 1, 4, 0, 2, 2, None, None, None, None, None, None) == binding.SIM_ECAPACITY
    assert L.sim_rollout_noalloc(binding.SIM_CARTPOLE, 349520, 4, 0, 2, 2, None, None, None, None, None, None) == binding.SIM_ECAPACITY
    done = torch.empty((2, fits), dtype=torch.uint8, device="cuda")
    binding.sim_rollout_noalloc(binding.SIM_CARTPOLE, fits, 4, 0, 2, 2, None, None, None, None, done, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(done.max()) <= 1
