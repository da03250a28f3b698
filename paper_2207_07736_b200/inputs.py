"""Seeded synthetic inputs and the workload table.

This module holds none of the method's arithmetic: it only names the workloads (sizes,
seeds, K sweeps) and draws the harness-made inputs (policy weights, forced actions) that
are handed identically to the CUDA library and to the CPU oracle.  It imports neither.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

CARTPOLE, ACROBOT, SYNTH = 0, 1, 2
MLP_PARAM_COUNT = 256 + 64 + 4096 + 64 + 128 + 2  # W1[64][4] b1[64] W2[64][64] b2[64] W3[2][64] b3[2]


@dataclass(frozen=True)
class Workload:
    name: str
    env_kind: int
    n_envs: int
    T: int
    state_dim: int = 4
    seed: int = 0
    k_sweep: tuple = (1,)
    mlp_seed: int | None = None          # None = uniform random policy
    trajectory: bool = True              # False = all four output pointers NULL
    note: str = ""


def synth_n_envs(state_dim: int, state_bytes: int = 4 << 30) -> int:
    """Number of synthetic envs whose state matrix fills `state_bytes` (4 GiB by default)."""
    return state_bytes // (4 * state_dim)


WORKLOADS = {
    "cfg1": Workload("cfg1", CARTPOLE, 1024, 200, k_sweep=(1,), note="CartPole, random policy, small"),
    "cfg2": Workload("cfg2", CARTPOLE, 65536, 1000, k_sweep=(1, 10, 100, 1000), note="CartPole, random policy"),
    "cfg3": Workload("cfg3", CARTPOLE, 1 << 20, 500, k_sweep=(1, 500), mlp_seed=1, note="CartPole, MLP 4-64-64-2 policy"),
    "cfg4": Workload("cfg4", ACROBOT, 1 << 18, 500, k_sweep=(1, 50, 500), note="Acrobot RK4, random torque"),
    **{
        "cfg5_S%d" % S: Workload("cfg5_S%d" % S, SYNTH, synth_n_envs(S), 256, state_dim=S,
                                 k_sweep=(1, 4, 16, 64, 256), trajectory=False,
                                 note="synthetic bandwidth-scaling simulator, 4 GiB of state")
        for S in (4, 64, 512, 4096)
    },
}


def mlp_params(seed: int = 1, bias_std: float = 0.0) -> np.ndarray:
    """Flat fp32 parameter vector of the 4-64-64-2 policy.

    Weights ~ N(0, 1/fan_in), drawn in float64 and rounded to fp32; biases are zero unless
    `bias_std` > 0 (tests use non-zero biases to exercise the bias terms).
    Layout: W1[64][4], b1[64], W2[64][64], b2[64], W3[2][64], b3[2], each W row = one output unit.
    """
    rng = np.random.default_rng(seed)
    parts = []
    for fan_out, fan_in in ((64, 4), (64, 64), (2, 64)):
        w = rng.standard_normal((fan_out, fan_in)) * fan_in ** -0.5
        b = rng.standard_normal(fan_out) * bias_std
        parts += [w.ravel(), b]
    out = np.concatenate(parts).astype(np.float32)
    assert out.size == MLP_PARAM_COUNT
    return out


def forced_actions(seed: int, T: int, n_envs: int, n_actions: int) -> np.ndarray:
    """int8 [T, n_envs] action indices for the step-with-given-actions path."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, n_actions, size=(T, n_envs), dtype=np.int8)


def sample_env_ids(seed: int, n_envs: int, count: int) -> np.ndarray:
    """Sorted sample of global env indices (always includes the first and the last env)."""
    rng = np.random.default_rng(seed)
    count = min(count, n_envs)
    ids = set(rng.choice(n_envs, size=count, replace=False).tolist()) | {0, n_envs - 1}
    return np.array(sorted(ids), dtype=np.uint32)
