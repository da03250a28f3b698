"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Only tests, the smoke check and the bench's CPU-baseline / reference legs import this
package.  It never imports the CUDA package and shares nothing with it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oracle.c"
_LIB = _HERE / "liboracle.so"

CARTPOLE, ACROBOT, SYNTH = 0, 1, 2
CFLAGS = ["-O2", "-ffp-contract=off", "-mfma", "-std=c11", "-fPIC", "-shared", "-fvisibility=hidden"]


def build(force: bool = False) -> Path:
    """Compile oracle.c into liboracle.so next to it (gcc, strict IEEE flags)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(".so.tmp%d" % os.getpid())
        subprocess.check_call(["gcc", *CFLAGS, str(_SRC), "-o", str(tmp), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_LIB))
        u32p, f32p = C.POINTER(C.c_uint32), C.POINTER(C.c_float)
        L.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.oracle_philox4x32_10.restype = None
        L.oracle_action_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        L.oracle_action_word.restype = C.c_uint32
        L.oracle_uniform01.argtypes = [C.c_uint32]
        L.oracle_uniform01.restype = C.c_float
        L.oracle_random_action.argtypes = [C.c_int, C.c_uint32]
        L.oracle_random_action.restype = C.c_int
        L.oracle_draw_state.argtypes = [C.c_int, C.c_int, C.c_uint64, C.c_uint32, C.c_uint32, f32p]
        L.oracle_draw_state.restype = None
        L.oracle_sincos_s.argtypes = [C.c_float, f32p, f32p]
        L.oracle_sincos_s.restype = None
        for name in ("oracle_sin_s", "oracle_cos_s", "oracle_exp_s", "oracle_tanh_s"):
            getattr(L, name).argtypes = [C.c_float]
            getattr(L, name).restype = C.c_float
        L.oracle_cartpole_accel.argtypes = [f32p, C.c_int, f32p, f32p, f32p]
        L.oracle_cartpole_accel.restype = None
        L.oracle_cartpole_step.argtypes = [f32p, C.c_int, f32p]
        L.oracle_cartpole_step.restype = C.c_int
        L.oracle_acrobot_dsdt.argtypes = [f32p, C.c_float, f32p]
        L.oracle_acrobot_dsdt.restype = None
        L.oracle_acrobot_step.argtypes = [f32p, C.c_int, f32p]
        L.oracle_acrobot_step.restype = C.c_int
        L.oracle_acrobot_observation.argtypes = [f32p, f32p]
        L.oracle_acrobot_observation.restype = None
        L.oracle_synth_step.argtypes = [f32p, C.c_int, C.c_int, f32p, f32p]
        L.oracle_synth_step.restype = C.c_int
        L.oracle_pairwise_sum.argtypes = [f32p, C.c_int]
        L.oracle_pairwise_sum.restype = C.c_float
        L.oracle_map_f32.argtypes = [C.c_int, f32p, C.c_int64, f32p]
        L.oracle_map_f32.restype = None
        L.oracle_mlp_logits.argtypes = [f32p, f32p, f32p]
        L.oracle_mlp_logits.restype = None
        L.oracle_sample_action.argtypes = [f32p, C.c_uint32]
        L.oracle_sample_action.restype = C.c_int
        L.oracle_rollout_x.argtypes = [C.c_int, C.c_int, C.c_uint64, C.c_int, C.c_int, C.c_int64, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_int,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p]
        L.oracle_rollout_x.restype = C.c_int
        L.oracle_action_bit.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        L.oracle_action_bit.restype = C.c_int
        L.oracle_episode_returns.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_void_p, C.c_void_p]
        L.oracle_episode_returns.restype = None
        L.oracle_reset.argtypes = [C.c_int, C.c_int, C.c_uint64, C.c_int64, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_reset.restype = C.c_int
        _lib = L
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _fp(a):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _vp(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ---------------------------------------------------------------- scalar pieces
def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    o = np.zeros(4, dtype=np.uint32)
    u32p = C.POINTER(C.c_uint32)
    lib().oracle_philox4x32_10(c.ctypes.data_as(u32p), k.ctypes.data_as(u32p), o.ctypes.data_as(u32p))
    return o


def action_word(seed, env, t):
    return int(lib().oracle_action_word(seed, env, t))


def action_bit(seed, env, t):
    return int(lib().oracle_action_bit(seed, env, t))


def uniform01(w):
    return np.float32(lib().oracle_uniform01(w))


def random_action(env_kind, w):
    return int(lib().oracle_random_action(env_kind, w))


def draw_state(env_kind, S, seed, env, r):
    out = np.zeros(S, dtype=np.float32)
    lib().oracle_draw_state(env_kind, S, seed, env, r, _fp(out))
    return out


def sincos_s(x):
    s, c = C.c_float(), C.c_float()
    lib().oracle_sincos_s(np.float32(x), C.byref(s), C.byref(c))
    return np.float32(s.value), np.float32(c.value)


def sin_s(x):
    return np.float32(lib().oracle_sin_s(np.float32(x)))


def cos_s(x):
    return np.float32(lib().oracle_cos_s(np.float32(x)))


def exp_s(x):
    return np.float32(lib().oracle_exp_s(np.float32(x)))


def tanh_s(x):
    return np.float32(lib().oracle_tanh_s(np.float32(x)))


def map_f32(which, x):
    """Elementwise sin_s / cos_s / exp_s / tanh_s over an array."""
    idx = {"sin": 0, "cos": 1, "exp": 2, "tanh": 3}[which]
    x = _f32(x).ravel()
    out = np.zeros_like(x)
    lib().oracle_map_f32(idx, _fp(x), x.size, _fp(out))
    return out


def pairwise_sum(q):
    q = _f32(q)
    return np.float32(lib().oracle_pairwise_sum(_fp(q), q.size))


def cartpole_accel(s, act):
    s = _f32(s)
    a, b, c = C.c_float(), C.c_float(), C.c_float()
    lib().oracle_cartpole_accel(_fp(s), int(act), C.byref(a), C.byref(b), C.byref(c))
    return np.float32(a.value), np.float32(b.value), np.float32(c.value)


def cartpole_step(s, act):
    s = _f32(s)
    out = np.zeros(4, dtype=np.float32)
    done = lib().oracle_cartpole_step(_fp(s), int(act), _fp(out))
    return out, int(done)


def acrobot_dsdt(y, a):
    y = _f32(y)
    out = np.zeros(4, dtype=np.float32)
    lib().oracle_acrobot_dsdt(_fp(y), np.float32(a), _fp(out))
    return out


def acrobot_step(s, act):
    s = _f32(s)
    out = np.zeros(4, dtype=np.float32)
    goal = lib().oracle_acrobot_step(_fp(s), int(act), _fp(out))
    return out, int(goal)


def acrobot_observation(s):
    s = _f32(s)
    out = np.zeros(6, dtype=np.float32)
    lib().oracle_acrobot_observation(_fp(s), _fp(out))
    return out


def synth_step(x, act):
    x = _f32(x)
    S = x.shape[0]
    out = np.zeros(S, dtype=np.float32)
    scratch = np.zeros(S, dtype=np.float32)
    done = lib().oracle_synth_step(_fp(x), S, int(act), _fp(out), _fp(scratch))
    return out, int(done)


def mlp_logits(params, obs):
    params, obs = _f32(params), _f32(obs)
    assert params.size == 4610
    out = np.zeros(2, dtype=np.float32)
    lib().oracle_mlp_logits(_fp(params), _fp(obs), _fp(out))
    return out


def sample_action(logits, w):
    logits = _f32(logits)
    return int(lib().oracle_sample_action(_fp(logits), int(w)))


def episode_returns(rew, done, carry=None):
    rew = np.ascontiguousarray(rew, dtype=np.float32)
    done = np.ascontiguousarray(done, dtype=np.uint8)
    T, n = rew.shape
    carry = np.zeros(n, dtype=np.float32) if carry is None else np.ascontiguousarray(carry, dtype=np.float32).copy()
    ret = np.zeros((T, n), dtype=np.float32)
    lib().oracle_episode_returns(_vp(rew), _vp(done), T, n, _vp(carry), _vp(ret))
    return ret, carry


# ---------------------------------------------------------------- whole pipeline
class OracleSim:
    """Plain CPU stepper over a list of global env indices (default: 0..n-1)."""

    def __init__(self, env_kind, n_envs=None, state_dim=4, seed=0, env_ids=None, compute_factor=1, action_stream=0):
        self.kind, self.S, self.seed = int(env_kind), int(state_dim), int(seed)
        self.compute_factor = int(compute_factor)
        self.action_stream = int(action_stream)
        if env_ids is None:
            env_ids = np.arange(n_envs, dtype=np.uint32)
        self.env_ids = np.ascontiguousarray(env_ids, dtype=np.uint32)
        self.n = int(self.env_ids.shape[0])
        self.state = np.zeros((self.n, self.S), dtype=np.float32)
        self.ep_len = np.zeros(self.n, dtype=np.uint32)
        self.reset_count = np.zeros(self.n, dtype=np.uint32)
        self.t = 0
        self.reset()

    def reset(self):
        rc = lib().oracle_reset(self.kind, self.S, self.seed, self.n, _vp(self.env_ids),
                                _vp(self.state), _vp(self.ep_len), _vp(self.reset_count))
        assert rc == 0
        self.t = 0

    def rollout(self, T, policy_params=None, actions=None, want=("obs", "act", "rew", "done")):
        n, S = self.n, self.S
        obs = np.zeros((T, n, S), dtype=np.float32) if "obs" in want else None
        act = np.zeros((T, n), dtype=np.int8) if "act" in want else None
        rew = np.zeros((T, n), dtype=np.float32) if "rew" in want else None
        done = np.zeros((T, n), dtype=np.uint8) if "done" in want else None
        nxt = np.zeros((T, n, S), dtype=np.float32) if "next_obs" in want else None
        pp = None if policy_params is None else _f32(policy_params)
        ga = None if actions is None else np.ascontiguousarray(actions, dtype=np.int8).reshape(T, n)
        rc = lib().oracle_rollout_x(self.kind, S, self.seed, self.compute_factor, self.action_stream, n, _vp(self.env_ids), _vp(self.state),
                                  _vp(self.ep_len), _vp(self.reset_count), self.t, T,
                                  _vp(pp), _vp(ga), _vp(obs), _vp(act), _vp(rew), _vp(done), _vp(nxt))
        assert rc == 0, "oracle_rollout rejected its arguments"
        self.t += T
        return {"obs": obs, "act": act, "rew": rew, "done": done, "next_obs": nxt}

    def step(self, actions):
        """One step with given actions; returns (next_obs, rew, done), Gym-style."""
        r = self.rollout(1, actions=np.asarray(actions).reshape(1, self.n), want=("rew", "done", "next_obs"))
        return r["next_obs"][0], r["rew"][0], r["done"][0]
