"""Thin ctypes binding of the C ABI in include/sim.h (argument marshalling only).

Every function has the name and argument order of its C counterpart.  Device pointers are
passed as integers (`tensor.data_ptr()`), or as torch tensors / None, which `_ptr` unwraps.
Nothing here computes: if the CUDA library is missing the import of the library fails loudly.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libsim_b200.so"

SIM_CARTPOLE, SIM_ACROBOT, SIM_SYNTH = 0, 1, 2
SIM_OK, SIM_EINVAL, SIM_ENOMEM, SIM_ECUDA, SIM_ESTATE, SIM_ECAPACITY = 0, -1, -2, -3, -4, -5
SIM_NOALLOC_SCRATCH_BYTES = 8 << 20
SIM_POLICY_PARAM_COUNT = 4610

# name -> (restype, argtypes); one entry per declaration in include/sim.h
SIGNATURES = {
    "sim_create": (C.c_int, [C.POINTER(C.c_void_p), C.c_int, C.c_int64, C.c_int, C.c_uint64]),
    "sim_destroy": (C.c_int, [C.c_void_p]),
    "sim_set_stream": (C.c_int, [C.c_void_p, C.c_void_p]),
    "sim_set_env_offset": (C.c_int, [C.c_void_p, C.c_uint64]),
    "sim_set_compute_factor": (C.c_int, [C.c_void_p, C.c_int]),
    "sim_set_action_stream": (C.c_int, [C.c_void_p, C.c_int]),
    "sim_set_policy_mode": (C.c_int, [C.c_void_p, C.c_int]),
    "sim_get_device_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_uint32)]),
    "sim_selfcheck_tensor_wait": (C.c_int, [C.c_void_p, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]),
    "sim_reset": (C.c_int, [C.c_void_p]),
    "sim_step": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "sim_rollout": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "sim_rollout_host": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "sim_get_state": (C.c_int, [C.c_void_p, C.c_void_p]),
    "sim_set_state": (C.c_int, [C.c_void_p, C.c_void_p]),
    "sim_get_counters": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_uint64)]),
    "sim_set_counters": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64]),
    "sim_policy_logits": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]),
    "sim_acrobot_observation": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "sim_episode_returns": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_void_p, C.c_void_p]),
    "sim_selfcheck_division": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_uint64)]),
    "sim_rollout_noalloc": (C.c_int, [C.c_int, C.c_int64, C.c_int, C.c_uint64, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_void_p]),
    "sim_launch_count": (C.c_int64, [C.c_void_p]),
    "sim_strerror": (C.c_char_p, [C.c_int]),
    "sim_last_cuda_error": (C.c_int, [C.c_void_p]),
}

_lib = None


def lib() -> C.CDLL:
    """Load libsim_b200.so (built by `paper_2207_07736_b200.build`); raise if it is absent."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                "CUDA library %s is missing: run `python -m paper_2207_07736_b200.build` "
                "(there is no CPU fallback)" % LIB_PATH)
        L = C.CDLL(str(LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)          # AttributeError if the library does not export it
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class SimError(RuntimeError):
    def __init__(self, code, cuda=0):
        self.code, self.cuda = code, cuda
        msg = lib().sim_strerror(code).decode()
        super().__init__("%s (code %d%s)" % (msg, code, ", cudaError %d" % cuda if cuda else ""))


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return C.c_void_p(x)
    if hasattr(x, "data_ptr"):
        return C.c_void_p(x.data_ptr())
    if hasattr(x, "ctypes"):                       # numpy array (host pointers of sim_rollout_host)
        return C.c_void_p(x.ctypes.data)
    raise TypeError("expected None, an address, a torch tensor or a numpy array")


def _check(code, handle=None):
    if code != SIM_OK:
        raise SimError(code, lib().sim_last_cuda_error(handle) if handle else 0)


def sim_create(env_kind, n_envs, state_dim=4, seed=0):
    h = C.c_void_p()
    _check(lib().sim_create(C.byref(h), env_kind, n_envs, state_dim, seed))
    return h


def sim_destroy(h):
    _check(lib().sim_destroy(h))


def sim_set_stream(h, cuda_stream):
    _check(lib().sim_set_stream(h, C.c_void_p(cuda_stream) if cuda_stream else None), h)


def sim_set_env_offset(h, env_offset):
    _check(lib().sim_set_env_offset(h, env_offset), h)


def sim_set_compute_factor(h, compute_factor):
    _check(lib().sim_set_compute_factor(h, compute_factor), h)


SIM_ACTIONS_WORD, SIM_ACTIONS_BITS = 0, 1


def sim_set_action_stream(h, mode):
    _check(lib().sim_set_action_stream(h, mode), h)


SIM_POLICY_EXACT, SIM_POLICY_TENSOR, SIM_POLICY_TENSOR_PRECISE = 0, 1, 2
SIM_STATUS_TENSOR_WAIT = 1


def sim_set_policy_mode(h, mode):
    _check(lib().sim_set_policy_mode(h, mode), h)


def sim_get_device_status(h) -> int:
    flags = C.c_uint32(0)
    _check(lib().sim_get_device_status(h, C.byref(flags)), h)
    return flags.value


def sim_selfcheck_tensor_wait(h):
    """(status word, threads that reported success) of the bounded-wait self-check launch."""
    status, completed = C.c_uint32(0), C.c_uint32(0)
    _check(lib().sim_selfcheck_tensor_wait(h, C.byref(status), C.byref(completed)), h)
    return status.value, completed.value


def sim_reset(h):
    _check(lib().sim_reset(h), h)


def sim_step(h, d_actions, d_next_obs=None, d_rew=None, d_done=None):
    _check(lib().sim_step(h, _ptr(d_actions), _ptr(d_next_obs), _ptr(d_rew), _ptr(d_done)), h)


def sim_rollout(h, T, K_fused, d_policy_params=None, out_obs=None, out_act=None, out_rew=None, out_done=None):
    _check(lib().sim_rollout(h, T, K_fused, _ptr(d_policy_params), _ptr(out_obs), _ptr(out_act), _ptr(out_rew), _ptr(out_done)), h)


def sim_rollout_host(h, T, K_fused, h_policy_params=None, h_obs=None, h_act=None, h_rew=None, h_done=None):
    _check(lib().sim_rollout_host(h, T, K_fused, _ptr(h_policy_params), _ptr(h_obs), _ptr(h_act), _ptr(h_rew), _ptr(h_done)), h)


def sim_get_state(h, d_state):
    _check(lib().sim_get_state(h, _ptr(d_state)), h)


def sim_set_state(h, d_state):
    _check(lib().sim_set_state(h, _ptr(d_state)), h)


def sim_get_counters(h, d_ep_len=None, d_reset_count=None):
    t = C.c_uint64()
    _check(lib().sim_get_counters(h, _ptr(d_ep_len), _ptr(d_reset_count), C.byref(t)), h)
    return t.value


def sim_set_counters(h, d_ep_len, d_reset_count, t):
    _check(lib().sim_set_counters(h, _ptr(d_ep_len), _ptr(d_reset_count), t), h)


def sim_policy_logits(h, d_obs, M, d_params, d_logits):
    _check(lib().sim_policy_logits(h, _ptr(d_obs), M, _ptr(d_params), _ptr(d_logits)), h)


def sim_acrobot_observation(h, d_state, M, d_obs6):
    _check(lib().sim_acrobot_observation(h, _ptr(d_state), M, _ptr(d_obs6)), h)


def sim_episode_returns(h, d_rew, d_done, T, n, d_carry, d_ret):
    _check(lib().sim_episode_returns(h, _ptr(d_rew), _ptr(d_done), T, n, _ptr(d_carry), _ptr(d_ret)), h)


def sim_selfcheck_division(h, nums_per_den):
    out = C.c_uint64()
    _check(lib().sim_selfcheck_division(h, nums_per_den, C.byref(out)), h)
    return out.value


def sim_rollout_noalloc(env_kind, n_envs, state_dim, seed, T, K_fused, d_policy_params=None, out_obs=None, out_act=None,
                        out_rew=None, out_done=None, cuda_stream=None):
    """Reset + rollout using the library's fixed scratch array; allocates nothing (see include/sim.h)."""
    _check(lib().sim_rollout_noalloc(env_kind, n_envs, state_dim, seed, T, K_fused, _ptr(d_policy_params), _ptr(out_obs), _ptr(out_act),
                                     _ptr(out_rew), _ptr(out_done), C.c_void_p(cuda_stream) if cuda_stream else None))


def sim_launch_count(h):
    return lib().sim_launch_count(h)


class Sim:
    """Owning wrapper of one handle, with torch tensors for the outputs (memory plumbing only)."""

    def __init__(self, env_kind, n_envs, state_dim=4, seed=0, device="cuda:0", env_offset=0, compute_factor=1, action_stream=0, policy_mode=0):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.kind, self.n, self.S, self.seed = env_kind, n_envs, state_dim, seed
        with torch.cuda.device(self.device):
            self.h = sim_create(env_kind, n_envs, state_dim, seed)
            if env_offset:
                sim_set_env_offset(self.h, env_offset)
                sim_reset(self.h)
            if compute_factor != 1:
                sim_set_compute_factor(self.h, compute_factor)
            if action_stream:
                sim_set_action_stream(self.h, action_stream)
            if policy_mode:
                sim_set_policy_mode(self.h, policy_mode)
        self.use_stream(None)

    def use_stream(self, stream):
        """Bind to a torch.cuda.Stream (None = torch's current stream on the device)."""
        st = stream or self.torch.cuda.current_stream(self.device)
        self.stream = st
        sim_set_stream(self.h, st.cuda_stream)

    def close(self):
        if self.h:
            with self.torch.cuda.device(self.device):
                sim_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        with self.torch.cuda.device(self.device):
            sim_reset(self.h)

    def alloc_outputs(self, T, want=("obs", "act", "rew", "done")):
        t, d, n, S = self.torch, self.device, self.n, self.S
        return {
            "obs": t.empty((T, n, S), dtype=t.float32, device=d) if "obs" in want else None,
            "act": t.empty((T, n), dtype=t.int8, device=d) if "act" in want else None,
            "rew": t.empty((T, n), dtype=t.float32, device=d) if "rew" in want else None,
            "done": t.empty((T, n), dtype=t.uint8, device=d) if "done" in want else None,
        }

    def rollout(self, T, K_fused, policy_params=None, out=None, want=("obs", "act", "rew", "done")):
        if out is None:
            out = self.alloc_outputs(T, want)
        with self.torch.cuda.device(self.device):
            sim_rollout(self.h, T, K_fused, policy_params, out.get("obs"), out.get("act"), out.get("rew"), out.get("done"))
        return out

    def step(self, actions):
        t, d = self.torch, self.device
        nxt = t.empty((self.n, self.S), dtype=t.float32, device=d)
        rew = t.empty((self.n,), dtype=t.float32, device=d)
        done = t.empty((self.n,), dtype=t.uint8, device=d)
        with t.cuda.device(d):
            sim_step(self.h, actions, nxt, rew, done)
        return nxt, rew, done

    def state(self):
        st = self.torch.empty((self.n, self.S), dtype=self.torch.float32, device=self.device)
        with self.torch.cuda.device(self.device):
            sim_get_state(self.h, st)
        return st

    def set_state(self, st):
        assert st.is_contiguous() and st.dtype == self.torch.float32 and tuple(st.shape) == (self.n, self.S)
        with self.torch.cuda.device(self.device):
            sim_set_state(self.h, st)

    def counters(self):
        t = self.torch
        ep = t.empty((self.n,), dtype=t.int32, device=self.device)
        rc = t.empty((self.n,), dtype=t.int32, device=self.device)
        with t.cuda.device(self.device):
            tt = sim_get_counters(self.h, ep, rc)
        return ep, rc, tt

    def set_counters(self, ep_len, reset_count, t):
        with self.torch.cuda.device(self.device):
            sim_set_counters(self.h, ep_len, reset_count, t)

    def policy_logits(self, obs, params):
        out = self.torch.empty((obs.shape[0], 2), dtype=self.torch.float32, device=self.device)
        with self.torch.cuda.device(self.device):
            sim_policy_logits(self.h, obs, obs.shape[0], params, out)
        return out

    def device_status(self):
        with self.torch.cuda.device(self.device):
            return sim_get_device_status(self.h)

    @property
    def launches(self):
        return sim_launch_count(self.h)
