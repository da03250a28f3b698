"""The C-ABI library loads and exports every symbol include/sim.h declares (no GPU needed),
and argument validation happens on the host before any CUDA work."""
import ctypes as C
import os
import re

import pytest

from paper_2207_07736_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sim_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(L):
    names = declared_functions()
    assert len(names) >= 15 and "sim_create" in names and "sim_rollout" in names and "sim_step" in names and "sim_reset" in names
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(binding.SIGNATURES), "python binding and header disagree"


def test_header_is_plain_c():
    import subprocess, tempfile
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "t.c")
        open(src, "w").write('#include "sim.h"\nint main(void){return SIM_POLICY_PARAM_COUNT==4610?0:1;}\n')
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", src, "-o", os.path.join(d, "t.o")])


def test_argument_errors_are_host_side(L):
    h = C.c_void_p()
    EINVAL = binding.SIM_EINVAL
    assert L.sim_create(None, 0, 8, 4, 0) == EINVAL
    assert L.sim_create(C.byref(h), 3, 8, 4, 0) == EINVAL            # unknown env kind
    assert L.sim_create(C.byref(h), -1, 8, 4, 0) == EINVAL
    assert L.sim_create(C.byref(h), 0, 0, 4, 0) == EINVAL            # n_envs out of range
    assert L.sim_create(C.byref(h), 0, 1 << 32, 4, 0) == EINVAL
    assert L.sim_create(C.byref(h), 0, 8, 8, 0) == EINVAL            # CartPole / Acrobot have 4 floats
    assert L.sim_create(C.byref(h), 1, 8, 64, 0) == EINVAL
    for bad in (0, 2, 3, 12, 48, 8192, -4):
        assert L.sim_create(C.byref(h), 2, 8, bad, 0) == EINVAL      # synthetic: power of two in [4, 4096]
    assert h.value is None
    for fn, args in [("sim_destroy", (None,)), ("sim_reset", (None,)), ("sim_set_stream", (None, None)),
                     ("sim_step", (None, None, None, None, None)), ("sim_get_state", (None, None)),
                     ("sim_rollout", (None, 1, 1, None, None, None, None, None)),
                     ("sim_rollout_host", (None, 1, 1, None, None, None, None, None)),
                     ("sim_set_policy_mode", (None, 1)), ("sim_get_device_status", (None, None)),
                     ("sim_selfcheck_tensor_wait", (None, None, None)), ("sim_set_action_stream", (None, 0)),
                     ("sim_set_compute_factor", (None, 1)), ("sim_set_env_offset", (None, 0)),
                     ("sim_episode_returns", (None, None, None, 1, 1, None, None)),
                     ("sim_acrobot_observation", (None, None, 1, None)), ("sim_policy_logits", (None, None, 1, None, None))]:
        assert getattr(L, fn)(*args) == EINVAL
    assert L.sim_launch_count(None) == -1 and L.sim_last_cuda_error(None) == 0
    for code in (0, -1, -2, -3, -4, -99):
        assert len(L.sim_strerror(code)) > 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
