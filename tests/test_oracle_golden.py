"""The oracle against worked transitions stored under tests/golden/: CartPole Euler steps and Acrobot
derivatives / RK4 steps that `tests/golden/make_dynamics_golden.py` evaluates in float64 straight from
the equations of motion (no oracle, no CUDA).  The fp32 oracle must agree within 2e-7 (absolute, scaled
by the magnitude where a value exceeds 1) and take the same done decision."""
import os

import numpy as np

import oracle


def rows(path):
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.replace("|", " ").split()


def close(got, want, tol=2e-7):
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    return bool(np.all(np.abs(got - want) <= tol * np.maximum(1.0, np.abs(want))))


def test_cartpole_steps_match_the_worked_values(golden_dir):
    n = 0
    for r in rows(os.path.join(golden_dir, "cartpole_steps.txt")):
        s, act, want, done = [float(v) for v in r[:4]], int(r[4]), [float(v) for v in r[5:9]], int(r[9])
        nxt, d = oracle.cartpole_step(np.array(s, dtype=np.float32), act)
        assert close(nxt, want), (s, act, nxt, want)
        assert d == done, (s, act)
        n += 1
    assert n >= 4


def test_acrobot_derivative_and_rk4_steps_match_the_worked_values(golden_dir):
    n = 0
    for r in rows(os.path.join(golden_dir, "acrobot_rk4_steps.txt")):
        s, torque = [float(v) for v in r[:4]], float(r[4])
        acc, want = [float(v) for v in r[5:7]], [float(v) for v in r[7:11]]
        d = oracle.acrobot_dsdt(np.array(s, dtype=np.float32), torque)
        assert d[0] == np.float32(s[2]) and d[1] == np.float32(s[3])
        assert close(d[2:], acc, 1e-6), (s, torque, d, acc)
        nxt, _ = oracle.acrobot_step(np.array(s, dtype=np.float32), int(torque) + 1)
        assert close(nxt, want), (s, torque, nxt, want)
        n += 1
    assert n >= 3


def test_golden_files_are_what_their_generator_writes(golden_dir, tmp_path):
    """The stored values are exactly what the committed float64 script produces."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_dynamics_golden", os.path.join(golden_dir, "make_dynamics_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.HERE = str(tmp_path)
    mod.main()
    for name in ("cartpole_steps.txt", "acrobot_rk4_steps.txt"):
        assert open(os.path.join(golden_dir, name)).read() == open(os.path.join(str(tmp_path), name)).read()
