"""The bench's reference arm and its roofline arithmetic (CPU only; the GPU arm is exercised on the B200)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2207_07736_b200 import inputs  # noqa: E402


def test_algorithmic_bytes_and_flops():
    w2, w5 = inputs.WORKLOADS["cfg2"], inputs.WORKLOADS["cfg5_S4096"]
    assert bench.algorithmic_bytes_per_env_step(w2, 1) == 22 + 48
    assert abs(bench.algorithmic_bytes_per_env_step(w2, 1000) - 22.048) < 1e-9
    assert bench.algorithmic_bytes_per_env_step(w5, 1) == 8 * 4096 + 16          # no trajectory for the synthetic config
    assert bench.algorithmic_bytes_per_env_step(w5, 4) == (8 * 4096 + 16) / 4
    assert bench.nominal_flops_per_env_step(w2) == (27, 52)
    assert bench.nominal_flops_per_env_step(inputs.WORKLOADS["cfg3"]) == (27 + 9094, 52 + 12205)
    assert bench.nominal_flops_per_env_step(w5) == (7 * 4096, 24 * 4096)


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "3",
                          "--cpu-seconds", "0.05"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "env_steps_per_sec" and line["unit"] == "env-steps/s"
    assert line["higher_is_better"] is True and line["steps"] == 2 and line["warmup"] == 3 and line["value"] > 1e5
    assert line["config"]["workload"] == "cfg2" and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1 and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "env-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_both_arms_print_the_same_config_keys():
    """The reference arm's `config` names the workload with the keys (and, for one GPU, the values) the CUDA arm prints."""
    import argparse
    w = inputs.WORKLOADS["cfg2"]
    args = argparse.Namespace(compute_factor=1, action_bits=False, policy_mode="exact")
    gpu = bench.config_dict(w, w.n_envs, 1000, args, bench.trajectory_bytes(w, w.n_envs), 1)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "3",
                          "--cpu-seconds", "0.05"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    ref = json.loads(out.stdout.strip().splitlines()[-1])["config"]
    assert ref == gpu
    assert gpu["trajectory_bytes_per_step"] == 22 * 65536 * 1000


def test_roofline_point_picks_the_binding_bound():
    hbm, fp32 = 6548.8, 74.44992
    w2, w3, w5 = inputs.WORKLOADS["cfg2"], inputs.WORKLOADS["cfg3"], inputs.WORKLOADS["cfg5_S4096"]
    p = bench.roofline_point(w2, 1000, 2.5e11, hbm, fp32)
    assert p["bound"] == "hbm" and abs(p["frac"] - 22.048 * 2.5e11 / 6548.8e9) < 1e-9
    p = bench.roofline_point(w3, 500, 4.17e9, hbm, fp32)
    assert p["bound"] == "alu" and abs(p["frac"] - 9121 * 4.17e9 / 74.44992e12) < 1e-9 and p["frac_expanded_ledger"] > p["frac"]
    assert bench.roofline_point(w5, 1, 1.37e8, hbm, fp32)["bound"] == "hbm"            # state streaming
    assert bench.roofline_point(w5, 256, 3.4e8, hbm, fp32)["bound"] == "alu"           # fused: the sine


def test_compact_summary_marks_target_points():
    sweep = {"1": {"env_steps_per_sec": 1.0e9, "frac": 0.7, "meets_60pct": True, "target_point": True},
             "4": {"env_steps_per_sec": 2.0e9, "frac": 0.3, "meets_60pct": False, "target_point": True},
             "16": {"env_steps_per_sec": 3.0e9, "frac": 0.1, "meets_60pct": False, "target_point": False}}
    out = bench.compact_summary({"w": {"k_sweep": sweep}}, "cfg2", {"1000": {"env_steps_per_sec": 2.5e11, "frac": 0.85, "meets_60pct": True, "target_point": True}})
    assert out == ["w K1=1e+09/0.70* K4=2e+09/0.30! K16=3e+09/0.10", "cfg2 K1000=2.5e+11/0.85*"]
    # every side pass names a workload of the table or one of the extra (non-task) ones, and the target table only names side passes
    keys = {k for k, _, _ in bench.SIDE_PASSES}
    assert all(w in inputs.WORKLOADS or w in bench.EXTRA_WORKLOADS for _, w, _ in bench.SIDE_PASSES)
    assert set(bench.TARGET_POINTS) - {"cfg2"} <= keys


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1"],
                         capture_output=True, text=True, timeout=60, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
