#!/usr/bin/env python
"""Benchmark of the batched environment-stepping hot path on B200.

A "step" is one pass of the whole hot path over one batch: one `sim_rollout` of the workload's
N envs for its T steps at one K_fused (launch prologue, K x (action selection, physics, reward /
done, auto-reset, trajectory write), launch epilogue), continuing from the state the previous
step left.  The metric is environment-steps per second.

    python bench.py                       # every workload of the table in inputs.py (one compact line each:
                                          # K_fused sweep with roofline fractions), then the cfg2 headline line
    python bench.py --workload cfg3       # one workload as the headline line (no side passes)
    python bench.py --impl reference      # the CPU oracle on the host cores, same metric
    torchrun ... bench.py --gpus N        # one rank per GPU, disjoint env ranges, no collective in the data path

The side passes follow one protocol per (workload, K_fused): reset, one warm-up rollout, then at least five
repetitions of (untimed reset, rollout bracketed by CUDA events on the sim's stream); median and minimum are
reported.  The roofline of a point is the larger of (algorithmic bytes / measured HBM copy rate) and (nominal
flops / fp32 peak); `frac` is roofline time / measured time and `meets_60pct` says whether it reaches 0.6.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2207_07736_b200 import inputs, shard  # noqa: E402

FP32_LANES_PER_SM = 128
XU_LANES_PER_SM = 16                      # special-function unit: measured 15.9 tanh.approx.f32 per clock and SM
TANH_PER_ENV_STEP = 128
HBM_NOMINAL_GBS = 8000.0                  # the vendor's headline figure, for context beside the measured copy rate
TRAJ_BYTES_S4 = 22          # obs 16 + act 1 + rew 4 + done 1
# nominal / operation-expanded flops per env-step (fma = 2, any other fp32 op = 1, integer work = 0)
FLOPS = {"cartpole": (27, 52), "acrobot": (181, 455), "mlp": (9094, 12205)}
# padded tensor-core contractions of the two tensor policy modes (flop per env-step, FP16 operands)
TENSOR_FLOPS_PER_ENV_STEP = {"tensor": 2 * (16 * 64 + 80 * 64 + 80 * 16), "tensor_precise": 2 * (32 * 64 + 192 * 64)}
MUFU_PER_ENV_STEP = {"tensor": 128, "tensor_precise": 160}      # special-function instructions per env-step (tanh; or one ex2 each and one shared rcp per four)
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused rollout kernel, from the ncu
# captures summarised under profiles/ (keyed by workload and K_fused; other shapes report null)
NCU_TRAFFIC_BYTES = {("cfg2", 1000): 1.3863e9}
# tensor-mode policy: captured on a reduced cfg3 (N = 262 144, T = 100: 533.19 MB for 2.62e7 env-steps) and scaled
# to the full launch by env-steps (the traffic is the trajectory, proportional to env-steps)
NCU_TRAFFIC_BYTES_TENSOR = {("cfg3", 500): 533.19e6 / 2.62144e7 * (1048576 * 500)}
NCU_TRAFFIC_BYTES_TENSOR_PRECISE = {("cfg3", 500): 532.45e6 / 2.62144e7 * (1048576 * 500)}   # same reduced case, precise tensor mode
POLICY_MODES = ("exact", "tensor", "tensor_precise")
# the side passes of the default run: (key, workload, policy mode)
SIDE_PASSES = (("cfg1", "cfg1", "exact"), ("cfg3", "cfg3", "exact"), ("cfg3_tensor", "cfg3", "tensor"),
               ("cfg3_tensor_precise", "cfg3", "tensor_precise"), ("cfg4", "cfg4", "exact"),
               ("cfg5_S4", "cfg5_S4", "exact"), ("cfg5_S64", "cfg5_S64", "exact"), ("cfg5_S512", "cfg5_S512", "exact"),
               ("cfg5_S4096", "cfg5_S4096", "exact"), ("cfg2_N1048576_T200", "cfg2_N1048576_T200", "exact"))
# points the 60 % target is stated for (the largest CartPole and the synthetic-simulator configs); the others are reported only
TARGET_POINTS = {"cfg2": (1000,), "cfg3": (500,), "cfg3_tensor": (500,), "cfg3_tensor_precise": (500,),
                 "cfg5_S4": (1, 4, 16, 64, 256), "cfg5_S64": (1, 4, 16, 64, 256), "cfg5_S512": (1, 4, 16, 64, 256),
                 "cfg5_S4096": (1, 4, 16, 64, 256)}


def algorithmic_bytes_per_env_step(w, K):
    traj = (4 * w.state_dim + 6) if w.trajectory else 0
    return traj + (2 * 4 * w.state_dim + 16) / K


def nominal_flops_per_env_step(w):
    if w.env_kind == inputs.SYNTH:
        return 7 * w.state_dim, 24 * w.state_dim
    if w.env_kind == inputs.ACROBOT:
        return FLOPS["acrobot"]
    base = FLOPS["cartpole"]
    if w.mlp_seed is not None:
        return base[0] + FLOPS["mlp"][0], base[1] + FLOPS["mlp"][1]
    return base


def roofline_point(w, K, env_steps_per_sec, hbm_gbs, fp32_tflops, compute_factor=1):
    """Binding roofline of one (workload, K_fused) point and the fraction reached: the larger of the
    HBM time (algorithmic bytes) and the fp32 time (nominal flop ledger) per env-step."""
    fl_nom, fl_exp = nominal_flops_per_env_step(w)
    if compute_factor != 1:                                   # only the dynamics repeat, not the policy
        dyn = nominal_flops_per_env_step(w if w.mlp_seed is None else inputs.WORKLOADS["cfg2"])
        fl_nom += (compute_factor - 1) * dyn[0]
        fl_exp += (compute_factor - 1) * dyn[1]
    t_hbm = algorithmic_bytes_per_env_step(w, K) / (hbm_gbs * 1e9)
    t_nom = fl_nom / (fp32_tflops * 1e12)
    t_exp = fl_exp / (fp32_tflops * 1e12)
    t_meas = 1.0 / env_steps_per_sec
    bound = "hbm" if t_hbm >= t_nom else "alu"
    t_bound = max(t_hbm, t_nom)
    return {"bound": bound, "bound_env_steps_per_sec": 1.0 / t_bound, "frac": t_bound / t_meas,
            "frac_expanded_ledger": max(t_hbm, t_exp) / t_meas, "hbm_frac": t_hbm / t_meas, "fp32_nominal_frac": t_nom / t_meas,
            "flops_nominal": fl_nom, "flops_expanded": fl_exp}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), float(d.get("bf16_tflops", 1590.0)), "measured"
    return 6650.0, 1965.0, 1590.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the bench runs (read-only); `window` summarises
    the samples taken between two host times."""

    NAMES = {0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x4: "sw_power_cap",
             0x80: "hw_power_brake_slowdown"}

    def __init__(self, index, period=0.002):
        super().__init__(daemon=True)
        self.period, self.samples, self.max_mhz, self.ok = period, [], None, False
        self._halt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, r))
            except Exception:
                pass
            time.sleep(self.period)

    def window(self, t0, t1):
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        if not sel:                                               # shorter than one period: the nearest sample
            sel = sorted(self.samples, key=lambda s: abs(s[0] - 0.5 * (t0 + t1)))[:1]
        reasons = set()
        for _, _, r in sel:
            reasons |= {name for bit, name in self.NAMES.items() if r & bit}
        med = statistics.median([s[1] for s in sel]) if sel else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(reasons), "samples": len(sel)}

    def stop(self):
        self._halt.set()
        self.join(timeout=1.0)


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def config_dict(w, n, K, args, traj_bytes, world):
    """The `config` object of the JSON line; both arms print the same keys."""
    return {"workload": w.name, "env": ["cartpole", "acrobot", "synthetic"][w.env_kind], "n_envs_per_gpu": n, "T": w.T,
            "state_dim": w.state_dim, "k_fused": K, "compute_factor": args.compute_factor,
            "action_stream": "bits" if args.action_bits else "word",
            "policy": "mlp_4_64_64_2" if w.mlp_seed is not None else "uniform_random", "policy_mode": args.policy_mode,
            "trajectory_bytes_per_step": traj_bytes,
            "l2": "each step writes %.2f GB of trajectory (> 126 MB L2); no flush between steps" % (traj_bytes / 1e9) if traj_bytes > 2e8
            else "state (%.2f GB) streamed from HBM every launch" % (n * w.state_dim * 4 / 1e9),
            "parallelism": "dp%d (disjoint env ranges, no collective)" % world}


def trajectory_bytes(w, n):
    return (4 * w.state_dim + 6) * n * w.T if w.trajectory else 0


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_rate(w, budget_s, n_sample=None, compute_factor=1):
    """env-steps/s of the single-threaded oracle on a bounded sample of the workload."""
    import oracle
    n = n_sample or min(w.n_envs, 256 if w.mlp_seed is not None else max(4, 4096 * 4 // w.state_dim))
    params = None if w.mlp_seed is None else inputs.mlp_params(w.mlp_seed)
    ids = inputs.sample_env_ids(3, w.n_envs, n)
    sim = oracle.OracleSim(w.env_kind, state_dim=w.state_dim, seed=w.seed, env_ids=ids, compute_factor=compute_factor)
    want = ("obs", "act", "rew", "done") if w.trajectory else ()
    steps = 0
    t0 = time.perf_counter()
    passes = 0
    while True:
        sim.rollout(w.T, policy_params=params, want=want)
        steps += sim.n * w.T
        passes += 1
        if time.perf_counter() - t0 >= budget_s:
            break
    dt = time.perf_counter() - t0
    return steps / dt, "%d envs x T=%d x %d passes (%.1f s)" % (sim.n, w.T, passes, dt)


def oracle_rate_multicore(w, budget_s, cores, compute_factor=1):
    """The same oracle, one thread per core over disjoint env ranges (ctypes releases the GIL inside the C
    call): the analogue of the paper's multi-threaded C++ simulator (Section 3.2)."""
    import threading as th
    import numpy as np
    import oracle
    per = 64 if w.mlp_seed is not None else max(2, 2048 * 4 // w.state_dim)
    params = None if w.mlp_seed is None else inputs.mlp_params(w.mlp_seed)
    want = ("obs", "act", "rew", "done") if w.trajectory else ()
    sims = []
    for c in range(cores):
        lo = (c * per) % max(1, w.n_envs - per)
        ids = (lo + np.arange(per)).astype("uint32")
        sims.append(oracle.OracleSim(w.env_kind, state_dim=w.state_dim, seed=w.seed, env_ids=ids, compute_factor=compute_factor))
    counts = [0] * cores
    t_end = time.perf_counter() + budget_s

    def work(c):
        while time.perf_counter() < t_end:
            sims[c].rollout(w.T, policy_params=params, want=want)
            counts[c] += sims[c].n * w.T

    t0 = time.perf_counter()
    threads = [th.Thread(target=work, args=(c,)) for c in range(cores)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    dt = time.perf_counter() - t0
    return sum(counts) / dt, "%d threads x %d envs x T=%d (%.1f s)" % (cores, per, w.T, dt)


def run_reference(args, w):
    rank, _, world = shard.dist_env()
    if rank != 0:
        return 0
    per_step_budget = max(0.2, min(5.0, 60.0 / max(1, args.steps + args.warmup)))
    if args.cpu_seconds != 10.0:                                    # explicit budget per step
        per_step_budget = args.cpu_seconds
    for _ in range(args.warmup):
        oracle_rate(w, per_step_budget, compute_factor=args.compute_factor)
    rates, sample = [], ""
    t0 = time.perf_counter()
    for _ in range(args.steps):
        r, sample = oracle_rate(w, per_step_budget, compute_factor=args.compute_factor)
        rates.append(r)
    wall = time.perf_counter() - t0
    v = statistics.mean(rates)
    _, n = shard.env_range(0, max(1, world), w.n_envs)
    line = {
        "impl": "reference", "metric": "env_steps_per_sec", "value": v, "unit": "env-steps/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(w, n, args.k_fused or max(w.k_sweep), args, trajectory_bytes(w, n), max(1, world)),
        "cpu_baseline": {"value": v, "unit": "env-steps/s", "cores": 1, "kind": "oracle", "sample": "each step: " + sample},
        "e2e": {"value": v, "unit": "env-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def time_rollouts(torch, sim, w, K, reps, d_params, out):
    """Device time (ms) of `reps` rollouts, each from a fresh (untimed) reset and bracketed by its own pair of
    events on the sim's stream."""
    times = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sim.reset()
        e0.record()
        sim.rollout(w.T, K, d_params, out=out)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    return times


def policy_mode_code(binding, name):
    return {"exact": binding.SIM_POLICY_EXACT, "tensor": binding.SIM_POLICY_TENSOR, "tensor_precise": binding.SIM_POLICY_TENSOR_PRECISE}[name]


def sweep_workload(torch, binding, sim, w, n, d_params, out, sampler, peaks, reps, key, policy_mode="exact", compute_factor=1, ks=None):
    """K_fused sweep of one workload on an existing handle: per K the protocol of the module docstring, the
    binding roofline and the fraction reached, and the SM clock sampled while that K ran."""
    hbm_gbs, sm_max_mhz, bf16_tflops, _ = peaks
    sms = torch.cuda.get_device_properties(sim.device).multi_processor_count
    fp32_tflops = 2 * FP32_LANES_PER_SM * sms * sm_max_mhz * 1e6 / 1e12
    sweep = {}
    for k in (ks or w.k_sweep):
        time_rollouts(torch, sim, w, k, 1, d_params, out)                # warm-up rollout
        t_host0 = time.perf_counter()
        ts = time_rollouts(torch, sim, w, k, reps, d_params, out)
        t_host1 = time.perf_counter()
        med = statistics.median(ts)
        rate = n * w.T / (med * 1e-3)
        p = {"env_steps_per_sec": rate, "ms": med, "ms_min": min(ts), "reps": reps, "launches": -(-w.T // k),
             "bytes_per_env_step": algorithmic_bytes_per_env_step(w, k)}
        p.update(roofline_point(w, k, rate, hbm_gbs, fp32_tflops, compute_factor))
        if policy_mode != "exact" and w.mlp_seed is not None:
            # the contractions left the fp32 pipes, so `frac` on the stated roofline may exceed 1; the units that
            # bind the kernel instead are reported beside it
            p["sfu_frac"] = MUFU_PER_ENV_STEP[policy_mode] * rate / (XU_LANES_PER_SM * sms * sm_max_mhz * 1e6)
            p["tensor_frac"] = TENSOR_FLOPS_PER_ENV_STEP[policy_mode] * rate / (bf16_tflops * 1e12)
        p["meets_60pct"] = bool(p["frac"] >= 0.6)
        p["target_point"] = k in TARGET_POINTS.get(key, ())
        clk = sampler.window(t_host0, t_host1) if sampler is not None and sampler.ok else None
        if clk and clk["sm_mhz"]:
            p["sm_mhz"], p["clock_reasons"], p["clock_samples"] = clk["sm_mhz"], clk["reasons"], clk["samples"]
            p["ms_x_mhz"] = med * clk["sm_mhz"]                            # comparable across boxes whose clocks settle differently
            if p["bound"] == "alu":
                p["frac_at_sampled_clock"] = p["frac"] * sm_max_mhz / clk["sm_mhz"]
        sweep[str(k)] = p
    base = sweep.get("1")
    if base:
        for v in sweep.values():
            v["fusion_speedup_vs_k1"] = base["ms"] / v["ms"]
    return sweep


def k1_burst(torch, sim, w, sampler, peaks, launches=16, idle_s=1.5):
    """One-step launches of a state-streaming workload timed as a short burst after an idle pause, i.e. at the clock
    an unthrottled GPU runs at (the measured HBM copy rate they are compared with is itself a best-of-ten burst).  The
    sweep's own K = 1 figure is the sustained one: half a second per repetition, by which time the power cap has
    lowered the SM clock."""
    hbm_gbs = peaks[0]
    sim.reset()
    sim.rollout(4, 1, None, out={})                                      # warm-up launches
    torch.cuda.synchronize()
    time.sleep(idle_s)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    sim.rollout(launches, 1, None, out={})
    e1.record()
    e1.synchronize()
    t1 = time.perf_counter()
    ms = e0.elapsed_time(e1) / launches
    rate = w.n_envs / (ms * 1e-3)
    clk = sampler.window(t0, t1) if sampler is not None and sampler.ok else {}
    return {"launches": launches, "ms_per_launch": ms, "env_steps_per_sec": rate,
            "hbm_frac": algorithmic_bytes_per_env_step(w, 1) * rate / (hbm_gbs * 1e9), "sm_mhz": clk.get("sm_mhz"), "clock_reasons": clk.get("reasons"),
            "note": "%d one-step launches after %.1f s idle" % (launches, idle_s)}


def k1_graph(torch, sim, w, d_params, out, reps=7):
    """The launch-bound one-step-per-launch rollout replayed from a CUDA graph that the CALLER captures: the library's
    calls only enqueue kernels on the handle's stream, so reset + T one-step launches record into one graph."""
    st = torch.cuda.Stream(device=sim.device)
    prev = sim.stream
    sim.use_stream(st)
    try:
        with torch.cuda.stream(st):
            sim.reset()
            sim.rollout(w.T, 1, d_params, out=out)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            sim.reset()
            sim.rollout(w.T, 1, d_params, out=out)
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(st):
                e0.record()
                g.replay()
                e1.record()
            e1.synchronize()
            ts.append(e0.elapsed_time(e1))
        ms = statistics.median(ts)
        return {"ms": ms, "ms_min": min(ts), "reps": reps, "launches": w.T + 1, "us_per_launch": ms * 1e3 / (w.T + 1),
                "env_steps_per_sec": w.n_envs * w.T / (ms * 1e-3), "note": "reset + T one-step launches captured once by the caller, replayed"}
    except Exception as e:                                               # capture is the caller's feature, not the library's: report and go on
        return {"unavailable": "%s: %s" % (type(e).__name__, e)}
    finally:
        sim.use_stream(prev)


# Not a task config: the cfg2 kernel on a batch that fills the GPU (cfg2's 65 536 envs are 1.7 warps per scheduler), to show
# where the kernel itself stands against the store roofline.
EXTRA_WORKLOADS = {"cfg2_N1048576_T200": dataclasses.replace(inputs.WORKLOADS["cfg2"], name="cfg2_N1048576_T200", n_envs=1 << 20, T=200,
                                                             k_sweep=(200,), note="CartPole, random policy, 2^20 envs")}


def side_pass(torch, binding, key, wname, policy_mode, dev, sampler, peaks, reps):
    """One workload of the default run's side passes: its own handle and outputs, freed afterwards."""
    w = inputs.WORKLOADS.get(wname) or EXTRA_WORKLOADS[wname]
    sim = binding.Sim(w.env_kind, w.n_envs, w.state_dim, w.seed, device=dev, policy_mode=policy_mode_code(binding, policy_mode))
    d_params = None if w.mlp_seed is None else torch.from_numpy(inputs.mlp_params(w.mlp_seed)).to(dev)
    out = sim.alloc_outputs(w.T) if w.trajectory else {}
    burst = None
    try:
        if not w.trajectory and 1 in w.k_sweep:
            burst = k1_burst(torch, sim, w, sampler, peaks)              # first, while the GPU is still cool
        sweep = sweep_workload(torch, binding, sim, w, w.n_envs, d_params, out, sampler, peaks, reps, key, policy_mode)
        status = sim.device_status() if policy_mode != "exact" else 0
        graph = k1_graph(torch, sim, w, d_params, out) if key == "cfg1" else None
    finally:
        sim.close()
        del out
        torch.cuda.empty_cache()
    line = {"workload": key, "task_config": wname in inputs.WORKLOADS, "env": ["cartpole", "acrobot", "synthetic"][w.env_kind], "n_envs": w.n_envs, "T": w.T, "state_dim": w.state_dim,
            "policy": "mlp_4_64_64_2" if w.mlp_seed is not None else "uniform_random", "policy_mode": policy_mode,
            "trajectory": bool(w.trajectory), "unit": "env-steps/s", "k_sweep": sweep}
    if policy_mode != "exact":
        line["device_status"] = status
    if burst is not None:
        line["k1_burst"] = burst
    if graph is not None:
        line["k1_cuda_graph"] = graph
    below = [k for k, v in sweep.items() if v["target_point"] and not v["meets_60pct"]]
    line["target_points_below_60pct"] = below
    return line


def compact_summary(workloads, headline_key, headline_sweep):
    """One short string per workload: `K<k>=<env-steps/s>/<fraction of the binding roofline>`, with `*` after a point the
    60 % target is stated for that meets it and `!` after one that misses it.  Short enough to sit at the very end of the
    headline line, where a truncated record of the output still shows every workload."""
    def one(key, sweep):
        parts = []
        for k, v in sweep.items():
            mark = ("*" if v["meets_60pct"] else "!") if v.get("target_point") else ""
            parts.append("K%s=%.3g/%.2f%s" % (k, v["env_steps_per_sec"], v["frac"], mark))
        return key + " " + " ".join(parts)
    out = [one(key, line["k_sweep"]) for key, line in workloads.items()]
    if headline_sweep:
        out.append(one(headline_key, headline_sweep))
    return out


def run_gpu(args, w):
    import torch
    from paper_2207_07736_b200 import binding
    rank, local_rank, world = shard.dist_env()
    if world != args.gpus and world > 1:
        raise SystemExit("--gpus %d but WORLD_SIZE=%d" % (args.gpus, world))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the CPU oracle")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if not binding.LIB_PATH.exists():                               # normally built in-tree beforehand
        if local_rank == 0:
            from paper_2207_07736_b200 import build as _build
            _build.build()
        else:
            t_wait = time.time()
            while not binding.LIB_PATH.exists() and time.time() - t_wait < 600:
                time.sleep(1.0)
    dist = shard.init_process_group("nccl")
    peaks = measured_peaks()
    hbm_peak, sm_max_mhz, bf16_peak, peak_kind = peaks
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()

    # ---- side passes: every other workload of the table, one compact line each (single GPU only)
    workloads = {}
    if args.all_workloads and world == 1:
        for key, wname, mode in SIDE_PASSES:
            if args.only and key not in args.only.split(","):
                continue
            line = side_pass(torch, binding, key, wname, mode, dev, sampler, peaks, args.side_reps)
            workloads[key] = line
            print(json.dumps(line), flush=True)

    env_offset, n = shard.env_range(rank, world, w.n_envs)
    K = args.k_fused or max(w.k_sweep)
    sim = binding.Sim(w.env_kind, n, w.state_dim, w.seed, device=dev, env_offset=env_offset, compute_factor=args.compute_factor,
                      action_stream=1 if args.action_bits else 0, policy_mode=policy_mode_code(binding, args.policy_mode))
    d_params = None if w.mlp_seed is None else torch.from_numpy(inputs.mlp_params(w.mlp_seed)).to(dev)
    out = sim.alloc_outputs(w.T) if w.trajectory else {}
    traj_bytes = sum(t.numel() * t.element_size() for t in out.values() if t is not None)

    def one_step():
        sim.rollout(w.T, K, d_params, out=out)

    # warm-up: W steps; their duration sizes the ramp
    torch.cuda.synchronize()
    t_w = time.perf_counter()
    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    step_s = max(1e-5, (time.perf_counter() - t_w) / args.warmup)
    ramp_steps = max(1, int(args.ramp_s / step_s))

    # One uninterrupted run of steps on the stream: `ramp_steps` untimed steps that bring clocks and power to
    # their steady state, then EXACTLY --steps timed steps with no host synchronisation in between.
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches_ramp0 = sim.launches
    er, e0, e1 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    t_host0 = time.perf_counter()
    er.record()
    for _ in range(ramp_steps):
        one_step()
    launches0 = sim.launches
    e0.record()
    for _ in range(args.steps):
        one_step()
    e1.record()
    torch.cuda.synchronize()
    t_host1 = time.perf_counter()
    if dist is not None:
        dist.barrier()
    launches = sim.launches - launches0
    elapsed_ms = e0.elapsed_time(e1)
    sustained_ms = er.elapsed_time(e1)
    clocks = sampler.window(t_host0, t_host1)
    clocks["window"] = "ramp (%d steps) + timed steps, %.2f s of uninterrupted launches" % (ramp_steps, t_host1 - t_host0)
    units = float(n) * w.T * args.steps
    elapsed_ms, units_all = shard.reduce_timing(dist, elapsed_ms, units, device=dev)
    value = units_all / (elapsed_ms * 1e-3)
    sustained = {"value": float(n) * w.T * (ramp_steps + args.steps) / (sustained_ms * 1e-3) * world, "steps": ramp_steps + args.steps,
                 "ms_per_step": sustained_ms / (ramp_steps + args.steps), "launches": sim.launches - launches_ramp0,
                 "note": "the ramp and the timed steps together (this rank's clock)"}

    # ---- roofline of the dominant kernel (the fused rollout kernel; ceil(T/K) launches per step)
    launches_per_step = -(-w.T // K)
    launch_ms = elapsed_ms / (args.steps * launches_per_step)          # single stream, back-to-back launches
    bytes_per_env_step = algorithmic_bytes_per_env_step(w, K)
    k_per_launch = min(K, w.T)
    bytes_per_launch = bytes_per_env_step * n * k_per_launch
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    fp32_peak_tflops = 2 * FP32_LANES_PER_SM * sms * sm_max_mhz * 1e6 / 1e12
    sampled_mhz = clocks["sm_mhz"] or sm_max_mhz
    fp32_peak_sampled = 2 * FP32_LANES_PER_SM * sms * sampled_mhz * 1e6 / 1e12
    rate_rank = n * k_per_launch / (launch_ms * 1e-3)                   # env-steps/s of this GPU
    rp = roofline_point(w, K, rate_rank, hbm_peak, fp32_peak_tflops, args.compute_factor)
    fl_nom, fl_exp = rp["flops_nominal"], rp["flops_expanded"]
    if rp["bound"] == "hbm":
        achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                    "traffic": args.traffic_bytes, "peak_source": "MEASURED_PEAKS.json (of %s)" % peak_kind,
                    "algorithmic_bytes_per_launch": bytes_per_launch,
                    "frac_of_nominal_8TBs": achieved / HBM_NOMINAL_GBS}
    else:
        achieved = fl_nom * rate_rank / 1e12
        roofline = {"bound": "alu", "achieved": achieved, "peak": fp32_peak_tflops, "unit": "TFLOP/s", "frac": achieved / fp32_peak_tflops,
                    "traffic": args.traffic_bytes, "peak_source": "2 x 128 lanes x %d SMs x %.0f MHz (sm_max_mhz of MEASURED_PEAKS.json, of %s)" % (sms, sm_max_mhz, peak_kind),
                    "flops_ledger": "nominal %d flop/env-step (operation-expanded: %d)" % (fl_nom, fl_exp),
                    "frac_expanded_ledger": rp["frac_expanded_ledger"],
                    "frac_at_sampled_clock": achieved / fp32_peak_sampled,
                    "hbm_frac": rp["hbm_frac"], "hbm_frac_of_nominal_8TBs": rp["hbm_frac"] * hbm_peak / HBM_NOMINAL_GBS}
        if args.policy_mode != "exact" and w.mlp_seed is not None:
            # Tensor policy modes: the contractions are on the tensor cores, so `frac` on the stated roofline may
            # exceed 1; what binds the kernel is the special-function unit (16 lanes per SM)
            mufu = MUFU_PER_ENV_STEP[args.policy_mode]
            tfl = TENSOR_FLOPS_PER_ENV_STEP[args.policy_mode]
            roofline["sfu"] = {"ops_per_env_step": mufu, "achieved_tops": mufu * rate_rank / 1e12,
                               "peak_tops": XU_LANES_PER_SM * sms * sm_max_mhz * 1e6 / 1e12,
                               "frac": mufu * rate_rank / (XU_LANES_PER_SM * sms * sm_max_mhz * 1e6)}
            roofline["tensor"] = {"flops_per_env_step": tfl, "achieved_tflops": tfl * rate_rank / 1e12, "peak_tflops": bf16_peak,
                                  "frac": tfl * rate_rank / 1e12 / bf16_peak, "note": "FP16 tcgen05 contractions (padded shapes), against the measured dense bf16 peak"}
    roofline["fp32_peak_tflops"] = fp32_peak_tflops
    roofline["fp32_peak_at_sampled_clock"] = fp32_peak_sampled
    roofline["sampled_sm_mhz"] = clocks["sm_mhz"]
    roofline["meets_60pct"] = bool(roofline["frac"] >= 0.6)
    if roofline["traffic"] is None:
        table = NCU_TRAFFIC_BYTES if (args.policy_mode == "exact" or w.mlp_seed is None) else \
            NCU_TRAFFIC_BYTES_TENSOR if args.policy_mode == "tensor" else NCU_TRAFFIC_BYTES_TENSOR_PRECISE
        full = inputs.WORKLOADS.get(w.name)                          # None for a reduced (profiling) shape
        roofline["traffic"] = table.get((w.name, K)) if full is not None and n == full.n_envs and w.T == full.T else None
    roofline["kernel"] = "fused rollout kernel, K_fused=%d, %d launch(es) per step" % (K, launches_per_step)
    roofline["launch_ms"] = launch_ms
    roofline["launch_ms_x_mhz"] = launch_ms * sampled_mhz

    # ---- K_fused sweep (rank 0 reports its own GPU; same handle, a few repetitions each)
    sweep = {}
    if not args.no_sweep:
        sweep = sweep_workload(torch, binding, sim, w, n, d_params, out, sampler, peaks, max(5, min(args.steps, 10)), w.name,
                               args.policy_mode, args.compute_factor)

    # ---- end to end: host buffers, D2H of the trajectory (and H2D of the policy) inside the timed region
    e2e = None
    if not args.no_e2e:
        if w.trajectory:
            h = {"obs": torch.empty((w.T, n, w.state_dim), dtype=torch.float32).pin_memory(),
                 "act": torch.empty((w.T, n), dtype=torch.int8).pin_memory(),
                 "rew": torch.empty((w.T, n), dtype=torch.float32).pin_memory(),
                 "done": torch.empty((w.T, n), dtype=torch.uint8).pin_memory()}
        else:
            # no trajectory in this workload: the done flags are the only host-visible output (skipped when they
            # alone would exceed 4 GiB of pinned memory; the end-to-end number is then launch + synchronise)
            small = w.T * n <= (4 << 30)
            h = {"obs": None, "act": None, "rew": None, "done": torch.empty((w.T, n), dtype=torch.uint8).pin_memory() if small else None}
        h_params = None if w.mlp_seed is None else torch.from_numpy(inputs.mlp_params(w.mlp_seed)).pin_memory()
        k_host = min(K, max(1, w.T // 8))                               # chunked so that copies overlap compute
        del out
        torch.cuda.empty_cache()

        def host_step():
            binding.sim_rollout_host(sim.h, w.T, k_host, h_params, h["obs"], h["act"], h["rew"], h["done"])

        host_step()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        e_steps = max(1, min(args.steps, args.e2e_steps))
        t0 = time.perf_counter()
        for _ in range(e_steps):
            host_step()                                                 # returns after the last copy has landed
        torch.cuda.synchronize()
        dt_ms = (time.perf_counter() - t0) * 1e3
        dt_ms, e_units = shard.reduce_timing(dist, dt_ms, float(n) * w.T * e_steps, device=dev)
        d2h = sum(t.numel() * t.element_size() for t in h.values() if t is not None)
        e2e = {"value": e_units / (dt_ms * 1e-3), "unit": "env-steps/s", "h2d_bytes_per_step": 0 if h_params is None else h_params.numel() * 4,
               "d2h_bytes_per_step": d2h, "steps": e_steps, "k_fused_chunk": k_host, "d2h_gb_per_s": d2h * e_steps / (dt_ms * 1e-3) / 1e9,
               "note": "sim_rollout_host: trajectory copied to pinned host memory chunk by chunk while the next chunk computes"}
    sampler.stop()

    if rank != 0:
        return 0

    cpu = None
    if not args.no_cpu and world == 1:
        v, sample = oracle_rate(w, args.cpu_seconds, compute_factor=args.compute_factor)
        cpu = {"value": v, "unit": "env-steps/s", "cores": 1, "kind": "oracle", "sample": sample,
               "host_cores_available": os.cpu_count()}
        try:
            cores = len(os.sched_getaffinity(0))
        except Exception:
            cores = os.cpu_count() or 1
        if cores > 1:
            vm, sm = oracle_rate_multicore(w, min(5.0, args.cpu_seconds), cores, args.compute_factor)
            cpu["all_cores"] = {"value": vm, "cores": cores, "sample": sm}
            if e2e:
                e2e["ratio_to_oracle_all_cores"] = e2e["value"] / vm
        if e2e:
            e2e["ratio_to_oracle_1_core"] = e2e["value"] / v

    line = {
        "metric": "env_steps_per_sec", "value": value, "unit": "env-steps/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(w, n, K, args, traj_bytes, world),
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "sustained": sustained,
        "k_sweep": sweep,
    }
    if workloads:
        line["workloads"] = workloads
        line["target_points_below_60pct"] = {k: v["target_points_below_60pct"] for k, v in workloads.items() if v["target_points_below_60pct"]}
    summary = compact_summary(workloads, w.name, sweep)
    if summary:
        roofline["all_workloads"] = summary                              # also beside the headline's own roofline
        line["summary"] = summary                                        # last key: the end of the line names every workload
        line["summary_legend"] = "K<k_fused>=<env-steps/s>/<fraction of the binding roofline: max(bytes/HBM, nominal flops/fp32)>; * target point >= 0.6, ! target point below"
    print(json.dumps(line), flush=True)
    return 0


def run_grid(args):
    """Fusion speedup over the simulator-complexity grid of the paper (Section 4.2): state factor S and
    compute factor C of the synthetic simulator, K fused steps, normalised to K = 1.  One JSON line per (S, C)."""
    import torch
    from paper_2207_07736_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py --grid needs a CUDA device")
    T, ks = 64, (1, 8, 64)
    points = [(S, (128 << 20) // S, C) for S in (4, 64, 512, 4096) for C in (1, 4, 16, 64)]   # 512 MiB of state: streams from HBM at K = 1
    points += [(S, (32 << 20) // S, 1) for S in (4, 64, 512, 4096)]                            # the N axis: a quarter of the envs
    for S, n, C in points:
        sim = binding.Sim(inputs.SYNTH, n, S, 0, compute_factor=C)
        w = dataclasses.replace(inputs.WORKLOADS["cfg5_S%d" % S], n_envs=n, T=T)
        row = {"grid": "simulator_complexity", "S": S, "C": C, "n_envs": n, "T": T, "k": {}}
        for k in ks:
            time_rollouts(torch, sim, w, k, 1, None, {})
            ms = statistics.median(time_rollouts(torch, sim, w, k, 3, None, {}))
            row["k"][str(k)] = {"ms": ms, "env_steps_per_sec": n * T / (ms * 1e-3)}
        for k in ks:
            row["k"][str(k)]["fusion_speedup_vs_k1"] = row["k"]["1"]["ms"] / row["k"][str(k)]["ms"]
        print(json.dumps(row), flush=True)
        sim.close()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(inputs.WORKLOADS),
                    help="headline workload (default: cfg2, preceded by the side passes over every other workload)")
    ap.add_argument("--k-fused", type=int, default=0, help="K_fused of the timed steps (default: the largest of the workload's sweep)")
    ap.add_argument("--ramp-s", type=float, default=1.0, help="untimed steps run for about this long right before the timed steps, so the SM clock has settled")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--side-reps", type=int, default=5, help="timed repetitions per (workload, K_fused) of the side passes")
    ap.add_argument("--only", default="", help="comma-separated side passes to run (default: all)")
    ap.add_argument("--no-side", action="store_true", help="skip the side passes of the default run")
    ap.add_argument("--traffic-bytes", type=float, default=None, help="ncu dram bytes per launch, if captured for this shape")
    ap.add_argument("--n-envs", type=int, default=0, help="override the workload's env count (profiling on a reduced case)")
    ap.add_argument("--T", type=int, default=0, help="override the workload's step count (profiling on a reduced case)")
    ap.add_argument("--compute-factor", type=int, default=1, help="dynamics iterations per recorded step (the paper's knob C)")
    ap.add_argument("--policy-mode", choices=POLICY_MODES, default="exact",
                    help="MLP policy evaluation: exact fp32 (default), or one of the tensor-core tolerance modes")
    ap.add_argument("--action-bits", action="store_true", help="optional bit-sliced action stream (CartPole random policy; not the default workload)")
    ap.add_argument("--grid", action="store_true", help="fusion speedup over the S x C x K simulator-complexity grid (synthetic simulator)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    args.all_workloads = args.workload is None and not args.no_side and not (args.n_envs or args.T) and args.impl == "cuda" \
        and args.policy_mode == "exact" and args.compute_factor == 1 and not args.action_bits and not args.k_fused
    w = inputs.WORKLOADS[args.workload or "cfg2"]
    if args.n_envs or args.T:
        w = dataclasses.replace(w, name=w.name + "_reduced", n_envs=args.n_envs or w.n_envs, T=args.T or w.T)
    if args.grid:
        return run_grid(args)
    if args.impl == "reference":
        return run_reference(args, w)
    return run_gpu(args, w)


if __name__ == "__main__":
    sys.exit(main())
