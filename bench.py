#!/usr/bin/env python
"""Benchmark of the batched Pong rollout: env-steps/s on B200 and the achieved
fraction of the HBM roofline.

One "step" of this benchmark is one fused rollout launch over the whole batch:
by default N = 65,536 envs x T = 128 agent steps with in-kernel Philox actions,
vector observations float32[T,N,6] plus reward and done buffers, and the episode
statistics reduction, i.e. 8,388,608 env-steps and 243 MB written per step.
--workload selects one of the other configurations instead.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload rollout65k|rollout1m|pixels16k|step4096|small64|
                                cartpole65k|cartpole1m|policy65k]

Timing follows the paper's protocol (warm-up excluded, mean and spread over at least
five runs): five repeats are timed, each made of as many whole blocks of K launches
(--steps) as it takes to put at least 0.25 s of device time into the timed region, all
back to back with CUDA events between repeats only; `value` comes from the whole region,
`segments` holds the per-repeat rates, clocks are sampled inside it.
The default run also appends one short record for each of the other configurations
("configs").

Prints one JSON line (rank 0).  With --gpus N > 1 it must be launched with
torchrun, one rank per GPU; each rank simulates its own 65,536 envs (global env
ids rank*65536 ...), so the scaling is weak and there is no data-path
collective.  --impl reference times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SEED = 0
METRIC = "env-steps/sec on 1 B200 and achieved HBM GB/s fraction of roofline"
UNIT = "env-steps/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# The default workload ("rollout65k") is the one the headline metric is quoted
# on; the others are the remaining configurations, selectable with --workload.
# bytes: algorithmic bytes per env-step = outputs written per agent step plus the
# 32-byte state read and written once per launch (64 / T); the single-step API
# also reads one action byte.  CartPole: obs 16 + reward 4 + done 1, state 24 bytes.
# traffic: dram__bytes_read.sum + dram__bytes_write.sum of one launch from an ncu
# capture of that workload (profiles/; for the two vector rollouts a steady-state capture
# without cache flushes), None if not captured for the current kernel.
# alu_per_warp_step: integer-ALU-pipe instructions the kernel executes per warp and agent
# step, from the same profiles (sm__inst_executed_pipe_alu); with the ALU rate measured live
# it gives the secondary, compute-side ceiling of the rollout.
WORKLOADS = {
    "rollout65k": dict(
        name="fused vector-obs rollout, N=65536 envs, T=128 steps per launch, in-kernel Philox actions",
        n=65536, T=128, mode=0, obs_mode=0, frameskip=1, bytes=29.0 + 64.0 / 128,
        kernel="k_rollout_vector_chains", traffic=243.7e6, alu_per_warp_step=48.1),
    "rollout1m": dict(
        name="fused vector-obs rollout, N=1048576 envs, T=32 steps per launch, in-kernel Philox sticky actions",
        n=1048576, T=32, mode=1, obs_mode=0, frameskip=1, bytes=29.0 + 64.0 / 32,
        kernel="k_rollout_vector_tma", traffic=1038.8e6, alu_per_warp_step=38.9),
    "pixels16k": dict(
        name="pixel-obs rollout, N=16384 envs, T=64 agent steps per launch, frameskip 4, 4-frame ring uint8[N,4,84,84]",
        n=16384, T=64, mode=0, obs_mode=1, frameskip=4, bytes=7056.0 + 5.0 + 64.0 / 64,
        kernel="k_rollout_pixels_x4", traffic=7271.0e6),
    "step4096": dict(
        name="single-step API pong_step, N=4096 envs, one agent step per launch, actions from a device buffer",
        n=4096, T=1, mode=2, obs_mode=0, frameskip=1, bytes=94.0,
        kernel="k_rollout_vector", traffic=None),
    "cartpole65k": dict(
        name="CartPole fused rollout, N=65536 envs, T=128 steps per launch, in-kernel Philox actions",
        env="cartpole", n=65536, T=128, mode=0, obs_mode=0, frameskip=1, bytes=21.0 + 48.0 / 128,
        kernel="k_cartpole_chains", traffic=176.4e6),
    "cartpole1m": dict(
        name="CartPole fused rollout, N=1048576 envs, T=32 steps per launch, in-kernel Philox actions",
        env="cartpole", n=1048576, T=32, mode=0, obs_mode=0, frameskip=1, bytes=21.0 + 48.0 / 32,
        kernel="k_cartpole_rollout", traffic=753.6e6),
    "policy65k": dict(
        name="policy in the loop: gru_policy_encode -> gru_policy_cell (tcgen05, 2.0 M parameters, bf16) -> "
             "gru_policy_head -> pong_sample_actions -> pong_step, N=65536 envs, 32 agent steps per "
             "CUDA graph",
        env="policy", n=65536, T=32, mode=2, obs_mode=0, frameskip=1, bytes=94.0 + 12.0 + 4.0 + 1.0,
        kernel="k_gru_cell", traffic=None),
    "small64": dict(
        name="fused vector-obs rollout, N=64 envs, T=2000 steps per launch, in-kernel Philox actions",
        n=64, T=2000, mode=0, obs_mode=0, frameskip=1, bytes=29.0 + 64.0 / 2000,
        kernel="k_rollout_vector_tma", traffic=None),
}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only)."""

    def __init__(self, index, period=0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples = []          # (time, sm_mhz, reasons bitmask)
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev))
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)

    def summary(self, t0, t1):
        names = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        where = "timed region"
        if not inside:
            inside, where = self.samples, "whole run (timed region shorter than the sampling period)"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0,
                    "note": "NVML unavailable"}
        mhz = sorted(s[1] for s in inside)
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = [n for b, n in names.items() if mask & b]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(inside), "sampled_over": where}


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def oracle_sample(w):
    """The oracle on a bounded sample of a workload: its first envs, same T,
    action mode, obs mode and frameskip.  Returns (oracle, n_sample, call)."""
    import numpy as np
    import oracle
    from paper_2603_12145_b200.inputs import explicit_actions
    n_sample = min(w["n"], 256 if w["obs_mode"] == 1 else 8192)
    if w.get("env") == "policy":
        n_sample = 64
        return None, n_sample, policy_oracle_call(n_sample, w["T"])
    if w.get("env") == "cartpole":
        from oracle import cartpole as oracle_cartpole
        o = oracle_cartpole.OracleCartPole(n_sample, SEED)
        return o, n_sample, (lambda: o.rollout(w["T"], w["mode"]))
    o = oracle.OraclePong(n_sample, SEED, obs_mode=w["obs_mode"], frameskip=w["frameskip"])
    if w["mode"] == 2:
        acts = explicit_actions(w["T"], n_sample, seed=SEED)
        return o, n_sample, (lambda: o.rollout(w["T"], 2, acts))
    return o, n_sample, (lambda: o.rollout(w["T"], w["mode"]))


def policy_oracle_call(n_sample, T, hidden=576):
    """The whole agent step from the oracles alone (encoder, binary64 cell rounded once to
    bfloat16, head, sampling, env step), T steps per call on the first n_sample envs."""
    import numpy as np
    import oracle
    from oracle import gru_policy as ogp
    from paper_2603_12145_b200.inputs import policy_weights
    p = policy_weights(hidden, SEED)
    o = oracle.OraclePong(n_sample, SEED)
    state = {"obs": o.reset(), "h": np.zeros((n_sample, hidden), np.float32)}

    def call():
        words = o.fill_words(T)
        obs, h = state["obs"], state["h"]
        for i in range(T):
            x = ogp.encode(obs, p["enc_w"], p["enc_b"])
            h = ogp.bf16_round_f64(ogp.cell(x, h, p["w_ih"], p["w_hh"], p["b_ih"], p["b_hh"]))
            logits = ogp.head(h, p["head_w"], p["head_b"]).astype(np.float32)
            obs, _, done = o.step(oracle.sample_actions(logits, words[i]))
            h[done != 0] = 0.0
        state["obs"], state["h"] = obs, h

    return call


def cpu_oracle_rate(w, budget_s):
    """Env-steps/s of the CPU oracle, as it stands, on one host thread, repeated
    until the time budget is used."""
    o, n_sample, call = oracle_sample(w)
    call()                                      # warm-up (page-in, first touch)
    steps, reps, t0 = 0, 0, time.perf_counter()
    while True:
        call()
        steps += n_sample * w["T"]
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s:
            break
    return steps / dt, reps, dt, n_sample


def run_reference(args, rank):
    if rank != 0:
        return
    w = WORKLOADS[args.workload]
    WORKLOAD = w["name"]
    o, n_sample, call = oracle_sample(w)
    for _ in range(max(min(args.warmup, 5), 1)):
        call()
    # each step: one oracle call (T agent steps) on the first n_sample envs of the
    # workload; the run is capped at about two minutes whatever --steps says
    k = args.steps if args.steps > 0 else 50
    t0 = time.perf_counter()
    done_steps = 0
    for i in range(k):
        call()
        done_steps += 1
        if time.perf_counter() - t0 > 120.0:
            break
    dt = time.perf_counter() - t0
    value = done_steps * n_sample * w["T"] / dt
    sample = "envs 0..%d of the workload, T=%d per step, %d steps, single thread" % (
        n_sample - 1, w["T"], done_steps)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": done_steps, "warmup": max(args.warmup, 1), "ms_per_step": dt / done_steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"policy": "f64 cell, f32 encoder and head, int32 env", "cartpole": "f32"}.get(w.get("env"), "int32"),
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def run_policy(args, w, rank, world, local, full=True):
    """The policy-in-the-loop workload: K agent steps per CUDA graph replay; a launch of
    the benchmark is one replay.  full also times the same graph without the env-side
    kernels and without the policy, to report each part's share, and the end-to-end leg.
    The cell kernel alone is timed for the tensor roofline either way."""
    import torch
    import torch.distributed as dist
    from paper_2603_12145_b200 import gru_policy, policy_loop, pong, sharding
    from paper_2603_12145_b200.inputs import policy_weights
    import numpy as np

    N, K = w["n"], w["T"]
    hidden = 576
    steps = args.steps if (args.steps > 0 and full) else DEFAULT_STEPS["policy65k"]
    warmup = max(args.warmup, 3) if full else 3
    env_id_base, _ = sharding.shard(rank, world, N)
    gru_policy.load(build_if_missing=True)
    params = policy_weights(hidden, SEED)
    policy = gru_policy.GruPolicy(params, device="cuda:%d" % local)
    n_params = sum(int(np.asarray(v).size) for v in params.values())
    parts = max(1, args.parts)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_ranks(x):
        return sharding.max_over_ranks(x, device="cuda")

    def timed(with_env, with_policy=True):
        loop = policy_loop.PipelinedPolicyLoop(N, SEED, policy, K, parts=parts, env_id_base=env_id_base,
                                               device="cuda:%d" % local)
        loop.capture(with_env=with_env, with_policy=with_policy)
        for _ in range(warmup):
            loop.replay()
        loop.sync_and_check()
        per_ms, ms_total, w0, w1, blocks = timed_blocks(loop.replay, steps, barrier, max_ranks,
                                                        min_seconds=args.min_seconds)
        loop.sync_and_check()
        # launches made while capturing are replayed: count kernels per replay from what a step launches
        per_replay = parts * (K * ((3 if with_policy else 0) + (2 if with_env else 0)) + (1 if with_env else 0))
        return per_ms, max_ranks(ms_total), w0, w1, loop, len(per_ms) * blocks * steps * per_replay, blocks

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    per_ms, ms_env, w0, w1, loop, launches, blocks = timed(True)
    repeats = len(per_ms)
    replays = repeats * blocks * steps
    clocks = sampler.summary(w0, w1)
    ms_pol = ms_envk = None
    if full:
        p2, ms_pol, _, _, _, _, b2 = timed(False)
        ms_pol /= len(p2) * b2 * steps
        p3, ms_envk, _, _, _, _, b3 = timed(True, with_policy=False)
        ms_envk /= len(p3) * b3 * steps
    # the cell kernel alone, back to back, all N envs per launch, on operands of the loop's kind
    policy._stream()
    gen = torch.Generator(device="cuda:%d" % local).manual_seed(SEED)
    cx = torch.rand((N, hidden), device="cuda:%d" % local, generator=gen).to(torch.bfloat16)
    ch = (torch.rand((N, hidden), device="cuda:%d" % local, generator=gen) * 2 - 1).to(torch.bfloat16)
    cout = torch.empty_like(ch)
    cell_reps = 400 if full else 200
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        gru_policy.gru_policy_cell(policy.h, cx, ch, cout, N)
    e0.record()
    for _ in range(cell_reps):
        gru_policy.gru_policy_cell(policy.h, cx, ch, cout, N)
    e1.record()
    torch.cuda.synchronize()
    cell_ms = e0.elapsed_time(e1) / cell_reps
    policy.status()
    e2e = None
    stats = loop.episode_stats()
    if full:
        # end to end: the step's result (the env's episode statistics) is read back after every replay
        e2e_steps = max(args.e2e_steps, 1)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            loop.replay()
            stats = loop.episode_stats()
        e2e_s = time.perf_counter() - t0
        loop.sync_and_check()
        e2e = {"value": world * e2e_steps * N * K / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 0,
               "d2h_bytes_per_step": 24, "steps": e2e_steps,
               "api": "PolicyLoop.replay + read-back of the env's episode statistics"}
    sampler.stop()
    ms_replay = ms_env / replays
    value = world * N * K / (ms_replay * 1e-3)
    seg = spread([blocks * steps * N * K / (m * 1e-3) for m in per_ms])
    cell_flops = 2.0 * 6 * hidden * hidden * N          # the six H x H products of one agent step
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        peak_tf, peak_kind = float(peaks["bf16_tflops_sustained"]), "measured, sustained"
    except Exception:
        peak_tf, peak_kind = 1400.0, "fallback, sustained"
    achieved_tf = cell_flops / (cell_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": achieved_tf / peak_tf, "peak_source": peak_kind + " cuBLAS bf16",
                "traffic": None, "kernel": w["kernel"], "kernel_ms": cell_ms,
                "flops_per_launch": cell_flops,
                "note": "12 H^2 flops per env: the six H x H products of the GRU cell, timed back "
                        "to back over all N envs"}
    del loop, cx, ch, cout
    policy.close()
    torch.cuda.empty_cache()
    if not full:
        return {"workload_key": "policy65k", "workload": w["name"], "value": value, "unit": UNIT,
                "us_per_launch": ms_replay * 1e3, "agent_step_us": ms_replay / K * 1e3,
                "cell_kernel_us": cell_ms * 1e3, "steps": steps, "repeats": repeats,
                "blocks_per_repeat": blocks, "roofline": roofline, "segments": seg, "clocks": clocks,
                "dtype": "bf16 policy (f32 accumulate), int32 env", "gpu_launches": int(launches)}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_replay, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 policy (f32 accumulate), int32 env", "data": "synthetic",
        "repeats": repeats, "blocks_per_repeat": blocks,
        "config": {"workload": w["name"], "workload_key": args.workload, "n_envs_per_gpu": N,
                   "agent_steps_per_graph": K, "policy_parameters": n_params, "hidden": hidden,
                   "parallel_slices": parts,
                   "env_steps_per_step": N * K,
                   "l2": "the policy's activations (226 MB) and weights are read every step; no flush"},
        "roofline": roofline,
        "agent_step_us": ms_replay / K * 1e3,
        "policy_only_us_per_agent_step": ms_pol / K * 1e3,
        "env_kernels_only_us_per_agent_step": ms_envk / K * 1e3,
        "cell_kernel_us": cell_ms * 1e3,
        "env_kernels_share_of_step": ms_envk / ms_replay,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "segments": seg,
        "episode_stats": dict(zip(("episodes", "sum_return", "sum_length"), (int(v) for v in stats))),
    }
    if rank == 0:
        # CPU: the whole agent step from the oracles (encoder, binary64 cell, head, sampling, env step)
        n_s = 64
        call = policy_oracle_call(n_s, 1, hidden)
        c0, reps = time.perf_counter(), 0
        while time.perf_counter() - c0 < max(args.cpu_seconds, 0.2):
            call()
            reps += 1
        cpu_dt = time.perf_counter() - c0
        line["cpu_baseline"] = {"value": reps * n_s / cpu_dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "host_cores": os.cpu_count(),
                                "sample": "whole agent step (encoder, binary64 cell, head, sampling, env step) "
                                          "of envs 0..%d, %d steps, %.1f s, single thread" % (n_s - 1, reps, cpu_dt)}
    return line


def timed_blocks(launch, steps, barrier, max_over_ranks, min_seconds=0.25, min_repeats=5):
    """Times blocks of `steps` launches, back to back, with CUDA events on the launching
    stream: one untimed block sizes the run, then min_repeats repeats are timed, each made
    of as many whole blocks as it takes for the repeats to add up to min_seconds of device
    time (the paper's protocol: warm-up excluded, mean and spread over N >= 5 runs).  Events
    sit between repeats only, so the launches inside a repeat run back to back whatever
    `steps` is.  Returns the per-repeat times in ms, the total in ms, the wall-clock bracket
    of the timed region and the number of blocks per repeat."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        launch()
    e1.record()
    torch.cuda.synchronize()
    probe_ms = max(max_over_ranks(e0.elapsed_time(e1)), 1e-3)
    blocks = int(max(1, -(-(min_seconds * 1e3 / min_repeats) // probe_ms)))
    barrier()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(min_repeats + 1)]
    w0 = time.perf_counter()
    marks[0].record()
    for r in range(min_repeats):
        for _ in range(blocks * steps):
            launch()
        marks[r + 1].record()
    torch.cuda.synchronize()
    w1 = time.perf_counter()
    barrier()
    per = [marks[r].elapsed_time(marks[r + 1]) for r in range(min_repeats)]
    return per, marks[0].elapsed_time(marks[-1]), w0, w1, blocks


def spread(values):
    mean = sum(values) / len(values)
    std = (sum((x - mean) ** 2 for x in values) / len(values)) ** 0.5
    return {"n": len(values), "mean": mean, "std": std, "cv": std / mean if mean else 0.0}


DEFAULT_STEPS = {"rollout65k": 200, "rollout1m": 50, "pixels16k": 10, "step4096": 2000,
                 "cartpole65k": 200, "cartpole1m": 50, "small64": 20, "policy65k": 4}

def run_env(args, key, rank, world, local, full):
    """One env workload (Pong or CartPole).  full: the run's main workload (adds the
    end-to-end leg and the CUDA-graph figure's detail); otherwise a short record for the
    "configs" list.  Returns the JSON-ready dict on every rank."""
    import torch
    import torch.distributed as dist
    from paper_2603_12145_b200 import pong, sharding
    from paper_2603_12145_b200.inputs import explicit_actions

    w = WORKLOADS[key]
    N, T, mode = w["n"], w["T"], w["mode"]
    pixels = w["obs_mode"] == 1
    env_steps_per_launch = N * T
    warmup = max(args.warmup, 3)
    steps = args.steps if (args.steps > 0 and full) else DEFAULT_STEPS[key]

    env_id_base, _ = sharding.shard(rank, world, N)
    is_cartpole = w.get("env") == "cartpole"
    obs_width = 4 if is_cartpole else 6
    if is_cartpole:
        from paper_2603_12145_b200 import cartpole
        cartpole.load(build_if_missing=True)
        env = cartpole.CartPoleEnv(N, SEED, env_id_base=env_id_base)
        rollout_host = cartpole.cartpole_rollout_host
    else:
        env = pong.PongEnv(N, SEED, obs_mode=w["obs_mode"], frameskip=w["frameskip"],
                           env_id_base=env_id_base)
        rollout_host = pong.pong_rollout_host
    obs = env.ring if pixels else torch.empty((T, N, obs_width), dtype=torch.float32, device="cuda")
    reward = torch.empty((T, N), dtype=torch.float32, device="cuda")
    done = torch.empty((T, N), dtype=torch.uint8, device="cuda")
    acts_np = explicit_actions(T, N, seed=SEED)
    if is_cartpole:
        acts_np = acts_np & 1
    acts_d = torch.from_numpy(acts_np).cuda() if mode == 2 else None
    l2_note = ("each step writes %.0f MB of outputs, larger than the 126 MB L2; no flush"
               % (env_steps_per_launch * w["bytes"] / 1e6))
    flush = None
    if env_steps_per_launch * w["bytes"] < 200e6:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        l2_note = "outputs smaller than L2: a 256 MB buffer is rewritten before the timed region only " \
                  "(launch-latency-bound workload; flushing between launches would time the flush)"

    env._stream()
    if key == "step4096":
        # the C entry point itself, with the buffer addresses taken once: the
        # Python wrapper's per-call work would otherwise dominate a 3 us kernel
        ptrs = (acts_d.data_ptr(), obs.data_ptr(), reward.data_ptr(), done.data_ptr())

        def launch():
            pong.pong_step(env.h, *ptrs)
    else:
        def launch():
            env.rollout(T, mode, acts_d, obs, reward, done)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_ranks(x):
        return sharding.max_over_ranks(x, device="cuda")

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    for _ in range(warmup):
        launch()
    if flush is not None:
        flush.fill_(1)
    barrier()

    # ---- device-resident timing: repeated blocks of `steps` launches, CUDA events on the launching stream
    launches0 = env.launches
    per_ms, ms_total, w0, w1, blocks = timed_blocks(launch, steps, barrier, max_ranks,
                                                    min_seconds=args.min_seconds)
    launches = env.launches - launches0 - steps        # without the untimed sizing block
    repeats = len(per_ms)
    ms_total = max_ranks(ms_total)
    seg = spread([blocks * steps * env_steps_per_launch / (m * 1e-3) for m in per_ms])
    clocks = sampler.summary(w0, w1)
    stats = sharding.sum_stats(env.episode_stats(), device="cuda")

    # ---- single-step API only: the same launches replayed from a CUDA graph, which
    # removes the host's per-launch cost.  Valid for explicit actions on vector obs:
    # the env state lives on the device and the host-side step counter (which does
    # not advance on replay) only keys Philox draws and the pixel ring slot.
    graph_info = None
    if key == "step4096":
        per_graph, replays = 100, 50
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            env._stream()
            launch()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            env._stream()
            for _ in range(per_graph):
                launch()
        env._stream()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(replays):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        g_ms = g0.elapsed_time(g1) / (per_graph * replays)
        graph_info = {"launches_per_graph": per_graph, "replays": replays, "ms_per_step": g_ms,
                      "value": env_steps_per_launch / (g_ms * 1e-3), "unit": UNIT}

    # ---- end to end: host buffers in, host buffers out, through pong_rollout_host
    e2e = None
    if full:
        e2e_steps = max(args.e2e_steps, 1)
        acts_h = torch.from_numpy(acts_np).pin_memory()
        obs_h = (torch.zeros((N, 4, 84, 84), dtype=torch.uint8) if pixels
                 else torch.empty((T, N, obs_width), dtype=torch.float32)).pin_memory()
        rew_h = torch.empty((T, N), dtype=torch.float32).pin_memory()
        done_h = torch.empty((T, N), dtype=torch.uint8).pin_memory()
        env._stream()
        for _ in range(2):
            rollout_host(env.h, T, pong.ACT_EXPLICIT, acts_h, obs_h, rew_h, done_h)
        barrier()
        e0 = time.perf_counter()
        for _ in range(e2e_steps):
            rollout_host(env.h, T, pong.ACT_EXPLICIT, acts_h, obs_h, rew_h, done_h)
        torch.cuda.synchronize()
        e2e_s = max_ranks(time.perf_counter() - e0)
        h2d = acts_h.numel() + (obs_h.numel() if pixels else 0)
        d2h = obs_h.numel() * obs_h.element_size() + rew_h.numel() * 4 + done_h.numel()
        e2e = {"value": world * e2e_steps * env_steps_per_launch / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "api": "pong_rollout_host, pinned host buffers, explicit actions"}
    sampler.stop()
    barrier()

    total_launches = repeats * blocks * steps
    value = world * total_launches * env_steps_per_launch / (ms_total * 1e-3)
    peak, peak_kind = measured_peak()
    kernel_ms = ms_total / total_launches
    achieved = env_steps_per_launch * w["bytes"] / (kernel_ms * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": peak_kind + " copy bandwidth",
        "traffic": w["traffic"],
        "algorithmic_bytes_per_launch": env_steps_per_launch * w["bytes"],
        "bytes_per_env_step": w["bytes"],
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "kernel": w["kernel"], "kernel_ms": kernel_ms,
    }
    if w.get("alu_per_warp_step"):
        # secondary ceiling: what the integer pipe alone would allow.  Rate measured now on this
        # device (register-only add / max / min chains at full occupancy), instruction count per
        # warp-step from the kernel's ncu profile.
        alu_rate = pong.pong_measure_alu_rate(torch.cuda.current_stream().cuda_stream)
        ceiling = alu_rate / w["alu_per_warp_step"] * 32.0
        roofline["secondary"] = {
            "bound": "alu", "unit": UNIT, "ceiling": ceiling, "frac": value / world / ceiling,
            "alu_warp_instr_per_s": alu_rate, "alu_instr_per_warp_step": w["alu_per_warp_step"],
            "note": "integer-ALU rate measured live (pong_measure_alu_rate) / ALU instructions per "
                    "warp-step from the ncu profile of this kernel x 32 envs per warp"}
    episode_stats = ({"episodes": stats[0], "sum_length": stats[1]} if is_cartpole else
                     {"episodes": stats[0], "sum_return": stats[1], "sum_length": stats[2]})
    env.close()
    del obs, reward, done, flush
    torch.cuda.empty_cache()
    if not full:
        rec = {"workload_key": key, "workload": w["name"], "value": value, "unit": UNIT,
               "us_per_launch": kernel_ms * 1e3, "steps": steps, "repeats": repeats,
               "blocks_per_repeat": blocks, "bytes_per_env_step": w["bytes"], "achieved_gbs": achieved,
               "frac_of_measured": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
               "kernel": w["kernel"], "segments": seg, "clocks": clocks,
               "dtype": "f32" if is_cartpole else "int32", "gpu_launches": int(launches)}
        if "secondary" in roofline:
            rec["secondary"] = roofline["secondary"]
        if graph_info is not None:
            rec["cuda_graph"] = graph_info
        return rec
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": kernel_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32" if is_cartpole else "int32",
        "data": "synthetic", "repeats": repeats, "blocks_per_repeat": blocks,
        "config": {
            "workload": w["name"], "workload_key": key, "n_envs_per_gpu": N, "T": T,
            "frameskip": w["frameskip"], "seed": SEED, "env_steps_per_step": env_steps_per_launch,
            "l2": l2_note,
            "timing": "%d repeats of %d blocks of %d launches each, back to back, CUDA events between "
                      "repeats; value from the whole timed region, segments = per-repeat rates"
                      % (repeats, blocks, steps),
            "parallelism": "env shards per GPU, no collective" if world > 1 else "single GPU",
        },
        "roofline": roofline,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "segments": seg,
        "episode_stats": episode_stats,
    }
    if graph_info is not None:
        line["cuda_graph"] = graph_info
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0,
                    help="launches per block (default: per workload); five repeats of as many blocks "
                         "as it takes to time --min-seconds of work")
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="rollout65k", choices=sorted(WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--min-seconds", type=float, default=0.25)
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the short records of the other configurations")
    ap.add_argument("--parts", type=int, default=1,
                    help="policy65k: independent env slices run as parallel chains of one graph")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2603_12145_b200 import pong

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if world != args.gpus:
        raise SystemExit("--gpus %d needs torchrun with %d ranks (WORLD_SIZE=%d)" % (
            args.gpus, args.gpus, world))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pong.load(build_if_missing=True)

    w = WORKLOADS[args.workload]
    if w.get("env") == "policy":
        line = run_policy(args, w, rank, world, local, full=True)
    else:
        line = run_env(args, args.workload, rank, world, local, full=True)
    # the other configurations, one short record each (single GPU, default workload only)
    if world == 1 and args.workload == "rollout65k" and not args.no_configs:
        records = []
        for key in ("small64", "step4096", "pixels16k", "rollout1m", "cartpole65k", "cartpole1m",
                    "policy65k"):
            if WORKLOADS[key].get("env") == "policy":
                records.append(run_policy(args, WORKLOADS[key], rank, world, local, full=False))
            else:
                records.append(run_env(args, key, rank, world, local, full=False))
        line["configs"] = records
    if rank == 0:
        if world == 1 and w.get("env") != "policy":
            rate, reps, dt, n_sample = cpu_oracle_rate(w, args.cpu_seconds)
            line["cpu_baseline"] = {
                "value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
                "host_cores": os.cpu_count(),
                "sample": "envs 0..%d of the workload, T=%d per call, %d calls, %.1f s, "
                          "single thread" % (n_sample - 1, w["T"], reps, dt)}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
