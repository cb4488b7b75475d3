#!/usr/bin/env python
"""Benchmark of the PPO learn-iteration hot path (rollout inference + GAE + PPO update).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one whole learn iteration over one rollout of synthetic data:
T x (rslrl_act + rslrl_record_step), rslrl_gae, rslrl_ppo_update (E x M minibatch steps).
The metric is transitions/s = T * N_envs * K / time.  Rank 0 prints ONE JSON line.

  value   inputs already resident in device memory when the timed region starts
  e2e     the same iteration through the host-buffer entry points (pinned host memory,
          host<->device copies inside the timed region)
  roofline  the kernel family with the largest share of device time, from a separate pass of
          the same K steps with one CUDA event pair per launch
  cpu_baseline  the FP64 oracle, as it stands, on the host cores, on a bounded sample

With --gpus N > 1 every rank runs an independent replica of the workload on its own GPU: the path
has no inter-GPU exchange ("replicas only").  Started plainly (no WORLD_SIZE in the environment) the
script launches its N ranks itself through torch.distributed.run on 127.0.0.1.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_10771_b200 import workloads as WL  # noqa: E402

METRIC = "PPO learn-iteration transitions/s"
UNIT = "transitions/s"
WORKLOAD = WL.ROUGH                       # rough-terrain locomotion shape: the config the metric is quoted on
                                          # (--workload selects another of the five)
PRECISION = WL.PRECISION_BF16
ORACLE_SAMPLE_ENVS = 512                  # bounded sample for the CPU baseline: 512 of the 4096 environments


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------
# algorithmic work per learn iteration (real layer widths, no padding)
# ------------------------------------------------------------------------------------------
def hidden_flops_per_row(w, net):
    return sum(2 * i * o for i, o in w.layer_dims(net)[:-1])


def family_flops(w):
    """FLOPs of one learn iteration attributed to the tensor-core kernel families."""
    T, N = w.num_steps, w.num_envs
    steps = w.epochs * w.minibatches
    R = w.minibatch_rows * (2 if w.sym_enable else 1)
    fa, fc = hidden_flops_per_row(w, "actor"), hidden_flops_per_row(w, "critic")
    ha, hc = (2 * i * o for i, o in (w.layer_dims("actor")[-1], w.layer_dims("critic")[-1]))
    rollout = T * N * (fa + fc + ha + hc) + N * (fc + hc)        # fused forward + heads of act and of the last value
    fwd = steps * R * (fa + fc)
    dgrad = steps * R * sum(2 * i * o for net in ("actor", "critic") for i, o in w.layer_dims(net)[1:-1])
    wgrad = steps * R * sum(2 * i * o for net in ("actor", "critic") for i, o in w.layer_dims(net))
    return {"tc_mlp_fwd": rollout, "tc_gemm_fwd": fwd, "tc_gemm_dgrad": dgrad, "tc_gemm_wgrad": wgrad}


def hbm_family_bytes(w, storage_strides):
    """Algorithmic bytes per launch of the bandwidth-shaped kernels (what must be read plus what must be written)."""
    sa, sc, as_ = storage_strides
    T, N = w.num_steps, w.num_envs
    Bmb = w.minibatch_rows
    R = Bmb * (2 if w.sym_enable else 1)
    kp_a = -(-w.actor_obs_dim // 64) * 64
    kp_c = -(-w.critic_obs_dim // 64) * 64
    obs_read = 4 * w.actor_obs_dim + (0 if w.shared_obs else 4 * w.critic_obs_dim)
    if PRECISION == WL.PRECISION_BF16:
        obs_written = 2 * kp_a + (0 if w.shared_obs else 2 * kp_c)                # BF16 operand rows
    else:
        obs_written = 4 * sa + (0 if w.shared_obs else 4 * sc)                    # FP32 rows
    gather = Bmb * (4 + obs_read + 4 * 2 * w.num_actions + 4 * 4) \
        + R * (obs_written + 4 * as_) + Bmb * (2 * 4 * as_ + 4 * 4)
    P = w.num_params()
    return {"gather": gather, "gather_alone": gather, "adam": 28 * P, "gae_scan": 18 * T * N, "gae_normalize": 8 * T * N}


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, mean over the family's launches of one
# minibatch step) from the ncu capture summarised under profiles/, valid while the source of the kernels is the
# text that capture ran (recognised by the SHA-256 of the definitions of the three GEMM kernels); otherwise null.
NCU_TRAFFIC = {
    "source": "paper_2509_10771_b200/csrc/umma.cu",
    "begin": "// Weight gradient: D[features_in x features_out] = A^T B over the minibatch rows",
    "end": "// ------------------------------------------------------------------ fused forward chain",
    "sha256": "a7723f3fdc1eccda4f952e97d414ee14fdccc3c233978e074cd2a300bc7fdaeb",
    "bytes_per_launch": {"tc_gemm_fwd": 31.6e6, "tc_gemm_dgrad": 67.8e6, "tc_gemm_wgrad": 203.4e6},
}


def ncu_traffic(family):
    import hashlib
    try:
        src = open(os.path.join(ROOT, NCU_TRAFFIC["source"])).read()
        text = src[src.index(NCU_TRAFFIC["begin"]):src.index(NCU_TRAFFIC["end"])]
    except (OSError, ValueError):
        return None
    if hashlib.sha256(text.encode()).hexdigest() != NCU_TRAFFIC["sha256"]:
        return None
    return NCU_TRAFFIC["bytes_per_launch"].get(family)


def iteration_flops(w):
    T, N = w.num_steps, w.num_envs
    steps = w.epochs * w.minibatches
    R = w.minibatch_rows * (2 if w.sym_enable else 1)
    full = sum(2 * i * o for net in ("actor", "critic") for i, o in w.layer_dims(net))
    first = sum(2 * i * o for net in ("actor", "critic") for i, o in w.layer_dims(net)[:1])
    return T * N * full + steps * R * (3 * full - first)


# ------------------------------------------------------------------------------------------
# the oracle arm (CPU baseline and --impl reference)
# ------------------------------------------------------------------------------------------
def oracle_iteration_seconds(w, repeats=1):
    from oracle import ppo_oracle as O
    dims = (w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)
    theta = WL.make_params(w).astype(np.float64)
    inputs = WL.make_rollout_inputs(w)
    mir = WL.make_mirror(w) if w.sym_enable else None
    state = O.OptimState(theta, w.lr)
    times = []
    for it in range(repeats):
        t0 = time.perf_counter()
        storage = O.rollout(state.theta, dims, inputs, w, seed=w.seed, first_global_step=it * w.num_steps)
        O.ppo_update(state, dims, storage, w, seed=w.seed, iteration=it, sym=mir)
        times.append(time.perf_counter() - t0)
    return times


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args, rank):
    if rank != 0:
        return
    # every step is one whole learn iteration on a sample of the environments; the sample shrinks with the
    # number of steps asked for so that the run stays within about two minutes (about 8 ms per environment)
    n_iter = args.warmup + args.steps
    envs = ORACLE_SAMPLE_ENVS
    while envs > 64 and n_iter * envs * 0.008 > 120.0:
        envs //= 2
    w = WORKLOAD.scaled(min(envs, WORKLOAD.num_envs))
    envs = w.num_envs
    times = oracle_iteration_seconds(w, repeats=n_iter)[args.warmup:]
    total = sum(times)
    value = w.batch * len(times) / total
    sample = (f"{envs} of the {WORKLOAD.num_envs} environments of {WORKLOAD.name}, whole learn "
              f"iterations (T={w.num_steps}, E={w.epochs}, M={w.minibatches}), numpy float64")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.proc = None
        self.idx = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.idx)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------
# replicas: every rank times its own copy of the workload; the job's time is the slowest rank's
# ------------------------------------------------------------------------------------------
def max_over_ranks(values, world, device):
    """Element-wise maximum of `values` over the ranks of the default process group (identity for one rank)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(transitions_per_rank, world, ms):
    """Transitions per second of the whole job: every rank processed transitions_per_rank in ms (the slowest's)."""
    return transitions_per_rank * world / (ms * 1e-3)


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2509_10771_b200 import binding, build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    w = WORKLOAD
    T, N, A = w.num_steps, w.num_envs, w.num_actions
    inputs = WL.make_rollout_inputs(w, seed=rank)          # every replica draws its own rollout
    theta = WL.make_params(w, seed=rank)
    mirror = WL.make_mirror(w, seed=rank) if w.sym_enable else None
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()
    ctx = binding.Context(w, precision=PRECISION, stream=stream.cuda_stream, mirror=mirror)
    ctx.set_params(theta)
    view = ctx.storage_view()

    d_obs = torch.from_numpy(inputs["obs_actor"]).to(dev)
    d_obc = None if w.shared_obs else torch.from_numpy(inputs["obs_critic"]).to(dev)
    d_rew = torch.from_numpy(inputs["rewards"]).to(dev)
    d_done = torch.from_numpy(inputs["dones"]).to(dev)
    d_to = torch.from_numpy(inputs["timeouts"]).to(dev)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # 2x the 126 MB L2

    # device addresses of every step's rows, taken once: the timed loop passes plain pointers, as a simulator would
    p_obs = [d_obs[t].data_ptr() for t in range(T + 1)]
    p_obc = None if d_obc is None else [d_obc[t].data_ptr() for t in range(T + 1)]
    p_rew, p_done, p_to = ([x[t].data_ptr() for t in range(T)] for x in (d_rew, d_done, d_to))

    def iteration_device():
        for t in range(T):
            ctx.act(p_obs[t], None if p_obc is None else p_obc[t])
            ctx.record_step(p_rew[t], p_done[t], p_to[t])
        ctx.gae(p_obs[T] if p_obc is None else p_obc[T])
        ctx.ppo_update(want_stats=False)

    h_obs = torch.from_numpy(inputs["obs_actor"]).pin_memory()
    h_obc = None if w.shared_obs else torch.from_numpy(inputs["obs_critic"]).pin_memory()
    h_rew = torch.from_numpy(inputs["rewards"]).pin_memory()
    h_done = torch.from_numpy(inputs["dones"]).pin_memory()
    h_to = torch.from_numpy(inputs["timeouts"]).pin_memory()
    h_act = torch.empty((N, A), dtype=torch.float32).pin_memory()
    np_obs, np_rew, np_done, np_to, np_act = (x.numpy() for x in (h_obs, h_rew, h_done, h_to, h_act))
    np_obc = None if h_obc is None else h_obc.numpy()

    def iteration_host():
        for t in range(T):
            ctx.act_host(np_obs[t], None if np_obc is None else np_obc[t], np_act)   # H2D obs, D2H actions (waits for them)
            ctx.record_step_host(np_rew[t], np_done[t], np_to[t])
        ctx.gae_host(np_obs[T] if np_obc is None else np_obc[T])
        return ctx.ppo_update(want_stats=True)             # D2H of the update's scalars

    obs_bytes = N * w.actor_obs_dim * 4 + (0 if w.shared_obs else N * w.critic_obs_dim * 4)
    h2d = T * (obs_bytes + N * 4 + 2 * N) + N * w.critic_obs_dim * 4
    d2h = T * N * A * 4 + w.epochs * w.minibatches * 8 * 4

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps):
        """Sum of per-step device times (CUDA events on the launching stream); L2 flushed between steps."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in evs:
            flush_buf.zero_()
            a.record(stream)
            fn()
            b.record(stream)
        barrier()
        return sum(a.elapsed_time(b) for a, b in evs)      # ms

    def timed_one_interval(fn, steps):
        """The same K steps as ONE event interval (back to back, no flush in between: one iteration's working
        set, storage plus activations, is itself larger than the L2)."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        flush_buf.zero_()
        a.record(stream)
        for _ in range(steps):
            fn()
        b.record(stream)
        barrier()
        return a.elapsed_time(b)

    for _ in range(max(args.warmup, 3)):
        iteration_device()
    torch.cuda.synchronize()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)                          # runs across all timed passes below
    launches0 = binding.kernel_launch_count()
    sampler.start()
    ms_total = timed(iteration_device, args.steps)
    launches = binding.kernel_launch_count() - launches0
    ms_interval = timed_one_interval(iteration_device, args.steps)

    iteration_host()
    ms_e2e = timed(iteration_host, args.steps)

    # per-kernel pass: the same K steps with one event pair per launch
    binding.profile_enable(True)
    binding.profile_report()
    for _ in range(args.steps):
        flush_buf.zero_()
        iteration_device()
    torch.cuda.synchronize()
    prof = binding.profile_report()
    binding.profile_enable(False)
    clocks = sampler.stop()

    ms_total, ms_e2e, ms_interval = max_over_ranks([ms_total, ms_e2e, ms_interval], world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = read_peaks()
    value = whole_job_value(T * N * args.steps, world, ms_total)
    e2e_value = whole_job_value(T * N * args.steps, world, ms_e2e)

    total_prof_ms = sum(v["ms"] for v in prof.values()) or 1.0
    shares = {k: {"launches": v["launches"], "ms": round(v["ms"], 3), "share": round(v["ms"] / total_prof_ms, 4)}
              for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])}
    fam_flops = family_flops(w)
    tc = {k: v for k, v in prof.items() if k in fam_flops}
    top = max(tc, key=lambda k: tc[k]["ms"])
    achieved = fam_flops[top] * args.steps / (tc[top]["ms"] * 1e-3) / 1e12
    # the launches of the per-kernel pass are timed one by one (tens of microseconds each, clocks at their maximum,
    # no power cap): the burst peak is their denominator; the sustained one is printed beside it
    peak, peak_sus = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    tf32 = PRECISION == WL.PRECISION_TF32
    if tf32:
        # no TF32 peak has been measured on this machine: the BF16 figures times the nominal ratio of the two dense
        # peaks (1.1 / 2.25 PFLOP/s); the weight gradients of this mode run on the FP32 pipes and are no tensor family
        peak, peak_sus = peak * 1.1 / 2.25, peak_sus * 1.1 / 2.25
        tc = {k: v for k, v in tc.items() if k in ("tc_gemm_fwd", "tc_gemm_dgrad")}
        top = max(tc, key=lambda k: tc[k]["ms"])
        achieved = fam_flops[top] * args.steps / (tc[top]["ms"] * 1e-3) / 1e12

    def fam(k):
        tf = fam_flops[k] * args.steps / (tc[k]["ms"] * 1e-3) / 1e12
        return {"tflops": tf, "frac": tf / peak, "frac_of_sustained": tf / peak_sus,
                "avg_launch_us": 1e3 * tc[k]["ms"] / tc[k]["launches"]}

    roofline = {"bound": "tensor", "kernel": top, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "frac_of_sustained": achieved / peak_sus,
                "frac_of_nominal": achieved / (1100.0 if tf32 else 2250.0),
                "traffic": None if tf32 else ncu_traffic(top), "traffic_unit": "bytes per launch (ncu, dram read + write)",
                "peak_source": (f"bf16 burst (launches timed alone), {peaks['source']}; sustained {peak_sus}" if not tf32 else
                                f"bf16 burst, {peaks['source']}, x 1.1 / 2.25 (nominal tf32 / bf16 ratio); no tf32 peak measured"),
                "avg_launch_us": 1e3 * tc[top]["ms"] / tc[top]["launches"],
                "families": {k: fam(k) for k in tc},
                "timing": "separate pass over the same K steps with one CUDA event pair per launch; the forward and the "
                          "data-gradient launches of a minibatch step (one per layer, chained by programmatic dependent "
                          "launch) share one pair per step, divided by their number"}
    # bandwidth-shaped kernels of the same pass: algorithmic bytes per launch / mean launch time
    hbm_bytes = hbm_family_bytes(w, (view.obs_a_stride, view.obs_c_stride, view.act_stride))
    hbm = {}
    for k, nbytes in hbm_bytes.items():
        if k in prof and prof[k]["launches"]:
            us = 1e3 * prof[k]["ms"] / prof[k]["launches"]
            gbs = nbytes / (us * 1e-6) / 1e9
            hbm[k] = {"bytes_per_launch": nbytes, "avg_launch_us": us, "gbs": gbs, "frac": gbs / peaks["hbm_gbs"],
                      "frac_of_nominal_7700": gbs / 7700.0}
    roofline["hbm_families"] = hbm
    roofline["hbm_peak_gbs"] = peaks["hbm_gbs"]

    ws = WORKLOAD.scaled(min(ORACLE_SAMPLE_ENVS, WORKLOAD.num_envs))
    oracle_iteration_seconds(WORKLOAD.scaled(32), repeats=1)            # warms numpy / BLAS threads once (not timed)
    o_times = oracle_iteration_seconds(ws, repeats=1)
    sample = (f"one whole learn iteration on {ws.num_envs} of the {w.num_envs} environments of {w.name} "
              f"(T={w.num_steps}, E={w.epochs}, M={w.minibatches}), numpy float64, after one untimed warm-up "
              f"iteration on 32 environments")
    cpu = {"value": ws.batch / o_times[0], "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "tf32" if tf32 else "bf16", "data": "synthetic",
        "config": {"workload": w.name, "num_envs": N, "num_steps": T, "obs_dim": w.actor_obs_dim, "actions": A,
                   "epochs": w.epochs, "minibatches": w.minibatches, "symmetry": bool(w.sym_enable),
                   "precision": ("tf32" if tf32 else "bf16") + " operands, fp32 accumulate", "l2": "256 MiB buffer written between timed steps",
                   "parallelism": "replicas only" if world > 1 else "1 gpu"},
        "clocks": clocks,
        "one_interval": {"ms_per_step": ms_interval / args.steps,
                         "value": whole_job_value(T * N * args.steps, world, ms_interval),
                         "note": "the same K steps as one CUDA event interval, back to back, no L2 flush in between"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "iteration_tflops": iteration_flops(w) * args.steps * world / (ms_total * 1e-3) / 1e12,
        "kernel_shares": shares,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    ctx.destroy()
    if world > 1:
        dist.destroy_process_group()


def run_distill(args):
    """--task distill: the distillation iteration (T x (act + record_step) with the student, then
    rslrl_distill_update on stand-in expert actions) on the same workload, one GPU.  Prints its own JSON line:
    device-timed transitions/s, per-kernel shares, and the oracle's distillation update timed on a sample."""
    import torch
    from paper_2509_10771_b200 import binding, build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    w = WORKLOAD
    T, N = w.num_steps, w.num_envs
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    inputs = WL.make_rollout_inputs(w)
    ctx = binding.Context(w, precision=PRECISION, stream=stream.cuda_stream)
    ctx.set_params(WL.make_params(w))
    d_obs = torch.from_numpy(inputs["obs_actor"]).to(dev)
    d_rew = torch.from_numpy(inputs["rewards"]).to(dev)
    d_done = torch.from_numpy(inputs["dones"]).to(dev)
    d_to = torch.from_numpy(inputs["timeouts"]).to(dev)
    stride = ctx.storage_view().act_stride
    expert = np.zeros((T, N, stride), dtype=np.float32)
    expert[..., :w.num_actions] = WL.make_expert_actions(w)
    d_expert = torch.from_numpy(expert).to(dev)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def iteration():
        for t in range(T):
            ctx.act(d_obs[t])
            ctx.record_step(d_rew[t], d_done[t], d_to[t])
        ctx.distill_update(d_expert, want_stats=False)

    for _ in range(max(args.warmup, 3)):
        iteration()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in evs:
        flush_buf.zero_()
        a.record(stream)
        iteration()
        b.record(stream)
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in evs)
    binding.profile_enable(True)
    binding.profile_report()
    for _ in range(args.steps):
        iteration()
    torch.cuda.synchronize()
    prof = binding.profile_report()
    binding.profile_enable(False)
    total = sum(v["ms"] for v in prof.values()) or 1.0
    shares = {k: {"launches": v["launches"], "ms": round(v["ms"], 3), "share": round(v["ms"] / total, 4)}
              for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])}
    # the oracle's distillation update on a sample of the environments
    from oracle import ppo_oracle as O
    ws = WORKLOAD.scaled(ORACLE_SAMPLE_ENVS)
    dims = (ws.layer_dims("actor"), ws.layer_dims("critic"), ws.num_actions)
    state = O.OptimState(WL.make_params(ws).astype(np.float64), ws.lr)
    t0 = time.perf_counter()
    O.distill_update(state, dims, WL.make_rollout_inputs(ws)["obs_actor"], WL.make_expert_actions(ws), ws, seed=ws.seed, iteration=0)
    cpu_s = time.perf_counter() - t0
    line = {
        "metric": "distillation iteration transitions/s", "value": T * N * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "task": "distill", "num_envs": N, "num_steps": T, "epochs": w.epochs,
                   "minibatches": w.minibatches, "l2": "256 MiB buffer written between timed steps"},
        "kernel_shares": shares,
        "cpu_baseline": {"value": ws.batch / cpu_s, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": f"the oracle's distillation update on {ORACLE_SAMPLE_ENVS} of the {N} environments (rollout not included)"},
    }
    print(json.dumps(line), flush=True)
    ctx.destroy()


def run_rnd(args):
    """--task rnd: random network distillation on a state subset over one rollout's transitions, one GPU: the
    intrinsic reward of all T x N rows (rslrl_rnd_reward) followed by the predictor's training loop
    (rslrl_rnd_update, the workload's epochs x minibatches).  Prints its own JSON line."""
    import torch
    from paper_2509_10771_b200 import binding, build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    w = WORKLOAD
    T, N = w.num_steps, w.num_envs
    B = T * N
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    setup = WL.make_rnd_setup(w, num_idx=48, hidden=(256, 128, 64), embed_dim=32)
    obs = WL.make_rollout_inputs(w)["obs_actor"][:T].reshape(B, w.actor_obs_dim)
    d_obs = torch.from_numpy(obs).to(dev)
    d_rew = torch.zeros(B, device=dev)
    rnd = binding.Rnd(w.actor_obs_dim, setup["idx"], setup["hidden"], setup["embed_dim"], max_rows=B, lr=1e-3,
                      stream=stream.cuda_stream, max_batch=B, max_epochs=w.epochs, max_minibatches=w.minibatches,
                      precision=WL.PRECISION_TF32 if PRECISION == WL.PRECISION_TF32 else WL.PRECISION_FP32)
    rnd.set_params(setup["predictor"], setup["target"])
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    it = [0]

    def iteration():
        rnd.reward(d_obs, B, w.actor_obs_dim, weight=0.1, d_rewards_inout=d_rew)
        rnd.update(d_obs, B, w.actor_obs_dim, w.epochs, w.minibatches, seed=w.seed, iteration=it[0], want_loss=False)
        it[0] += 1

    for _ in range(max(args.warmup, 3)):
        iteration()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in evs:
        flush_buf.zero_()
        a.record(stream)
        iteration()
        b.record(stream)
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in evs)
    binding.profile_enable(True)
    binding.profile_report()
    for _ in range(min(args.steps, 10)):
        iteration()
    torch.cuda.synchronize()
    prof = binding.profile_report()
    binding.profile_enable(False)
    total = sum(v["ms"] for v in prof.values()) or 1.0
    shares = {k: {"launches": v["launches"], "ms": round(v["ms"], 3), "share": round(v["ms"] / total, 4)}
              for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])}
    # FP32 multiply-adds of one iteration: both nets forward on B rows for the reward, the target once more on B rows
    # for the update, then per training row the predictor's forward and its two backward products
    mac = sum(fi * fo for fi, fo in setup["dims"])
    flops = 2.0 * mac * (2 * B + B + w.epochs * B * 3)
    from types import SimpleNamespace
    from oracle import ppo_oracle as O
    rows_s = ORACLE_SAMPLE_ENVS * T
    hp = SimpleNamespace(epochs=w.epochs, minibatches=w.minibatches, elu_alpha=1.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8)
    state = O.OptimState(setup["predictor"].astype(np.float64), 1e-3)
    t0 = time.perf_counter()
    O.rnd_reward(state.theta, setup["target"], setup["dims"], obs[:rows_s], setup["idx"], 1.0)
    O.rnd_update(state, setup["target"], setup["dims"], obs[:rows_s], setup["idx"], hp, seed=w.seed, iteration=0)
    cpu_s = time.perf_counter() - t0
    line = {
        "metric": "random network distillation transitions/s", "value": B * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
        "dtype": "tf32" if PRECISION == WL.PRECISION_TF32 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "task": "rnd", "num_envs": N, "num_steps": T, "epochs": w.epochs,
                   "minibatches": w.minibatches, "num_idx": 48, "hidden": [256, 128, 64], "embed_dim": 32,
                   "l2": "256 MiB buffer written between timed steps"},
        ("tf32_tflops" if PRECISION == WL.PRECISION_TF32 else "fp32_tflops"): flops / (ms / args.steps * 1e-3) / 1e12,
        "kernel_shares": shares,
        "cpu_baseline": {"value": rows_s / cpu_s, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": f"the oracle's reward and predictor training on {ORACLE_SAMPLE_ENVS} of the {N} environments"},
    }
    print(json.dumps(line), flush=True)
    rnd.destroy()


def run_gru(args):
    """--task gru: the recurrent memory layer over one rollout (rslrl_gru_forward + rslrl_gru_backward, T steps
    of N environments, hidden width 256, resets at the workload's done rate), one GPU.  Prints its own JSON line."""
    import torch
    from paper_2509_10771_b200 import binding, build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    w = WORKLOAD
    T, N, D, H = w.num_steps, w.num_envs, w.actor_obs_dim, 256
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    inputs = WL.make_rollout_inputs(w)
    setup = WL.make_gru_setup(w, hidden_dim=H)
    stride = (D + 3) // 4 * 4
    xp = np.zeros((T, N, stride), dtype=np.float32)
    xp[..., :D] = inputs["obs_actor"][:T]
    d_x = torch.from_numpy(xp).to(dev)
    d_h0 = torch.from_numpy(setup["h0"]).to(dev)
    d_dn = torch.from_numpy(inputs["dones"]).to(dev)
    d_dh = torch.from_numpy(setup["dh"]).to(dev)
    d_h = torch.empty((T, N, H), device=dev)
    d_dx = torch.empty((T, N, stride), device=dev)
    d_dh0 = torch.empty((N, H), device=dev)
    tf32 = PRECISION == WL.PRECISION_TF32
    gru = binding.Gru(D, H, T, N, stream=stream.cuda_stream, precision=WL.PRECISION_TF32 if tf32 else WL.PRECISION_FP32)
    gru.set_params(setup["params"])
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def iteration():
        gru.forward(d_x, stride, d_h0, d_dn, T, N, d_h)
        gru.backward(d_dh, d_dx, stride, d_dh0)

    for _ in range(max(args.warmup, 3)):
        iteration()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in evs:
        flush_buf.zero_()
        a.record(stream)
        iteration()
        b.record(stream)
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in evs)
    binding.profile_enable(True)
    binding.profile_report()
    for _ in range(min(args.steps, 10)):
        iteration()
    torch.cuda.synchronize()
    prof = binding.profile_report()
    binding.profile_enable(False)
    total = sum(v["ms"] for v in prof.values()) or 1.0
    shares = {k: {"launches": v["launches"], "ms": round(v["ms"], 3), "share": round(v["ms"] / total, 4)}
              for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])}
    # multiply-adds per transition: forward (D + H) 3H, backward twice that (data and weight gradients)
    flops = 2.0 * 3 * (D + H) * 3 * H * T * N
    from oracle import gru_oracle as G
    ns = ORACLE_SAMPLE_ENVS
    p = G.unpack_gru(setup["params"], D, H)
    t0 = time.perf_counter()
    c = G.gru_sequence_forward(p, inputs["obs_actor"][:T, :ns], setup["h0"][:ns], inputs["dones"][:, :ns])
    G.gru_sequence_backward(p, c, setup["dh"][:, :ns])
    cpu_s = time.perf_counter() - t0
    line = {
        "metric": "recurrent layer forward + BPTT transitions/s", "value": T * N * args.steps / (ms * 1e-3), "unit": UNIT,
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
        "higher_is_better": True, "dtype": "tf32" if tf32 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "task": "gru", "num_envs": N, "num_steps": T, "input_dim": D, "hidden_dim": H,
                   "l2": "256 MiB buffer written between timed steps"},
        ("tf32_tflops" if tf32 else "fp32_tflops"): flops / (ms / args.steps * 1e-3) / 1e12,
        "kernel_shares": shares,
        "cpu_baseline": {"value": T * ns / cpu_s, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": f"the oracle's forward and backward pass on {ns} of the {N} environments"},
    }
    print(json.dumps(line), flush=True)
    gru.destroy()


def run_streams(args):
    """--task streams: the scan kernels at a bandwidth-shaped size through the stand-alone entry point (rslrl_gae_scan,
    T = 32 steps x 1,048,576 environments, 872 MB of algorithmic traffic per call), one GPU.  The learn iteration's own
    scan moves 2.6 MB and is bound by launch latency; this line is where the scan meets its memory roofline.  Its own
    JSON line; the gather's and Adam's figures at their own sizes are in the ppo line (roofline.hbm_families).  The line
    also carries Adam and the gradient reduction at 36 M parameters (the FP32 mode's update of two wide nets)."""
    import torch
    from paper_2509_10771_b200 import binding, build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    T, N = 32, 1 << 20
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    g = torch.Generator(device=dev); g.manual_seed(0)
    r = torch.randn((T, N), device=dev, generator=g) * 0.5
    v = torch.randn((T, N), device=dev, generator=g)
    lv = torch.randn((N,), device=dev, generator=g)
    d = (torch.rand((T, N), device=dev, generator=g) < 0.005).to(torch.uint8)
    to = d & (torch.rand((T, N), device=dev, generator=g) < 0.5).to(torch.uint8)
    ret = torch.empty((T, N), device=dev); adv = torch.empty((T, N), device=dev)
    scratch = torch.empty(binding.gae_scratch_bytes(T, N), dtype=torch.uint8, device=dev)
    peaks = read_peaks()
    out = {}
    for name, normalize, nbytes in (("gae_scan+gae_normalize", True, 26 * T * N), ("gae_scan", False, 18 * T * N)):
        for _ in range(max(args.warmup, 3)):
            binding.gae_scan(r, v, d, to, lv, ret, adv, T, N, 0.99, 0.95, normalize, True, 1e-8, scratch, stream=stream.cuda_stream)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        torch.cuda.synchronize()
        for a, b in evs:                    # 872 MB per call: far beyond the L2, no flush needed
            a.record(stream)
            binding.gae_scan(r, v, d, to, lv, ret, adv, T, N, 0.99, 0.95, normalize, True, 1e-8, scratch, stream=stream.cuda_stream)
            b.record(stream)
        torch.cuda.synchronize()
        us = 1e3 * sum(a.elapsed_time(b) for a, b in evs) / args.steps
        gbs = nbytes / (us * 1e-6) / 1e9
        out[name] = {"bytes_per_call": nbytes, "us": us, "gbs": gbs, "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_7700": gbs / 7700.0}
    # Adam (and the gradient reduction in front of it) at a bandwidth-shaped size: the FP32 mode's update of two
    # 64-4096-4096-256 nets (36 M parameters, 1 GB of algorithmic traffic per Adam launch) on a 512-transition rollout;
    # per-launch CUDA events of the library's own accounting
    del r, v, lv, d, to, ret, adv, scratch
    from dataclasses import replace
    w = replace(WL.TINY, name="wide_nets_for_adam", actor_obs_dim=64, critic_obs_dim=64, actor_hidden=(4096, 4096, 256),
                critic_hidden=(4096, 4096, 256), actor_obs_blocks=((64, "normal"),), critic_obs_blocks=((64, "normal"),))
    ctx = binding.Context(w, precision=WL.PRECISION_FP32, stream=stream.cuda_stream)
    ctx.set_params(WL.make_params(w))
    inp = WL.make_rollout_inputs(w)
    d_o = torch.from_numpy(inp["obs_actor"]).to(dev)
    d_r, d_d, d_t = (torch.from_numpy(inp[k]).to(dev) for k in ("rewards", "dones", "timeouts"))

    def wide_iteration():
        for t in range(w.num_steps):
            ctx.act(d_o[t]); ctx.record_step(d_r[t], d_d[t], d_t[t])
        ctx.gae(d_o[w.num_steps])
        ctx.ppo_update(want_stats=False)

    for _ in range(3):
        wide_iteration()
    torch.cuda.synchronize()
    binding.profile_enable(True)
    binding.profile_report()
    for _ in range(max(2, args.steps // 4)):
        wide_iteration()
    torch.cuda.synchronize()
    rep = binding.profile_report()
    binding.profile_enable(False)
    P = ctx.num_params
    for name, per_param in (("adam", 28), ("grad_reduce", 8)):
        if name in rep and rep[name]["launches"]:
            us = 1e3 * rep[name]["ms"] / rep[name]["launches"]
            gbs = per_param * P / (us * 1e-6) / 1e9
            out[name + "_36M_parameters"] = {"bytes_per_call": per_param * P, "us": us, "gbs": gbs, "frac": gbs / peaks["hbm_gbs"],
                                             "frac_of_nominal_7700": gbs / 7700.0}
    ctx.destroy()
    both = out["gae_scan+gae_normalize"]
    line = {
        "metric": "GAE scan + advantage normalisation transitions/s", "value": T * N / (both["us"] * 1e-6), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": both["us"] * 1e-3, "higher_is_better": True,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "gae_scan_T32_N1048576", "task": "streams", "l2": "inputs (872 MB per call) larger than the L2"},
        "roofline": {"bound": "hbm", "achieved": both["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": both["frac"],
                     "traffic": None, "peak_source": f"copy bandwidth, {peaks['source']}", "kernels": out},
    }
    print(json.dumps(line), flush=True)


def free_port():
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def spawn_ranks(n):
    """Started plainly with --gpus N > 1: run this script again as N ranks (one per GPU) under torch.distributed.run."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    global WORKLOAD, PRECISION
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD.name, choices=sorted(WL.WORKLOADS),
                    help="which of the five synthetic workloads to time (default: the one the metric is quoted on)")
    ap.add_argument("--precision", default="bf16", choices=["bf16", "tf32"],
                    help="operand precision of the products on the tensor cores (ppo task, default bf16; gru and rnd tasks: tf32 selects the tensor-core mode, anything else FP32)")
    ap.add_argument("--task", default="ppo", choices=["ppo", "distill", "rnd", "gru", "streams"],
                    help="ppo: the learn iteration the metric is quoted on (default); distill: the distillation iteration; "
                         "rnd: random network distillation over one rollout; gru: the recurrent layer over one rollout; "
                         "streams: the GAE scan at a bandwidth-shaped size")
    ap.add_argument("--envs", type=int, default=0,
                    help="run the workload on this many environments instead of its own number (a size a profiler "
                         "capture can hold; the workload's name in the JSON line then ends in @<envs>)")
    args = ap.parse_args()
    WORKLOAD = WL.WORKLOADS[args.workload]
    if args.envs > 0:
        WORKLOAD = WORKLOAD.scaled(args.envs)
    PRECISION = WL.PRECISION_TF32 if args.precision == "tf32" else WL.PRECISION_BF16
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
    elif args.task == "distill":
        if rank == 0:
            run_distill(args)
    elif args.task == "rnd":
        if rank == 0:
            run_rnd(args)
    elif args.task == "gru":
        if rank == 0:
            run_gru(args)
    elif args.task == "streams":
        if rank == 0:
            run_streams(args)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
