"""Achieved memory bandwidth of the streaming kernels (GAE scan + normalisation, minibatch gather,
gradient reduction, Adam) at sizes where bandwidth, not launch latency, decides their time.

    python -m paper_2509_10771_b200.bandwidth_report [--envs 1048576] [--steps 32]

Two parts, one JSON object on stdout:
  * the stand-alone GAE scan (rslrl_gae_scan) on T x N synthetic transitions, timed with CUDA
    events over repeated calls; algorithmic bytes = 26 per transition (10 read + 8 written by the
    scan, 4 read + 4 written by the normalisation);
  * one learn iteration of the rough_terrain_symmetry workload (65,536 envs x 32 steps) with the
    library's per-launch event timing: gather, grad_reduce and adam with their algorithmic bytes.
Peak = the measured copy bandwidth in MEASURED_PEAKS.json beside the repository root if present.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np


def main():
    import torch
    from . import binding, build, workloads as WL

    ap = argparse.ArgumentParser()
    ap.add_argument("--envs", type=int, default=1 << 20)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--repeats", type=int, default=20)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    build.build()
    dev = torch.device("cuda", 0)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    peak = None
    try:
        peak = json.load(open(os.path.join(root, "MEASURED_PEAKS.json")))["hbm_gbs"]
    except Exception:
        pass
    out = {"peak_gbs": peak}

    # ---- stand-alone scan ------------------------------------------------------------------
    T, N = args.steps, args.envs
    g = torch.Generator(device="cpu").manual_seed(0)
    rew = torch.randn((T, N), generator=g).to(dev)
    val = torch.randn((T, N), generator=g).to(dev)
    done = (torch.rand((T, N), generator=g) < 0.005).to(torch.uint8).to(dev)
    tout = (done * (torch.rand((T, N), generator=g) < 0.5).to(torch.uint8).to(dev))
    last = torch.randn((N,), generator=g).to(dev)
    ret = torch.empty((T, N), device=dev)
    adv = torch.empty((T, N), device=dev)
    scratch = torch.empty(binding.gae_scratch_bytes(T, N), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def timed_scan(normalize):
        def scan():
            binding.gae_scan(rew, val, done, tout, last, ret, adv, T, N, 0.99, 0.95, normalize, True, 1e-8, scratch,
                             stream.cuda_stream)
        for _ in range(3):
            scan()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.repeats):
            scan()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.repeats

    ms_scan = timed_scan(False)
    ms = timed_scan(True)
    gbs = 26.0 * T * N / (ms * 1e-3) / 1e9
    out["gae_scan"] = {"T": T, "N": N, "ms": ms, "algorithmic_bytes": 26 * T * N, "gbs": gbs,
                       "frac_of_peak": gbs / peak if peak else None,
                       "scan_only_ms": ms_scan, "scan_only_gbs": 18.0 * T * N / (ms_scan * 1e-3) / 1e9,
                       "normalize_only_gbs": 8.0 * T * N / (max(ms - ms_scan, 1e-6) * 1e-3) / 1e9,
                       "note": "working set %.0f MB: larger than the 126 MB L2" % (26.0 * T * N / 1e6)}

    # ---- kernels of one update at the largest workload -----------------------------------------
    del rew, val, done, tout, last, ret, adv
    w = WL.ROUGH_SYM
    mir = WL.make_mirror(w)
    ctx = binding.Context(w, precision=WL.PRECISION_BF16, stream=stream.cuda_stream, mirror=mir)
    ctx.set_params(WL.make_params(w))
    inputs = WL.make_rollout_inputs(w)
    d_obs = torch.from_numpy(inputs["obs_actor"]).to(dev)
    d_rew = torch.from_numpy(inputs["rewards"]).to(dev)
    d_done = torch.from_numpy(inputs["dones"]).to(dev)
    d_to = torch.from_numpy(inputs["timeouts"]).to(dev)

    def iteration():
        for t in range(w.num_steps):
            ctx.act(d_obs[t])
            ctx.record_step(d_rew[t], d_done[t], d_to[t])
        ctx.gae(d_obs[w.num_steps])
        ctx.ppo_update(want_stats=False)

    iteration()
    torch.cuda.synchronize()
    binding.profile_enable(True)
    binding.profile_report()
    iteration()
    torch.cuda.synchronize()
    prof = binding.profile_report()
    binding.profile_enable(False)
    steps = w.epochs * w.minibatches
    Bmb = w.minibatch_rows
    A4 = (w.num_actions + 3) // 4 * 4
    kp = (w.actor_obs_dim + 63) // 64 * 64
    P = int(binding.load_library().rslrl_num_params(binding.model_cfg(w)))
    # per minibatch row: FP32 observation row, actions, old mean, four scalars read; two BF16 observation rows
    # (original + mirrored), two action rows, old mean, old sigma, four scalars written
    gather_bytes = Bmb * (4 * w.actor_obs_dim + 4 * 2 * A4 + 16) + Bmb * (2 * 2 * kp + 4 * 4 * A4 + 16)
    fams = {
        "gather": gather_bytes,
        "adam": 28 * P,                                            # 16 B read + 12 B written per parameter
        "gae_scan": 18 * w.num_steps * w.num_envs,
        "gae_normalize": 8 * w.num_steps * w.num_envs,
    }
    rows = {}
    for name, nbytes in fams.items():
        if name not in prof:
            continue
        ms_k = prof[name]["ms"] / prof[name]["launches"]
        gb = nbytes / (ms_k * 1e-3) / 1e9
        rows[name] = {"launches": prof[name]["launches"], "ms_per_launch": ms_k, "algorithmic_bytes": nbytes, "gbs": gb,
                      "frac_of_peak": gb / peak if peak else None}
    out["rough_terrain_symmetry"] = rows
    ctx.destroy()
    print(json.dumps(out))


if __name__ == "__main__":
    main()
