"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI, run the oracle
on the same seeded inputs, compare element by element."""
from __future__ import annotations

from typing import Dict

import numpy as np

from oracle import ppo_oracle as O
from paper_2509_10771_b200 import workloads as WL


def assert_close(got, want, tol: float, name: str = "", max_outlier_frac: float = 0.0, outlier_abs: float = 0.0,
                 outlier_factor: float = 0.0):
    """|got - want| <= tol * |want| + tol * rms(want), element by element.

    ``max_outlier_frac`` > 0 allows that fraction of elements to miss the bound as long as they
    stay within ``outlier_abs`` (used only where an element is a discontinuous function of the
    inputs, e.g. Adam's first step at a gradient entry that is zero to rounding).  With ``outlier_factor``
    the allowed outliers must instead stay within that multiple of their own bound (used at sizes of tens of
    millions of elements, where the tail of the BF16 rounding error crosses any fixed multiple of its spread)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    if want.size == 0:
        return
    rms = float(np.sqrt(np.mean(want * want)))
    err = np.abs(got - want)
    bound = tol * np.abs(want) + tol * rms
    bad = err > bound
    if bad.any():
        frac = bad.mean()
        worst = int(np.argmax(err - bound))
        msg = (f"{name}: {bad.sum()} / {bad.size} elements outside tol={tol:g} (rms {rms:.3g}); worst flat index "
               f"{worst}: got {got.ravel()[worst]!r} want {want.ravel()[worst]!r}")
        if outlier_factor > 0.0:
            assert frac <= max_outlier_frac and np.all(err[bad] <= outlier_factor * bound[bad]), msg
        else:
            assert frac <= max_outlier_frac and err[bad].max() <= outlier_abs, msg


def rel_l2(got, want) -> float:
    got = np.asarray(got, dtype=np.float64); want = np.asarray(want, dtype=np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


class _DevView:
    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2}


_TYPESTR = {np.dtype(np.float32): "<f4", np.dtype(np.uint8): "|u1", np.dtype(np.int32): "<i4"}


def dev_to_numpy(ptr: int, shape, dtype=np.float32) -> np.ndarray:
    """Copy a device buffer owned by the library into a numpy array."""
    import torch
    t = torch.as_tensor(_DevView(ptr, shape, _TYPESTR[np.dtype(dtype)]), device="cuda")
    return t.cpu().numpy().copy()


def numpy_to_dev(ptr: int, arr: np.ndarray):
    """Overwrite a device buffer owned by the library with a numpy array of the same shape."""
    import torch
    t = torch.as_tensor(_DevView(ptr, arr.shape, _TYPESTR[arr.dtype]), device="cuda")
    t.copy_(torch.from_numpy(np.ascontiguousarray(arr)))
    torch.cuda.synchronize()


def dims_of(w: WL.Workload):
    return (w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)


def gpu_rollout(ctx, w: WL.Workload, inputs: Dict[str, np.ndarray]):
    """T x (act, record_step) + gae through the C ABI with device-resident inputs."""
    import torch
    dev = torch.device("cuda")
    oa = torch.from_numpy(inputs["obs_actor"]).to(dev)
    oc = oa if w.shared_obs else torch.from_numpy(inputs["obs_critic"]).to(dev)
    rew = torch.from_numpy(inputs["rewards"]).to(dev)
    dn = torch.from_numpy(inputs["dones"]).to(dev)
    to = torch.from_numpy(inputs["timeouts"]).to(dev)
    for t in range(w.num_steps):
        ctx.act(oa[t], None if w.shared_obs else oc[t])
        ctx.record_step(rew[t], dn[t], to[t])
    ctx.gae(oc[w.num_steps])
    torch.cuda.synchronize()


def read_storage(ctx, w: WL.Workload, with_obs: bool = True) -> Dict[str, np.ndarray]:
    s = ctx.storage_view()
    T, N, A = w.num_steps, w.num_envs, w.num_actions
    out = {}
    if with_obs:
        out["obs_actor"] = dev_to_numpy(s.obs_actor, (T, N, s.obs_a_stride))[..., :w.actor_obs_dim]
        out["obs_critic"] = dev_to_numpy(s.obs_critic, (T, N, s.obs_c_stride))[..., :w.critic_obs_dim]
    out["actions"] = dev_to_numpy(s.actions, (T, N, s.act_stride))[..., :A]
    out["mu"] = dev_to_numpy(s.mu, (T, N, s.act_stride))[..., :A]
    out["sigma"] = dev_to_numpy(s.sigma, (T, s.act_stride))[..., :A]
    for k in ("logp", "values", "rewards", "returns", "advantages"):
        out[k] = dev_to_numpy(getattr(s, k), (T, N))
    out["dones"] = dev_to_numpy(s.dones, (T, N), np.uint8)
    out["timeouts"] = dev_to_numpy(s.timeouts, (T, N), np.uint8)
    return out


def write_storage(ctx, w: WL.Workload, st: Dict[str, np.ndarray]):
    """Load an oracle-made rollout into the library's storage (oracle -> CUDA direction only)."""
    s = ctx.storage_view()

    def padded(x, stride):
        out = np.zeros((*x.shape[:-1], stride), dtype=np.float32)
        out[..., :x.shape[-1]] = x
        return out

    numpy_to_dev(s.obs_actor, padded(st["obs_actor"].astype(np.float32), s.obs_a_stride))
    if not w.shared_obs:
        numpy_to_dev(s.obs_critic, padded(st["obs_critic"].astype(np.float32), s.obs_c_stride))
    numpy_to_dev(s.actions, padded(st["actions"].astype(np.float32), s.act_stride))
    numpy_to_dev(s.mu, padded(st["mu"].astype(np.float32), s.act_stride))
    numpy_to_dev(s.sigma, padded(st["sigma"].astype(np.float32), s.act_stride))
    for k in ("logp", "values", "rewards", "returns", "advantages"):
        numpy_to_dev(getattr(s, k), st[k].astype(np.float32))
    numpy_to_dev(s.dones, st["dones"].astype(np.uint8))
    numpy_to_dev(s.timeouts, st["timeouts"].astype(np.uint8))


def oracle_rollout(w: WL.Workload, theta: np.ndarray, inputs, first_global_step: int = 0):
    return O.rollout(theta.astype(np.float64), dims_of(w), inputs, w, seed=w.seed,
                     first_global_step=first_global_step)
