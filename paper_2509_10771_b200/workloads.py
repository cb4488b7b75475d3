"""Seeded synthetic workloads for the PPO hot path.

This module only *describes* workloads (shapes, hyper-parameters) and draws their
synthetic inputs (observations, rewards, done / time-out flags, initial weights,
mirror tables) from numpy's seeded generators.  It contains none of the method's
arithmetic: no network evaluation, no advantage estimation, no loss.  Both the CPU
oracle's tests and the CUDA path's tests / benchmark feed on the arrays made here, so
the two sides always see byte-identical inputs.

The shapes stand in for the locomotion tasks the paper alludes to in its
"Applications in Research" section (legged locomotion in massively parallel
simulation); the paper itself prints no shapes, so the five named workloads below
are the ones this library is measured on.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

PRECISION_FP32 = 0
PRECISION_TF32 = 1
PRECISION_BF16 = 2


@dataclass(frozen=True)
class Workload:
    """One PPO learn-iteration workload: storage shape, networks, hyper-parameters."""

    name: str
    num_envs: int
    num_steps: int
    actor_obs_dim: int
    critic_obs_dim: int
    num_actions: int
    actor_hidden: Tuple[int, ...]
    critic_hidden: Tuple[int, ...]
    shared_obs: bool = True          # actor and critic read the same observation tensor
    # observation recipe: list of (width, "normal" | "uniform") blocks, per network
    actor_obs_blocks: Tuple[Tuple[int, str], ...] = ()
    critic_obs_blocks: Tuple[Tuple[int, str], ...] = ()
    reward_std: float = 0.1
    done_prob: float = 0.05
    timeout_frac: float = 0.3
    # PPO hyper-parameters
    gamma: float = 0.99
    lam: float = 0.95
    clip: float = 0.2
    value_clip: float = 0.2
    value_coef: float = 1.0
    entropy_coef: float = 0.01
    use_clipped_value_loss: bool = True
    epochs: int = 1
    minibatches: int = 2
    lr: float = 1e-3
    lr_min: float = 1e-5
    lr_max: float = 1e-2
    lr_factor: float = 1.5
    desired_kl: float = 0.01
    adaptive_lr: bool = True
    max_grad_norm: float = 1.0
    adam_b1: float = 0.9
    adam_b2: float = 0.999
    adam_eps: float = 1e-8
    normalize_adv: bool = True
    adv_std_unbiased: bool = True
    adv_eps: float = 1e-8
    elu_alpha: float = 1.0
    init_log_std: float = 0.0
    sym_enable: bool = False
    sym_coef: float = 0.0
    precision: int = PRECISION_FP32
    seed: int = 0

    @property
    def batch(self) -> int:
        return self.num_envs * self.num_steps

    @property
    def minibatch_rows(self) -> int:
        return self.batch // self.minibatches

    def layer_dims(self, net: str) -> List[Tuple[int, int]]:
        """(fan_in, fan_out) of every linear layer of ``net`` in ("actor", "critic")."""
        if net == "actor":
            dims = [self.actor_obs_dim, *self.actor_hidden, self.num_actions]
        else:
            dims = [self.critic_obs_dim, *self.critic_hidden, 1]
        return list(zip(dims[:-1], dims[1:]))

    def num_params(self) -> int:
        n = sum(i * o + o for i, o in self.layer_dims("actor")) + self.num_actions
        n += sum(i * o + o for i, o in self.layer_dims("critic"))
        return n

    def scaled(self, num_envs: int, name: Optional[str] = None, **kw) -> "Workload":
        """Same workload on fewer (or more) environments."""
        return replace(self, num_envs=num_envs, name=name or f"{self.name}@{num_envs}", **kw)


def _blocks(*b):
    return tuple(b)


TINY = Workload(
    name="tiny", num_envs=64, num_steps=8, actor_obs_dim=16, critic_obs_dim=16, num_actions=4,
    actor_hidden=(32, 32), critic_hidden=(32, 32),
    actor_obs_blocks=_blocks((16, "normal")), critic_obs_blocks=_blocks((16, "normal")),
    reward_std=0.1, done_prob=0.05, timeout_frac=0.3, epochs=1, minibatches=2)

FLAT = Workload(
    name="flat_terrain", num_envs=4096, num_steps=24, actor_obs_dim=48, critic_obs_dim=48,
    num_actions=12, actor_hidden=(128, 128, 128), critic_hidden=(128, 128, 128),
    actor_obs_blocks=_blocks((48, "normal")), critic_obs_blocks=_blocks((48, "normal")),
    reward_std=0.5, done_prob=0.005, timeout_frac=0.5, epochs=5, minibatches=4)

ROUGH = Workload(
    name="rough_terrain", num_envs=4096, num_steps=24, actor_obs_dim=235, critic_obs_dim=235,
    num_actions=12, actor_hidden=(512, 256, 128), critic_hidden=(512, 256, 128),
    actor_obs_blocks=_blocks((48, "normal"), (187, "uniform")),
    critic_obs_blocks=_blocks((48, "normal"), (187, "uniform")),
    reward_std=0.5, done_prob=0.005, timeout_frac=0.5, epochs=5, minibatches=4)

HUMANOID = Workload(
    name="humanoid_asymmetric", num_envs=8192, num_steps=24, actor_obs_dim=123,
    critic_obs_dim=300, num_actions=37, actor_hidden=(512, 256, 128),
    critic_hidden=(512, 256, 128), shared_obs=False,
    actor_obs_blocks=_blocks((123, "normal")), critic_obs_blocks=_blocks((300, "normal")),
    reward_std=1.0, done_prob=0.01, timeout_frac=0.3, epochs=5, minibatches=8)

ROUGH_SYM = Workload(
    name="rough_terrain_symmetry", num_envs=65536, num_steps=32, actor_obs_dim=235,
    critic_obs_dim=235, num_actions=12, actor_hidden=(512, 256, 128),
    critic_hidden=(512, 256, 128),
    actor_obs_blocks=_blocks((48, "normal"), (187, "uniform")),
    critic_obs_blocks=_blocks((48, "normal"), (187, "uniform")),
    reward_std=0.5, done_prob=0.005, timeout_frac=0.5, epochs=5, minibatches=16,
    sym_enable=True, sym_coef=1.0, precision=PRECISION_BF16)

WORKLOADS: Dict[str, Workload] = {w.name: w for w in (TINY, FLAT, ROUGH, HUMANOID, ROUGH_SYM)}
CONFIGS: Tuple[Workload, ...] = (TINY, FLAT, ROUGH, HUMANOID, ROUGH_SYM)


# --------------------------------------------------------------------------------------
# input generators (numpy seeded streams; float32 / uint8 arrays, C-contiguous)
# --------------------------------------------------------------------------------------
def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(stream)]))


def _draw_obs(rng: np.random.Generator, shape_prefix, blocks) -> np.ndarray:
    parts = []
    for width, law in blocks:
        shp = (*shape_prefix, width)
        if law == "normal":
            parts.append(rng.standard_normal(shp, dtype=np.float32))
        elif law == "uniform":
            parts.append((rng.random(shp, dtype=np.float32) * 2.0 - 1.0).astype(np.float32))
        else:
            raise ValueError(law)
    return np.ascontiguousarray(np.concatenate(parts, axis=-1))


def make_rollout_inputs(w: Workload, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Observations for T+1 steps, rewards and flags for T steps.

    Returns ``obs_actor[T+1][N][Da]``, ``obs_critic[T+1][N][Dc]`` (the same array object as
    ``obs_actor`` when the workload shares observations), ``rewards[T][N]`` float32,
    ``dones[T][N]`` and ``timeouts[T][N]`` uint8 with timeouts a subset of dones.
    """
    seed = w.seed if seed is None else seed
    T, N = w.num_steps, w.num_envs
    obs_a = _draw_obs(_rng(seed, 3), (T + 1, N), w.actor_obs_blocks)
    assert obs_a.shape[-1] == w.actor_obs_dim
    if w.shared_obs:
        obs_c = obs_a
    else:
        obs_c = _draw_obs(_rng(seed, 4), (T + 1, N), w.critic_obs_blocks)
        assert obs_c.shape[-1] == w.critic_obs_dim
    rew = (_rng(seed, 5).standard_normal((T, N), dtype=np.float32) * np.float32(w.reward_std))
    u = _rng(seed, 6).random((T, N))
    dones = (u < w.done_prob)
    u2 = _rng(seed, 7).random((T, N))
    timeouts = dones & (u2 < w.timeout_frac)
    assert not np.any(timeouts & ~dones)
    return {
        "obs_actor": obs_a, "obs_critic": obs_c, "rewards": rew.astype(np.float32),
        "dones": dones.astype(np.uint8), "timeouts": timeouts.astype(np.uint8),
    }


def make_expert_actions(w: Workload, seed: Optional[int] = None) -> np.ndarray:
    """Stand-in for an expert policy's relabelling of a student rollout: ``[T][N][A]`` float32 ~ N(0,1)
    (stream 9 of the workload's seed)."""
    seed = w.seed if seed is None else seed
    return _rng(seed, 9).standard_normal((w.num_steps, w.num_envs, w.num_actions), dtype=np.float32)


def rnd_layer_dims(num_idx: int, hidden: Sequence[int], embed_dim: int) -> List[Tuple[int, int]]:
    """(fan_in, fan_out) of the layers num_idx -> hidden... -> embed_dim of a distillation net."""
    widths = [num_idx, *hidden, embed_dim]
    return [(widths[i], widths[i + 1]) for i in range(len(widths) - 1)]


def make_rnd_setup(w: Workload, num_idx: int = 12, hidden: Sequence[int] = (128, 64), embed_dim: int = 32,
                   seed: Optional[int] = None) -> Dict[str, object]:
    """A state subset and the two nets of random network distillation for workload ``w`` (stream 10):
    ``idx`` = num_idx distinct entries of the actor observation (sorted), ``predictor`` / ``target`` = flat
    float32 vectors W1[in][out], b1, ... drawn like ``make_params``; the target is drawn four times wider
    so that the two nets differ at the start."""
    seed = w.seed if seed is None else seed
    rng = _rng(seed, 10)
    idx = np.sort(rng.choice(w.actor_obs_dim, size=num_idx, replace=False)).astype(np.int32)
    dims = rnd_layer_dims(num_idx, hidden, embed_dim)

    def draw(scale):
        parts = []
        for fi, fo in dims:
            bound = scale / np.sqrt(fi)
            parts.append(((rng.random(fi * fo + fo, dtype=np.float32) * 2.0 - 1.0) * bound).astype(np.float32))
        return np.concatenate(parts)

    return {"idx": idx, "dims": dims, "hidden": tuple(hidden), "embed_dim": embed_dim, "predictor": draw(1.0),
            "target": draw(4.0)}


def make_gru_setup(w: Workload, hidden_dim: int = 256, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Inputs of a recurrent memory layer over one rollout of workload ``w`` (stream 11): ``params`` flat float32
    in the order W_i[D][3H], b_i, W_h[H][3H], b_h drawn U(-1/sqrt(H), 1/sqrt(H)), ``h0[N][H]`` ~ 0.5 N(0,1) and
    ``dh[T][N][H]`` ~ N(0,1) / (T N) standing in for the gradient a downstream network sends back.  Observations
    and done flags are those of ``make_rollout_inputs``."""
    seed = w.seed if seed is None else seed
    rng = _rng(seed, 11)
    D, H, T, N = w.actor_obs_dim, hidden_dim, w.num_steps, w.num_envs
    n = D * 3 * H + 3 * H + H * 3 * H + 3 * H
    bound = 1.0 / np.sqrt(H)
    params = ((rng.random(n, dtype=np.float32) * 2.0 - 1.0) * bound).astype(np.float32)
    h0 = (rng.standard_normal((N, H), dtype=np.float32) * np.float32(0.5))
    dh = (rng.standard_normal((T, N, H), dtype=np.float32) / np.float32(T * N))
    return {"params": params, "h0": h0, "dh": dh, "hidden_dim": H}


def param_layout(w: Workload) -> List[Tuple[str, int, Tuple[int, ...]]]:
    """Flat parameter order: (name, offset, shape).

    actor W1[in][out], b1, ..., Wout, bout, log_std, then critic W1, b1, ..., Wout, bout.
    Weights are row-major ``[fan_in][fan_out]``.
    """
    out, off = [], 0
    for net in ("actor", "critic"):
        for li, (fi, fo) in enumerate(w.layer_dims(net)):
            out.append((f"{net}.W{li}", off, (fi, fo))); off += fi * fo
            out.append((f"{net}.b{li}", off, (fo,))); off += fo
        if net == "actor":
            out.append(("actor.log_std", off, (w.num_actions,))); off += w.num_actions
    assert off == w.num_params()
    return out


def make_params(w: Workload, seed: Optional[int] = None) -> np.ndarray:
    """Initial parameters, flat float32: U(-1/sqrt(fan_in), 1/sqrt(fan_in)), log_std constant."""
    seed = w.seed if seed is None else seed
    rng = _rng(seed, 8)
    flat = np.zeros(w.num_params(), dtype=np.float32)
    fan_in = 1
    for name, off, shape in param_layout(w):
        n = int(np.prod(shape))
        if name.endswith("log_std"):
            flat[off:off + n] = np.float32(w.init_log_std)
        else:
            if len(shape) == 2:          # a bias follows its weight and shares its fan-in
                fan_in = shape[0]
            bound = 1.0 / np.sqrt(fan_in)
            flat[off:off + n] = ((rng.random(n, dtype=np.float32) * 2.0 - 1.0) * bound).astype(np.float32)
    return flat


def _signed_involution(rng: np.random.Generator, dim: int, swap_frac: float = 0.4):
    """A signed permutation S with S^2 = I: disjoint transpositions + fixed points.

    ``(S x)[i] = sign[i] * x[perm[i]]``.  Swapped pairs carry a common sign, fixed points a
    free sign, which is exactly what makes S an involution.
    """
    order = rng.permutation(dim)
    n_pairs = int(dim * swap_frac) // 2
    perm = np.arange(dim, dtype=np.int32)
    sign = np.ones(dim, dtype=np.float32)
    for p in range(n_pairs):
        i, j = int(order[2 * p]), int(order[2 * p + 1])
        perm[i], perm[j] = j, i
        s = np.float32(1.0 if rng.random() < 0.5 else -1.0)
        sign[i] = sign[j] = s
    for i in order[2 * n_pairs:]:
        sign[int(i)] = np.float32(1.0 if rng.random() < 0.5 else -1.0)
    return perm, sign


def make_mirror(w: Workload, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Left/right mirror tables for actor obs, critic obs and actions (int32 perm, float32 sign)."""
    seed = w.seed if seed is None else seed
    rng = _rng(seed, 9)
    po, so = _signed_involution(rng, w.actor_obs_dim)
    if w.shared_obs:
        pc, sc = po.copy(), so.copy()
    else:
        pc, sc = _signed_involution(rng, w.critic_obs_dim)
    pa, sa = _signed_involution(rng, w.num_actions)
    return {"obs_perm": po, "obs_sign": so, "cobs_perm": pc, "cobs_sign": sc,
            "act_perm": pa, "act_sign": sa}


def identity_mirror(w: Workload) -> Dict[str, np.ndarray]:
    """The trivial mirror S = I (used by degenerate-case tests)."""
    return {"obs_perm": np.arange(w.actor_obs_dim, dtype=np.int32),
            "obs_sign": np.ones(w.actor_obs_dim, dtype=np.float32),
            "cobs_perm": np.arange(w.critic_obs_dim, dtype=np.int32),
            "cobs_sign": np.ones(w.critic_obs_dim, dtype=np.float32),
            "act_perm": np.arange(w.num_actions, dtype=np.int32),
            "act_sign": np.ones(w.num_actions, dtype=np.float32)}
