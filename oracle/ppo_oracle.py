"""Plain FP64 CPU oracle of the PPO learn-iteration hot path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares no code with the CUDA library and imports nothing from it; it is the
slow, obviously-correct statement of what that library must compute.

What it follows.  The paper (RSL-RL, "Features / Algorithms" and "Implementation
Details") names PPO after Schulman et al. 2017, an actor-critic with MLP networks, a
"proper handling of episodic timeouts", environments in same-step-reset mode, and a
symmetry augmentation with an optional symmetry loss ("Auxiliary Techniques"); it prints
no equation.  Every function below is therefore the textbook definition that those names
denote, written out in numpy float64 with no blocking, fusion or reordering:

* ``act``                 -- MLP actor/critic, diagonal Gaussian policy with a state-independent
                             learned log-std, sample + log-density           (PPO, Algorithms)
* ``gae``                 -- generalised advantage estimation as a reverse recursion with
                             time-out bootstrapping           (Implementation Details: timeouts,
                             same-step reset)
* ``normalize_advantages``-- (A - mean) / (std + eps) over the whole rollout
* ``ppo_loss_and_grads``  -- clipped surrogate, clipped value loss, entropy bonus, KL(old||new),
                             optional symmetry loss, and their exact gradient by reverse mode
* ``clip_coefficient`` / ``adaptive_lr`` / ``adam_step`` -- global-norm clipping, the
                             KL-adaptive learning-rate rule, Adam (Kingma & Ba) with bias
                             correction
* ``ppo_update``          -- the epoch x minibatch loop over a keyed permutation
* ``distill_loss_and_grads`` / ``distill_update`` -- the behaviour-cloning step of "Algorithms": the
                             student (the actor net) is rolled out, its transitions are relabelled
                             with the expert's actions, and the student's mean is regressed on them
                             (mean squared error, the paper names no loss) over the same keyed
                             minibatches, with global-norm clipping and Adam, no learning-rate rule
* ``rnd_reward`` / ``rnd_loss_and_grads`` / ``rnd_update`` -- the curiosity bonus of "Auxiliary
                             Techniques": random network distillation (Burda et al. 2019) on a subset of
                             the state: r_int = mean_j (f_j(s) - g_j(s))^2 with a fixed random target g and
                             a trained predictor f, and the predictor's regression step
* ``philox4x32_10``, ``gaussian_noise``, ``feistel_permutation`` -- the counter-based random
                             streams the method draws from (Salmon et al., SC'11), so that a
                             second implementation can reproduce noise and shuffles bit for bit.

Pins (tests/test_oracle_*.py): Philox known-answer vectors; Gaussian log-density vs
scipy.stats; GAE vs brute-force discounted sums, lambda=0 / lambda=1 / gamma=0 closed forms
and the two-pass time-out formulation; normalisation vs numpy ddof=1; ratio=1 surrogate;
losses and every gradient block vs torch float64 autograd and central finite differences;
Adam vs torch.optim.Adam and a hand-computed first step; permutation bijectivity by brute
force.  No function here is "parity unpinned" against the definitions; what *cannot* be
pinned is agreement with the public RSL-RL code base (not available): the readings taken
where the paper is silent are listed in the design notes.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64
_MASK32 = np.uint64(0xFFFFFFFF)

# ======================================================================================
# Counter-based randomness (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
# as 1, 2, 3", SC'11): Philox-4x32 with 10 rounds.
# ======================================================================================
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)   # golden ratio
_PHILOX_W1 = np.uint64(0xBB67AE85)   # sqrt(3) - 1


def philox4x32_10(counter: np.ndarray, key: Sequence[int]) -> np.ndarray:
    """Philox-4x32-10 block function.

    ``counter``: uint array [..., 4]; ``key``: two 32-bit words.  Returns uint32 [..., 4].
    One round maps (c0,c1,c2,c3) to (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0));
    the key is bumped by the Weyl constants between rounds.
    """
    c = np.asarray(counter).astype(np.uint64) & _MASK32
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0 = np.uint64(int(key[0]) & 0xFFFFFFFF)
    k1 = np.uint64(int(key[1]) & 0xFFFFFFFF)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & _MASK32
            k1 = (k1 + _PHILOX_W1) & _MASK32
        p0 = _PHILOX_M0 * c0          # 32x32 -> 64 bit products, exact in uint64
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


STREAM_NOISE = 1
STREAM_PERM = 2


def _seed_key(seed: int) -> Tuple[int, int]:
    return seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF


def uniform_open01(bits: np.ndarray) -> np.ndarray:
    """Map uint32 words to the open interval (0,1): u = ((x >> 9) + 1/2) * 2^-23.

    24 significant bits, so u is exactly representable in float32 as well as float64.
    """
    return ((bits >> np.uint32(9)).astype(F64) + 0.5) * (2.0 ** -23)


def gaussian_noise(seed: int, global_step: int, num_envs: int, num_actions: int) -> np.ndarray:
    """Standard-normal noise eps[num_envs][num_actions] for one rollout step.

    Counter (env n, global_step, quad j, STREAM_NOISE) -> four words (x0..x3) -> uniforms
    (u0..u3) -> two Box-Muller pairs:
        eps[4j+0] = sqrt(-2 ln u0) cos(2 pi u1),  eps[4j+1] = sqrt(-2 ln u0) sin(2 pi u1),
        eps[4j+2] = sqrt(-2 ln u2) cos(2 pi u3),  eps[4j+3] = sqrt(-2 ln u2) sin(2 pi u3).
    """
    quads = (num_actions + 3) // 4
    n = np.arange(num_envs, dtype=np.uint64)[:, None]
    j = np.arange(quads, dtype=np.uint64)[None, :]
    ctr = np.stack(np.broadcast_arrays(n, np.uint64(global_step), j, np.uint64(STREAM_NOISE)), axis=-1)
    u = uniform_open01(philox4x32_10(ctr, _seed_key(seed)))          # [N][quads][4]
    r01 = np.sqrt(-2.0 * np.log(u[..., 0]))
    r23 = np.sqrt(-2.0 * np.log(u[..., 2]))
    eps = np.stack([r01 * np.cos(2.0 * np.pi * u[..., 1]), r01 * np.sin(2.0 * np.pi * u[..., 1]),
                    r23 * np.cos(2.0 * np.pi * u[..., 3]), r23 * np.sin(2.0 * np.pi * u[..., 3])], axis=-1)
    return eps.reshape(num_envs, quads * 4)[:, :num_actions]


FEISTEL_ROUNDS = 6


def feistel_permutation(seed: int, iteration: int, epoch: int, size: int) -> np.ndarray:
    """Keyed bijection perm[0..size) -> [0..size): the minibatch shuffle of one epoch.

    A balanced Feistel network over 2h bits (2h = the smallest even width with 2^(2h) >= size),
    FEISTEL_ROUNDS rounds, round function = word 0 of Philox(counter=(right half, epoch,
    iteration, STREAM_PERM | round << 8), key=seed) masked to h bits; values that land
    outside [0,size) are fed through the network again ("cycle walking") until they fall
    inside.  A Feistel network is a bijection of its domain for any round function, and
    cycle walking restricts a bijection to a bijection of the sub-range.
    """
    if size <= 0:
        return np.zeros(0, dtype=np.int64)
    bits = max(2, int(size - 1).bit_length())
    bits += bits & 1
    h = bits // 2
    hmask = np.uint64((1 << h) - 1)
    key = _seed_key(seed)

    def network(x: np.ndarray) -> np.ndarray:
        left, right = x >> np.uint64(h), x & hmask
        for rnd in range(FEISTEL_ROUNDS):
            ctr = np.stack(np.broadcast_arrays(right, np.uint64(epoch), np.uint64(iteration),
                                               np.uint64(STREAM_PERM | (rnd << 8))), axis=-1)
            f = philox4x32_10(ctr, key)[..., 0].astype(np.uint64) & hmask
            left, right = right, left ^ f
        return (left << np.uint64(h)) | right

    x = network(np.arange(size, dtype=np.uint64))
    while True:
        outside = x >= np.uint64(size)
        if not outside.any():
            break
        x[outside] = network(x[outside])
    return x.astype(np.int64)


# ======================================================================================
# Networks
# ======================================================================================
def unpack_params(flat: np.ndarray, actor_dims: Sequence[Tuple[int, int]],
                  critic_dims: Sequence[Tuple[int, int]], num_actions: int) -> Dict[str, object]:
    """Split the flat parameter vector.

    Order: actor W1[in][out], b1, ..., Wout, bout, log_std[A]; critic W1, b1, ..., Wout, bout.
    Returns {"actor": [(W,b),...], "log_std": vec, "critic": [(W,b),...]} as float64 views/copies.
    """
    flat = np.asarray(flat, dtype=F64)
    off = 0
    out: Dict[str, object] = {}
    for net, dims in (("actor", actor_dims), ("critic", critic_dims)):
        layers = []
        for fi, fo in dims:
            W = flat[off:off + fi * fo].reshape(fi, fo); off += fi * fo
            b = flat[off:off + fo]; off += fo
            layers.append((W, b))
        out[net] = layers
        if net == "actor":
            out["log_std"] = flat[off:off + num_actions]; off += num_actions
    assert off == flat.size, (off, flat.size)
    return out


def pack_grads(g: Dict[str, object]) -> np.ndarray:
    parts = []
    for net in ("actor", "critic"):
        for W, b in g[net]:
            parts += [W.ravel(), b.ravel()]
        if net == "actor":
            parts.append(np.asarray(g["log_std"]).ravel())
    return np.concatenate(parts)


def elu(z: np.ndarray, alpha: float) -> np.ndarray:
    return np.where(z > 0.0, z, alpha * np.expm1(np.minimum(z, 0.0)))


def mlp_forward(x: np.ndarray, layers, alpha: float) -> Tuple[np.ndarray, List[np.ndarray]]:
    """h_0 = x; h_l = ELU(h_{l-1} W_l + b_l) on hidden layers; linear head.

    Returns (head output, [h_0, h_1, ..., h_L]) -- the post-activations the backward needs.
    """
    hs = [np.asarray(x, dtype=F64)]
    for W, b in layers[:-1]:
        hs.append(elu(hs[-1] @ W + b, alpha))
    W, b = layers[-1]
    return hs[-1] @ W + b, hs


def mlp_backward(d_out: np.ndarray, hs: List[np.ndarray], layers, alpha: float):
    """Reverse mode through ``mlp_forward``: returns [(dW_l, db_l)] for every layer.

    dZ_out = d_out; dW_l = h_{l-1}^T dZ_l; db_l = column sums of dZ_l;
    dh_{l-1} = dZ_l W_l^T; dZ_{l-1} = dh_{l-1} * ELU'(z_{l-1}) with ELU' written in terms of the
    stored post-activation: 1 where h > 0, else h + alpha.
    """
    grads = [None] * len(layers)
    dZ = d_out
    for l in range(len(layers) - 1, -1, -1):
        W, _ = layers[l]
        grads[l] = (hs[l].T @ dZ, dZ.sum(axis=0))
        if l > 0:
            dH = dZ @ W.T
            dZ = dH * np.where(hs[l] > 0.0, 1.0, hs[l] + alpha)
    return grads


_HALF_LOG_2PI = 0.5 * math.log(2.0 * math.pi)


def gaussian_log_prob(a: np.ndarray, mu: np.ndarray, log_std: np.ndarray) -> np.ndarray:
    """log N(a; mu, diag(sigma^2)) summed over action dims, sigma = exp(log_std)."""
    sigma = np.exp(log_std)
    return (-(a - mu) ** 2 / (2.0 * sigma ** 2) - log_std - _HALF_LOG_2PI).sum(axis=-1)


def gaussian_entropy(log_std: np.ndarray) -> float:
    """Entropy of the diagonal Gaussian: sum_i (1/2 + 1/2 log 2 pi + log sigma_i)."""
    return float((0.5 + _HALF_LOG_2PI + log_std).sum())


# ======================================================================================
# (1) act
# ======================================================================================
def act(params, obs_actor: np.ndarray, obs_critic: np.ndarray, alpha: float,
        seed: int, global_step: int) -> Dict[str, np.ndarray]:
    """One rollout step over all environments: mu = actor(o_a), V = critic(o_c),
    a = mu + sigma * eps with eps from ``gaussian_noise``, log-density of a."""
    mu, _ = mlp_forward(obs_actor, params["actor"], alpha)
    v, _ = mlp_forward(obs_critic, params["critic"], alpha)
    log_std = np.asarray(params["log_std"], dtype=F64)
    sigma = np.exp(log_std)
    eps = gaussian_noise(seed, global_step, mu.shape[0], mu.shape[1])
    actions = mu + sigma * eps
    return {"actions": actions, "mu": mu, "sigma": sigma, "values": v[:, 0],
            "logp": gaussian_log_prob(actions, mu, log_std), "eps": eps}


# ======================================================================================
# (2) GAE with time-out bootstrapping, advantage normalisation
# ======================================================================================
def gae(rewards: np.ndarray, values: np.ndarray, dones: np.ndarray, timeouts: np.ndarray,
        last_values: np.ndarray, gamma: float, lam: float) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (returns[T][N], advantages[T][N]), advantages not yet normalised.

    For t = T-1 .. 0, per environment, with V_T = last_values and A_T = 0:
        r~_t  = r_t + gamma * V_t * timeout_t     (a time-out is not a failure: bootstrap from
                                                   the value of the state it was cut at; with
                                                   same-step reset the next observation already
                                                   belongs to the new episode)
        delta = r~_t + gamma * V_{t+1} * (1 - done_t) - V_t
        A_t   = delta + gamma * lam * (1 - done_t) * A_{t+1}
        R_t   = A_t + V_t
    """
    rewards = np.asarray(rewards, dtype=F64); values = np.asarray(values, dtype=F64)
    T, N = rewards.shape
    adv = np.zeros((T, N), dtype=F64)
    ret = np.zeros((T, N), dtype=F64)
    next_adv = np.zeros(N, dtype=F64)
    next_val = np.asarray(last_values, dtype=F64)
    for t in range(T - 1, -1, -1):
        not_done = 1.0 - dones[t].astype(F64)
        r_boot = rewards[t] + gamma * values[t] * timeouts[t].astype(F64)
        delta = r_boot + gamma * next_val * not_done - values[t]
        next_adv = delta + gamma * lam * not_done * next_adv
        adv[t] = next_adv
        ret[t] = next_adv + values[t]
        next_val = values[t]
    return ret, adv


def normalize_advantages(adv: np.ndarray, eps: float = 1e-8, unbiased: bool = True) -> np.ndarray:
    """(A - mean) / (std + eps) over every transition of the rollout."""
    a = np.asarray(adv, dtype=F64)
    n = a.size
    mean = a.sum() / n
    var = ((a - mean) ** 2).sum() / (n - 1 if unbiased else n)
    return (a - mean) / (math.sqrt(var) + eps)


# ======================================================================================
# (3) PPO minibatch update
# ======================================================================================
def mirror(x: np.ndarray, perm: np.ndarray, sign: np.ndarray) -> np.ndarray:
    """(S x)[..., i] = sign[i] * x[..., perm[i]]."""
    return np.asarray(sign, dtype=F64) * x[..., np.asarray(perm, dtype=np.int64)]


def ppo_loss_and_grads(params, batch: Dict[str, np.ndarray], hp, sym: Optional[Dict] = None):
    """Losses, KL and the exact gradient for one minibatch.

    ``batch``: obs_actor[B][Da], obs_critic[B][Dc], actions[B][A], logp_old[B], values_old[B],
    returns[B], advantages[B] (already normalised), mu_old[B][A], sigma_old[B][A].
    ``hp``: any object with clip, value_clip, value_coef, entropy_coef, use_clipped_value_loss,
    elu_alpha, sym_coef.  ``sym``: mirror tables or None.

    With B' the number of rows in the (possibly mirrored) batch:
        ratio = exp(logp_new - logp_old)
        L_s   = mean_B' max(-A ratio, -A clip(ratio, 1-c, 1+c))
        V_c   = V_old + clip(V - V_old, -c_v, c_v)
        L_v   = mean_B' max((V-R)^2, (V_c-R)^2)          (plain (V-R)^2 when clipping is off)
        H     = entropy of the policy (identical for every row)
        L_sym = mean over B x A of (mu(S_o o) - S_a sg[mu(o)])^2
        L     = L_s + k_v L_v - k_e H + k_sym L_sym
        KL    = mean_B sum_i [log(s_i/s_old,i) + (s_old,i^2 + (mu_old,i - mu_i)^2)/(2 s_i^2) - 1/2]
    Mirrored rows (appended after the B originals) reuse A, R, V_old, logp_old of their source
    row; the KL uses the B original rows only.
    Returns (stats dict, gradient dict shaped like ``params``).
    """
    alpha = hp.elu_alpha
    oa = np.asarray(batch["obs_actor"], dtype=F64)
    oc = np.asarray(batch["obs_critic"], dtype=F64)
    a = np.asarray(batch["actions"], dtype=F64)
    logp_old = np.asarray(batch["logp_old"], dtype=F64)
    v_old = np.asarray(batch["values_old"], dtype=F64)
    R = np.asarray(batch["returns"], dtype=F64)
    A_hat = np.asarray(batch["advantages"], dtype=F64)
    mu_old = np.asarray(batch["mu_old"], dtype=F64)
    sigma_old = np.asarray(batch["sigma_old"], dtype=F64)
    B = oa.shape[0]
    nA = a.shape[1]
    if sym is not None:
        oa = np.concatenate([oa, mirror(oa, sym["obs_perm"], sym["obs_sign"])], axis=0)
        oc = np.concatenate([oc, mirror(oc, sym["cobs_perm"], sym["cobs_sign"])], axis=0)
        a = np.concatenate([a, mirror(a, sym["act_perm"], sym["act_sign"])], axis=0)
        logp_old = np.concatenate([logp_old, logp_old]); v_old = np.concatenate([v_old, v_old])
        R = np.concatenate([R, R]); A_hat = np.concatenate([A_hat, A_hat])
    Bp = oa.shape[0]

    mu, hs_a = mlp_forward(oa, params["actor"], alpha)
    v2, hs_c = mlp_forward(oc, params["critic"], alpha)
    V = v2[:, 0]
    log_std = np.asarray(params["log_std"], dtype=F64)
    sigma = np.exp(log_std)

    # ---- losses --------------------------------------------------------------------
    logp = gaussian_log_prob(a, mu, log_std)
    ratio = np.exp(logp - logp_old)
    s_unclipped = -A_hat * ratio
    s_clipped = -A_hat * np.clip(ratio, 1.0 - hp.clip, 1.0 + hp.clip)
    L_s = np.maximum(s_unclipped, s_clipped).sum() / Bp
    if hp.use_clipped_value_loss:
        V_c = v_old + np.clip(V - v_old, -hp.value_clip, hp.value_clip)
        e_unclipped, e_clipped = (V - R) ** 2, (V_c - R) ** 2
        L_v = np.maximum(e_unclipped, e_clipped).sum() / Bp
    else:
        L_v = ((V - R) ** 2).sum() / Bp
    H = gaussian_entropy(log_std)
    kl_rows = (np.log(sigma / sigma_old) + (sigma_old ** 2 + (mu_old - mu[:B]) ** 2) / (2.0 * sigma ** 2)
               - 0.5).sum(axis=1)
    KL = kl_rows.sum() / B
    L_sym = 0.0
    if sym is not None:
        target = mirror(mu[:B], sym["act_perm"], sym["act_sign"])      # no gradient flows here
        diff = mu[B:] - target
        L_sym = (diff ** 2).sum() / (B * nA)
    k_sym = hp.sym_coef if sym is not None else 0.0
    L = L_s + hp.value_coef * L_v - hp.entropy_coef * H + k_sym * L_sym

    # ---- gradient of L ----------------------------------------------------------------
    # surrogate: d/dlogp of max(-A r, -A clip(r)).  Inside the clip range both branches are
    # the same function; outside, the clipped branch is constant, so the gradient is -A r
    # where the unclipped branch is the larger one and 0 otherwise.
    inside = (ratio >= 1.0 - hp.clip) & (ratio <= 1.0 + hp.clip)
    take_unclipped = inside | (s_unclipped > s_clipped)
    dlogp = np.where(take_unclipped, -A_hat * ratio, 0.0) / Bp
    dmu = dlogp[:, None] * (a - mu) / sigma ** 2
    dlog_std = (dlogp[:, None] * ((a - mu) ** 2 / sigma ** 2 - 1.0)).sum(axis=0)
    dlog_std = dlog_std - hp.entropy_coef * np.ones(nA)            # dH/dlog_std_i = 1
    if hp.use_clipped_value_loss:
        v_inside = np.abs(V - v_old) <= hp.value_clip
        take_e_unclipped = v_inside | (e_unclipped > e_clipped)
        dV = np.where(take_e_unclipped, 2.0 * (V - R), 0.0)
    else:
        dV = 2.0 * (V - R)
    dV = hp.value_coef * dV / Bp
    if sym is not None:
        dmu[B:] += k_sym * 2.0 * diff / (B * nA)

    g_actor = mlp_backward(dmu, hs_a, params["actor"], alpha)
    g_critic = mlp_backward(dV[:, None], hs_c, params["critic"], alpha)
    grads = {"actor": g_actor, "critic": g_critic, "log_std": dlog_std}
    stats = {"loss": float(L), "surrogate": float(L_s), "value_loss": float(L_v), "entropy": H,
             "kl": float(KL), "sym_loss": float(L_sym), "mu": mu, "values": V, "logp": logp,
             "ratio": ratio, "dmu": dmu, "dV": dV}
    return stats, grads


def clip_coefficient(grad_norm: float, max_norm: float) -> float:
    """Global-norm clipping factor min(1, max_norm / (||g|| + 1e-6))."""
    return min(1.0, max_norm / (grad_norm + 1e-6))


def adaptive_lr(lr: float, kl: float, hp) -> float:
    """KL-adaptive step size: shrink by ``lr_factor`` when KL > 2 d, grow when KL < d / 2,
    clamped to [lr_min, lr_max]; d = desired_kl."""
    if not hp.adaptive_lr:
        return lr
    if kl > 2.0 * hp.desired_kl:
        return max(hp.lr_min, lr / hp.lr_factor)
    if kl < hp.desired_kl / 2.0:
        return min(hp.lr_max, lr * hp.lr_factor)
    return lr


def adam_step(theta: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, step: int,
              lr: float, b1: float, b2: float, eps: float):
    """One Adam step (Kingma & Ba, Algorithm 1); ``step`` is the 1-based count of this step.

    m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
    theta <- theta - lr * (m / (1-b1^step)) / (sqrt(v / (1-b2^step)) + eps).
    """
    m = b1 * m + (1.0 - b1) * g
    v = b2 * v + (1.0 - b2) * g * g
    m_hat = m / (1.0 - b1 ** step)
    v_hat = v / (1.0 - b2 ** step)
    return theta - lr * m_hat / (np.sqrt(v_hat) + eps), m, v


class OptimState:
    """Flat parameters with Adam moments, step count, current learning rate."""

    def __init__(self, theta: np.ndarray, lr: float):
        self.theta = np.asarray(theta, dtype=F64).copy()
        self.m = np.zeros_like(self.theta)
        self.v = np.zeros_like(self.theta)
        self.step = 0
        self.lr = float(lr)


def gather_minibatch(storage: Dict[str, np.ndarray], rows: np.ndarray) -> Dict[str, np.ndarray]:
    """Pick transitions ``rows`` (indices into the flattened [T][N] storage, t-major)."""
    T, N = storage["rewards"].shape
    t_idx = rows // N
    flat = lambda x: x.reshape(T * N, *x.shape[2:])
    return {
        "obs_actor": flat(storage["obs_actor"])[rows], "obs_critic": flat(storage["obs_critic"])[rows],
        "actions": flat(storage["actions"])[rows], "logp_old": flat(storage["logp"])[rows],
        "values_old": flat(storage["values"])[rows], "returns": flat(storage["returns"])[rows],
        "advantages": flat(storage["advantages"])[rows], "mu_old": flat(storage["mu"])[rows],
        "sigma_old": storage["sigma"][t_idx],
    }


def ppo_minibatch_step(state: OptimState, dims, batch, hp, sym=None):
    """Forward, loss, backward, KL-adaptive lr, clip, Adam on one minibatch.

    The learning rate is adapted from this minibatch's KL *before* its optimizer step.
    Returns the stats of ``ppo_loss_and_grads`` plus grad (flat, pre-clip), grad_norm, lr.
    """
    actor_dims, critic_dims, nA = dims
    params = unpack_params(state.theta, actor_dims, critic_dims, nA)
    stats, grads = ppo_loss_and_grads(params, batch, hp, sym)
    g = pack_grads(grads)
    state.lr = adaptive_lr(state.lr, stats["kl"], hp)
    g_norm = math.sqrt(float((g * g).sum()))
    coef = clip_coefficient(g_norm, hp.max_grad_norm)
    state.step += 1
    state.theta, state.m, state.v = adam_step(state.theta, g * coef, state.m, state.v, state.step,
                                              state.lr, hp.adam_b1, hp.adam_b2, hp.adam_eps)
    stats.update({"grad": g, "grad_norm": g_norm, "lr": state.lr})
    return stats


def ppo_update(state: OptimState, dims, storage: Dict[str, np.ndarray], hp, seed: int,
               iteration: int, sym=None, max_steps: Optional[int] = None) -> List[Dict]:
    """The epoch x minibatch loop.  Every epoch draws a fresh ``feistel_permutation`` of the
    B = T*N transitions and cuts it into ``hp.minibatches`` contiguous chunks of B / M rows.
    Returns the per-step stats (tensors dropped except for the first step)."""
    T, N = storage["rewards"].shape
    B = T * N
    if B % hp.minibatches:
        raise ValueError("batch not divisible by the number of minibatches")
    rows_per = B // hp.minibatches
    out = []
    for e in range(hp.epochs):
        perm = feistel_permutation(seed, iteration, e, B)
        for k in range(hp.minibatches):
            if max_steps is not None and len(out) >= max_steps:
                return out
            rows = perm[k * rows_per:(k + 1) * rows_per]
            st = ppo_minibatch_step(state, dims, gather_minibatch(storage, rows), hp, sym)
            if out:
                for key in ("mu", "values", "logp", "ratio", "dmu", "dV"):
                    st.pop(key, None)
            st["rows"] = rows if not out else None
            out.append(st)
    return out


# ======================================================================================
# Distillation ("Algorithms": a behaviour-cloning algorithm similar to DAgger: roll out the
# student, relabel the data with expert actions, train the student on it).  The paper names no
# loss; the reading taken is the mean squared error between the student's action mean and the
# expert's action, L = mean over rows and actions of (mu_student - a_expert)^2.  Only the actor
# net receives a gradient (log_std and the critic get zero), the learning rate stays fixed.
# ======================================================================================
def distill_loss_and_grads(params, obs_actor: np.ndarray, expert_actions: np.ndarray, hp):
    """L = sum_{r,i} (mu_i(o_r) - a*_{r,i})^2 / (B A) and its exact gradient (same layout as params)."""
    oa = np.asarray(obs_actor, dtype=F64)
    target = np.asarray(expert_actions, dtype=F64)
    B, nA = target.shape
    mu, hs = mlp_forward(oa, params["actor"], hp.elu_alpha)
    diff = mu - target
    L = (diff ** 2).sum() / (B * nA)
    dmu = 2.0 * diff / (B * nA)
    g_actor = mlp_backward(dmu, hs, params["actor"], hp.elu_alpha)
    g_critic = [(np.zeros_like(np.asarray(W, dtype=F64)), np.zeros_like(np.asarray(b, dtype=F64)))
                for W, b in params["critic"]]
    grads = {"actor": g_actor, "critic": g_critic, "log_std": np.zeros(nA)}
    return {"loss": float(L), "mu": mu, "dmu": dmu}, grads


def distill_update(state: OptimState, dims, obs_actor: np.ndarray, expert_actions: np.ndarray, hp, seed: int,
                   iteration: int, max_steps: Optional[int] = None) -> List[Dict]:
    """Epoch x minibatch loop of the distillation step over obs_actor[T][N][Da] / expert_actions[T][N][A]:
    the same keyed permutation and contiguous chunks as ``ppo_update``; per minibatch the loss above,
    global-norm clipping and Adam with the fixed learning rate ``state.lr``."""
    T, N = expert_actions.shape[:2]
    B = T * N
    if B % hp.minibatches:
        raise ValueError("batch not divisible by the number of minibatches")
    rows_per = B // hp.minibatches
    actor_dims, critic_dims, nA = dims
    obs = np.asarray(obs_actor)[:T].reshape(B, -1)
    tgt = np.asarray(expert_actions).reshape(B, -1)
    out = []
    for e in range(hp.epochs):
        perm = feistel_permutation(seed, iteration, e, B)
        for k in range(hp.minibatches):
            if max_steps is not None and len(out) >= max_steps:
                return out
            rows = perm[k * rows_per:(k + 1) * rows_per]
            params = unpack_params(state.theta, actor_dims, critic_dims, nA)
            stats, grads = distill_loss_and_grads(params, obs[rows], tgt[rows], hp)
            g = pack_grads(grads)
            g_norm = math.sqrt(float((g * g).sum()))
            coef = clip_coefficient(g_norm, hp.max_grad_norm)
            state.step += 1
            state.theta, state.m, state.v = adam_step(state.theta, g * coef, state.m, state.v, state.step,
                                                      state.lr, hp.adam_b1, hp.adam_b2, hp.adam_eps)
            st = {"loss": stats["loss"], "grad": g, "grad_norm": g_norm, "lr": state.lr}
            out.append(st)
    return out


# ======================================================================================
# Random network distillation on a subset of the state ("Auxiliary Techniques": a curiosity-driven
# intrinsic reward based on RND, computed "using only a subset of the full state").  Following Burda
# et al. 2019: a fixed, randomly initialised target MLP g and a predictor MLP f of the same shape read
# s = o[idx]; the bonus is the predictor's squared error, the predictor is trained to reduce it.
# Readings where the paper is silent: the error is averaged over the E outputs; the bonus enters the
# stored reward as r + w * r_int; the predictor has its own Adam (no clipping, fixed learning rate)
# and sees the same keyed minibatches as the policy update.
# ======================================================================================
def unpack_mlp(flat: np.ndarray, dims: Sequence[Tuple[int, int]]):
    """[(W[in][out], b), ...] from the flat order W1, b1, W2, b2, ..."""
    flat = np.asarray(flat, dtype=F64)
    off, layers = 0, []
    for fi, fo in dims:
        W = flat[off:off + fi * fo].reshape(fi, fo); off += fi * fo
        b = flat[off:off + fo]; off += fo
        layers.append((W, b))
    assert off == flat.size, (off, flat.size)
    return layers


def rnd_reward(theta_f: np.ndarray, theta_g: np.ndarray, dims, obs: np.ndarray, idx: np.ndarray, alpha: float):
    """r_int[row] = mean_j (f_j(s) - g_j(s))^2 with s = obs[row][idx]; also returns f(s), g(s) and f's activations."""
    s = np.asarray(obs, dtype=F64)[:, np.asarray(idx)]
    f, hs = mlp_forward(s, unpack_mlp(theta_f, dims), alpha)
    g, _ = mlp_forward(s, unpack_mlp(theta_g, dims), alpha)
    return ((f - g) ** 2).mean(axis=1), f, g, hs


def rnd_loss_and_grads(theta_f: np.ndarray, theta_g: np.ndarray, dims, obs: np.ndarray, idx: np.ndarray, alpha: float):
    """L = mean over rows of r_int, and dL/dtheta_f (flat, same order as theta_f)."""
    r, f, g, hs = rnd_reward(theta_f, theta_g, dims, obs, idx, alpha)
    B, E = f.shape
    d_out = 2.0 * (f - g) / (B * E)
    grads = mlp_backward(d_out, hs, unpack_mlp(theta_f, dims), alpha)
    flat = np.concatenate([x.ravel() for W, b in grads for x in (W, b)])
    return float(r.mean()), flat


def rnd_update(state: OptimState, theta_g: np.ndarray, dims, obs: np.ndarray, idx: np.ndarray, hp, seed: int,
               iteration: int, max_steps: Optional[int] = None) -> List[Dict]:
    """Predictor training over obs[B][D]: hp.epochs x hp.minibatches steps over ``feistel_permutation`` chunks,
    Adam on ``state`` (the predictor's parameters and moments) with the fixed learning rate state.lr."""
    B = obs.shape[0]
    if B % hp.minibatches:
        raise ValueError("batch not divisible by the number of minibatches")
    rows_per = B // hp.minibatches
    out = []
    for e in range(hp.epochs):
        perm = feistel_permutation(seed, iteration, e, B)
        for k in range(hp.minibatches):
            if max_steps is not None and len(out) >= max_steps:
                return out
            rows = perm[k * rows_per:(k + 1) * rows_per]
            L, g = rnd_loss_and_grads(state.theta, theta_g, dims, obs[rows], idx, hp.elu_alpha)
            state.step += 1
            state.theta, state.m, state.v = adam_step(state.theta, g, state.m, state.v, state.step, state.lr,
                                                      hp.adam_b1, hp.adam_b2, hp.adam_eps)
            out.append({"loss": L, "grad": g})
    return out


# ======================================================================================
# a whole learn iteration (rollout replay + GAE + update), used by parity tests and the
# timed CPU baseline
# ======================================================================================
def rollout(state_theta: np.ndarray, dims, inputs: Dict[str, np.ndarray], hp, seed: int,
            first_global_step: int = 0) -> Dict[str, np.ndarray]:
    """Replay T pre-generated observation steps through ``act`` and fill the storage, then
    V_T = critic(o_T), GAE and normalisation.  ``inputs`` as made by the workload generators."""
    actor_dims, critic_dims, nA = dims
    params = unpack_params(state_theta, actor_dims, critic_dims, nA)
    T, N = inputs["rewards"].shape
    st = {k: [] for k in ("actions", "mu", "sigma", "logp", "values")}
    for t in range(T):
        o = act(params, inputs["obs_actor"][t], inputs["obs_critic"][t], hp.elu_alpha, seed,
                first_global_step + t)
        for k in st:
            st[k].append(o[k])
    storage = {k: np.stack(v) for k, v in st.items()}
    storage["obs_actor"] = np.asarray(inputs["obs_actor"][:T], dtype=F64)
    storage["obs_critic"] = np.asarray(inputs["obs_critic"][:T], dtype=F64)
    storage["rewards"] = np.asarray(inputs["rewards"], dtype=F64)
    storage["dones"] = inputs["dones"]; storage["timeouts"] = inputs["timeouts"]
    last_v, _ = mlp_forward(inputs["obs_critic"][T], params["critic"], hp.elu_alpha)
    storage["last_values"] = last_v[:, 0]
    ret, adv = gae(storage["rewards"], storage["values"], storage["dones"], storage["timeouts"],
                   storage["last_values"], hp.gamma, hp.lam)
    storage["returns"] = ret
    storage["advantages_raw"] = adv
    storage["advantages"] = (normalize_advantages(adv, hp.adv_eps, hp.adv_std_unbiased)
                             if hp.normalize_adv else adv)
    return storage
