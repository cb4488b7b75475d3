"""Pins for the oracle's arithmetic: closed forms, brute force, library routines, autograd
and finite differences (no GPU).  A plausible mistake anywhere in oracle/ppo_oracle.py -- a
dropped term, a wrong sign, an index off by one, a transposed operand -- fails one of these."""
import math
from types import SimpleNamespace

import numpy as np
import pytest
import scipy.stats
import torch

from oracle import ppo_oracle as O
from paper_2509_10771_b200 import workloads as WL


# --------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------
def hp(**kw):
    d = dict(gamma=0.99, lam=0.95, clip=0.2, value_clip=0.2, value_coef=1.0, entropy_coef=0.01,
             use_clipped_value_loss=True, elu_alpha=1.0, sym_coef=1.0, lr=1e-3, lr_min=1e-5,
             lr_max=1e-2, lr_factor=1.5, desired_kl=0.01, adaptive_lr=True, max_grad_norm=1.0,
             adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8, epochs=1, minibatches=2,
             normalize_adv=True, adv_std_unbiased=True, adv_eps=1e-8)
    d.update(kw)
    return SimpleNamespace(**d)


def small_problem(seed=0, B=40, Da=7, Dc=9, A=3, hidden_a=(8, 6), hidden_c=(5, 7)):
    rng = np.random.default_rng(seed)
    adims = list(zip([Da, *hidden_a], [*hidden_a, A]))
    cdims = list(zip([Dc, *hidden_c], [*hidden_c, 1]))
    P = sum(i * o + o for i, o in adims) + A + sum(i * o + o for i, o in cdims)
    theta = rng.normal(0, 0.5, P)
    # old policy = a perturbed copy, so ratios straddle the clip range on both sides
    theta_old = theta + rng.normal(0, 0.08, P)
    oa, oc = rng.normal(size=(B, Da)), rng.normal(size=(B, Dc))
    p_old = O.unpack_params(theta_old, adims, cdims, A)
    mu_old, _ = O.mlp_forward(oa, p_old["actor"], 1.0)
    v_old, _ = O.mlp_forward(oc, p_old["critic"], 1.0)
    sig_old = np.exp(p_old["log_std"])
    a = mu_old + sig_old * rng.normal(size=(B, A))
    batch = dict(obs_actor=oa, obs_critic=oc, actions=a,
                 logp_old=O.gaussian_log_prob(a, mu_old, p_old["log_std"]),
                 values_old=v_old[:, 0], returns=v_old[:, 0] + rng.normal(0, 0.5, B),
                 advantages=rng.normal(size=B), mu_old=mu_old,
                 sigma_old=np.broadcast_to(sig_old, (B, A)).copy())
    return theta, (adims, cdims, A), batch


def torch_loss(theta_t, dims, batch, h, sym=None):
    """The same loss written with torch ops (autograd supplies the gradient)."""
    adims, cdims, A = dims
    off = 0
    nets = {}
    for net, dd in (("actor", adims), ("critic", cdims)):
        layers = []
        for fi, fo in dd:
            W = theta_t[off:off + fi * fo].reshape(fi, fo); off += fi * fo
            b = theta_t[off:off + fo]; off += fo
            layers.append((W, b))
        nets[net] = layers
        if net == "actor":
            log_std = theta_t[off:off + A]; off += A
    t = lambda x: torch.as_tensor(np.asarray(x), dtype=torch.float64)

    def mlp(x, layers):
        for W, b in layers[:-1]:
            x = torch.nn.functional.elu(x @ W + b, alpha=h.elu_alpha)
        W, b = layers[-1]
        return x @ W + b

    oa, oc, a = t(batch["obs_actor"]), t(batch["obs_critic"]), t(batch["actions"])
    lp_old, v_old, R, Ah = (t(batch[k]) for k in ("logp_old", "values_old", "returns", "advantages"))
    B = oa.shape[0]
    if sym is not None:
        mir = lambda x, p, s: t(s) * x[:, torch.as_tensor(np.asarray(p), dtype=torch.long)]
        oa = torch.cat([oa, mir(oa, sym["obs_perm"], sym["obs_sign"])])
        oc = torch.cat([oc, mir(oc, sym["cobs_perm"], sym["cobs_sign"])])
        a = torch.cat([a, mir(a, sym["act_perm"], sym["act_sign"])])
        lp_old, v_old, R, Ah = (torch.cat([x, x]) for x in (lp_old, v_old, R, Ah))
    mu, V = mlp(oa, nets["actor"]), mlp(oc, nets["critic"])[:, 0]
    dist = torch.distributions.Normal(mu, torch.exp(log_std).expand_as(mu))
    logp = dist.log_prob(a).sum(-1)
    ratio = torch.exp(logp - lp_old)
    L_s = torch.max(-Ah * ratio, -Ah * torch.clamp(ratio, 1 - h.clip, 1 + h.clip)).mean()
    if h.use_clipped_value_loss:
        Vc = v_old + (V - v_old).clamp(-h.value_clip, h.value_clip)
        L_v = torch.max((V - R) ** 2, (Vc - R) ** 2).mean()
    else:
        L_v = ((V - R) ** 2).mean()
    H = dist.entropy().sum(-1).mean()
    L = L_s + h.value_coef * L_v - h.entropy_coef * H
    L_sym = torch.zeros((), dtype=torch.float64)
    if sym is not None:
        tgt = (t(sym["act_sign"]) * mu[:B][:, torch.as_tensor(np.asarray(sym["act_perm"]), dtype=torch.long)]).detach()
        L_sym = torch.nn.functional.mse_loss(mu[B:], tgt)
        L = L + h.sym_coef * L_sym
    old = torch.distributions.Normal(t(batch["mu_old"]), t(batch["sigma_old"]))
    new = torch.distributions.Normal(mu[:B], torch.exp(log_std).expand_as(mu[:B]))
    kl = torch.distributions.kl_divergence(old, new).sum(-1).mean()
    return L, dict(surrogate=L_s, value_loss=L_v, entropy=H, kl=kl, sym_loss=L_sym)


def rand_mirror(rng, Da, Dc, A):
    po, so = WL._signed_involution(rng, Da)
    pc, sc = WL._signed_involution(rng, Dc)
    pa, sa = WL._signed_involution(rng, A, swap_frac=0.7)
    return dict(obs_perm=po, obs_sign=so, cobs_perm=pc, cobs_sign=sc, act_perm=pa, act_sign=sa)


# --------------------------------------------------------------------------------------
# networks and the Gaussian policy
# --------------------------------------------------------------------------------------
def test_elu_values_and_continuity():
    z = np.array([-30.0, -1.0, -1e-12, 0.0, 1e-12, 2.5])
    e = O.elu(z, 1.0)
    assert e[0] == pytest.approx(-1.0, abs=1e-12)
    assert e[1] == pytest.approx(math.exp(-1) - 1)
    assert e[3] == 0.0 and e[5] == 2.5
    assert abs(e[2] - e[4]) < 1e-11
    assert O.elu(np.array([-1.0]), 0.5)[0] == pytest.approx(0.5 * (math.exp(-1) - 1))


def test_mlp_forward_matches_torch_and_orientation():
    rng = np.random.default_rng(0)
    layers = [(rng.normal(size=(5, 4)), rng.normal(size=4)), (rng.normal(size=(4, 3)), rng.normal(size=3)),
              (rng.normal(size=(3, 2)), rng.normal(size=2))]
    x = rng.normal(size=(6, 5))
    out, hs = O.mlp_forward(x, layers, 1.0)
    xt = torch.tensor(x)
    for W, b in layers[:-1]:
        xt = torch.nn.functional.elu(torch.nn.functional.linear(xt, torch.tensor(W.T.copy()), torch.tensor(b)))
    xt = torch.nn.functional.linear(xt, torch.tensor(layers[-1][0].T.copy()), torch.tensor(layers[-1][1]))
    assert np.allclose(out, xt.numpy(), rtol=1e-13, atol=1e-13)
    assert len(hs) == 3 and hs[0].shape == (6, 5) and hs[2].shape == (6, 3)


def test_gaussian_log_prob_and_entropy_closed_forms():
    rng = np.random.default_rng(2)
    a, mu, ls = rng.normal(size=(5, 4)), rng.normal(size=(5, 4)), rng.normal(0, 0.3, size=4)
    want = scipy.stats.norm.logpdf(a, loc=mu, scale=np.exp(ls)).sum(axis=1)
    assert np.allclose(O.gaussian_log_prob(a, mu, ls), want, rtol=1e-13)
    assert O.gaussian_entropy(ls) == pytest.approx(scipy.stats.norm.entropy(scale=np.exp(ls)).sum(), rel=1e-13)
    # log_std = 0: per-dimension entropy of the unit normal, 1.4189385332...
    assert O.gaussian_entropy(np.zeros(4)) == pytest.approx(4 * 1.4189385332046727, rel=1e-15)
    # hand value: a = mu + sigma in 1-D with sigma = 2 -> -1/2 - ln 2 - ln sqrt(2 pi)
    assert O.gaussian_log_prob(np.array([[3.0]]), np.array([[1.0]]), np.array([math.log(2.0)]))[0] == \
        pytest.approx(-0.5 - math.log(2.0) - 0.5 * math.log(2 * math.pi))
    # the density integrates to one
    xs = np.linspace(-12, 12, 200001)[:, None]
    dens = np.exp(O.gaussian_log_prob(xs, np.array([[0.3]]), np.array([0.4])))
    assert np.trapezoid(dens, xs[:, 0]) == pytest.approx(1.0, abs=1e-9)


def test_act_composition():
    w = WL.TINY
    theta = WL.make_params(w)
    inp = WL.make_rollout_inputs(w)
    params = O.unpack_params(theta, w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)
    out = O.act(params, inp["obs_actor"][0], inp["obs_critic"][0], 1.0, seed=5, global_step=3)
    eps = O.gaussian_noise(5, 3, w.num_envs, w.num_actions)
    assert np.allclose(out["actions"], out["mu"] + eps)               # log_std = 0 -> sigma = 1
    assert np.allclose(out["logp"], scipy.stats.norm.logpdf(eps).sum(axis=1), rtol=1e-12)
    assert out["values"].shape == (w.num_envs,) and out["sigma"].shape == (w.num_actions,)


def test_unpack_layout_matches_workload_layout():
    w = WL.HUMANOID.scaled(8)
    theta = np.arange(w.num_params(), dtype=np.float64)
    p = O.unpack_params(theta, w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)
    for name, off, shape in WL.param_layout(w):
        net, leaf = name.split(".")
        if leaf == "log_std":
            got = p["log_std"]
        else:
            got = p[net][int(leaf[1:])][0 if leaf[0] == "W" else 1]
        assert got.shape == shape and got.ravel()[0] == off
    assert np.array_equal(O.pack_grads({"actor": p["actor"], "critic": p["critic"], "log_std": p["log_std"]}), theta)


# --------------------------------------------------------------------------------------
# GAE
# --------------------------------------------------------------------------------------
def gae_inputs(seed=0, T=9, N=5, p_done=0.25):
    rng = np.random.default_rng(seed)
    r, v, lv = rng.normal(size=(T, N)), rng.normal(size=(T, N)), rng.normal(size=N)
    d = (rng.random((T, N)) < p_done).astype(np.uint8)
    to = (d & (rng.random((T, N)) < 0.5)).astype(np.uint8)
    return r, v, d, to, lv


def test_gae_lambda_zero_is_td_residual():
    r, v, d, to, lv = gae_inputs()
    z = np.zeros_like(d)
    ret, adv = O.gae(r, v, z, z, lv, 0.9, 0.0)
    vnext = np.concatenate([v[1:], lv[None]])
    assert np.allclose(adv, r + 0.9 * vnext - v, rtol=1e-14)
    assert np.allclose(ret, adv + v)


def test_gae_lambda_one_is_discounted_return_minus_value():
    r, v, d, to, lv = gae_inputs(1)
    z = np.zeros_like(d)
    g = 0.93
    ret, adv = O.gae(r, v, z, z, lv, g, 1.0)
    T, N = r.shape
    for t in range(T):
        want = sum(g ** k * r[t + k] for k in range(T - t)) + g ** (T - t) * lv
        assert np.allclose(ret[t], want, rtol=1e-13)
        assert np.allclose(adv[t], want - v[t], rtol=1e-12, atol=1e-13)


def test_gae_gamma_zero_and_constant_reward_closed_form():
    r, v, d, to, lv = gae_inputs(2)
    ret, adv = O.gae(r, v, d, to, lv, 0.0, 0.7)
    assert np.allclose(adv, r - v)
    T, N, g, c = 12, 3, 0.9, 0.7
    z = np.zeros((T, N), dtype=np.uint8)
    lv = np.array([0.0, 1.0, -2.0])
    ret, _ = O.gae(np.full((T, N), c), np.zeros((T, N)), z, z, lv, g, 1.0)
    for t in range(T):
        assert np.allclose(ret[t], c * (1 - g ** (T - t)) / (1 - g) + g ** (T - t) * lv)


def test_gae_general_matches_brute_force_sum():
    """A_t = sum_k (gamma lam)^k [prod_{j<k} (1-d_{t+j})] delta_{t+k}, written as a double loop."""
    r, v, d, to, lv = gae_inputs(3, T=11, N=6)
    g, lam = 0.97, 0.9
    ret, adv = O.gae(r, v, d, to, lv, g, lam)
    T, N = r.shape
    vnext = np.concatenate([v[1:], lv[None]])
    delta = r + g * v * to + g * vnext * (1 - d) - v
    for n in range(N):
        for t in range(T):
            acc, alive = 0.0, 1.0
            for k in range(T - t):
                acc += (g * lam) ** k * alive * delta[t + k, n]
                alive *= 1.0 - d[t + k, n]
            assert adv[t, n] == pytest.approx(acc, rel=1e-12, abs=1e-13)
            assert ret[t, n] == pytest.approx(acc + v[t, n], rel=1e-12, abs=1e-13)


def test_gae_done_cuts_and_timeout_bootstraps():
    r, v, d, to, lv = gae_inputs(4)
    ones, z = np.ones_like(d), np.zeros_like(d)
    _, adv = O.gae(r, v, ones, z, lv, 0.99, 0.95)           # every step terminal, no time-outs
    assert np.allclose(adv, r - v)
    _, adv = O.gae(r, v, ones, ones, lv, 0.99, 0.95)        # every step a time-out
    assert np.allclose(adv, r + 0.99 * v - v)
    # two-pass formulation: fold gamma*V_t*timeout into the reward, then GAE without time-outs
    ret1, adv1 = O.gae(r, v, d, to, lv, 0.99, 0.95)
    ret2, adv2 = O.gae(r + 0.99 * v * to, v, d, z, lv, 0.99, 0.95)
    assert np.allclose(adv1, adv2, rtol=1e-14) and np.allclose(ret1, ret2, rtol=1e-14)
    # a done at (t, n) screens everything after it
    t0, n0 = 4, 2
    d2 = d.copy(); d2[t0, n0] = 1
    _, a = O.gae(r, v, d2, to, lv, 0.99, 0.95)
    r3, v3, lv3 = r.copy(), v.copy(), lv + 5.0
    r3[t0 + 1:, n0] += 3.0; v3[t0 + 1:, n0] -= 2.0
    _, b = O.gae(r3, v3, d2, to, lv3, 0.99, 0.95)
    assert np.allclose(a[:t0 + 1, n0], b[:t0 + 1, n0])
    assert not np.allclose(a[t0 + 1:, n0], b[t0 + 1:, n0])


def test_normalize_advantages():
    a = np.random.default_rng(5).normal(3.0, 2.0, size=(7, 11))
    n = O.normalize_advantages(a, 1e-8, True)
    assert np.allclose(n, (a - a.mean()) / (a.std(ddof=1) + 1e-8), rtol=1e-13)
    assert abs(n.mean()) < 1e-14 and n.std(ddof=1) == pytest.approx(1.0, rel=1e-7)
    b = O.normalize_advantages(a, 1e-8, False)
    assert np.allclose(b, (a - a.mean()) / (a.std(ddof=0) + 1e-8), rtol=1e-13)


# --------------------------------------------------------------------------------------
# losses and gradients
# --------------------------------------------------------------------------------------
def test_ratio_one_gives_minus_mean_advantage_and_zero_kl():
    theta, dims, batch = small_problem(0)
    adims, cdims, A = dims
    p = O.unpack_params(theta, adims, cdims, A)
    mu, _ = O.mlp_forward(batch["obs_actor"], p["actor"], 1.0)
    v, _ = O.mlp_forward(batch["obs_critic"], p["critic"], 1.0)
    batch.update(mu_old=mu, sigma_old=np.broadcast_to(np.exp(p["log_std"]), mu.shape).copy(),
                 logp_old=O.gaussian_log_prob(batch["actions"], mu, p["log_std"]), values_old=v[:, 0])
    st, g = O.ppo_loss_and_grads(p, batch, hp())
    assert np.allclose(st["ratio"], 1.0, rtol=1e-14)
    assert st["surrogate"] == pytest.approx(-batch["advantages"].mean(), rel=1e-13)
    assert st["kl"] == pytest.approx(0.0, abs=1e-15)
    # V == V_old: clipped and unclipped value losses coincide with the plain MSE
    assert st["value_loss"] == pytest.approx(((v[:, 0] - batch["returns"]) ** 2).mean(), rel=1e-13)
    # at ratio 1 the policy gradient is -mean(A grad logp): check it on log_std
    a, Ah = batch["actions"], batch["advantages"]
    want = (-(Ah[:, None]) * ((a - mu) ** 2 / np.exp(2 * p["log_std"]) - 1)).mean(axis=0) - 0.01
    assert np.allclose(g["log_std"], want, rtol=1e-12)


@pytest.mark.parametrize("seed,clipv,symmetric", [(0, True, False), (1, False, False), (2, True, True), (3, True, True)])
def test_losses_and_gradients_match_autograd(seed, clipv, symmetric):
    theta, dims, batch = small_problem(seed)
    adims, cdims, A = dims
    h = hp(use_clipped_value_loss=clipv, entropy_coef=0.03, value_coef=0.7, sym_coef=0.6)
    sym = rand_mirror(np.random.default_rng(seed), adims[0][0], cdims[0][0], A) if symmetric else None
    st, g = O.ppo_loss_and_grads(O.unpack_params(theta, adims, cdims, A), batch, h, sym)
    # both branches of both clips must be exercised, or the test proves nothing
    r = st["ratio"]
    assert (r < 0.8).any() and (r > 1.2).any() and ((r > 0.8) & (r < 1.2)).any()
    assert (np.abs(st["values"][:len(batch["values_old"])] - batch["values_old"]) > 0.2).any()
    tt = torch.tensor(theta, dtype=torch.float64, requires_grad=True)
    L, parts = torch_loss(tt, dims, batch, h, sym)
    L.backward()
    assert st["loss"] == pytest.approx(L.item(), rel=1e-12)
    for k in ("surrogate", "value_loss", "entropy", "kl", "sym_loss"):
        assert st[k] == pytest.approx(parts[k].item(), rel=1e-11, abs=1e-14), k
    assert np.allclose(O.pack_grads(g), tt.grad.numpy(), rtol=1e-10, atol=1e-13)


def test_gradients_match_central_finite_differences():
    theta, dims, batch = small_problem(7, B=24)
    adims, cdims, A = dims
    h = hp()
    # no mirror here: the symmetry target carries a stop-gradient, so the analytic gradient is
    # not the derivative of the scalar loss (autograd with detach() pins that term instead)
    sym = None
    loss = lambda th: O.ppo_loss_and_grads(O.unpack_params(th, adims, cdims, A), batch, h, sym)[0]["loss"]
    g = O.pack_grads(O.ppo_loss_and_grads(O.unpack_params(theta, adims, cdims, A), batch, h, sym)[1])
    rng = np.random.default_rng(1)
    idx = np.unique(np.concatenate([rng.integers(0, theta.size, 60), np.arange(theta.size - 5, theta.size)]))
    eps = 1e-6
    for i in idx:
        e = np.zeros_like(theta); e[i] = eps
        fd = (loss(theta + e) - loss(theta - e)) / (2 * eps)
        assert g[i] == pytest.approx(fd, rel=2e-5, abs=1e-8), i


def test_symmetry_identity_mirror_and_equivariant_net():
    theta, dims, batch = small_problem(3)
    adims, cdims, A = dims
    h = hp()
    ident = dict(obs_perm=np.arange(adims[0][0]), obs_sign=np.ones(adims[0][0]),
                 cobs_perm=np.arange(cdims[0][0]), cobs_sign=np.ones(cdims[0][0]),
                 act_perm=np.arange(A), act_sign=np.ones(A))
    p = O.unpack_params(theta, adims, cdims, A)
    s0, g0 = O.ppo_loss_and_grads(p, batch, h, None)
    s1, g1 = O.ppo_loss_and_grads(p, batch, h, ident)
    assert s1["sym_loss"] == 0.0
    for k in ("loss", "surrogate", "value_loss", "kl"):
        assert s1[k] == pytest.approx(s0[k], rel=1e-13)
    assert np.allclose(O.pack_grads(g1), O.pack_grads(g0), rtol=1e-12, atol=1e-15)
    # an actor that is equivariant by construction: one linear layer with S_a^T W^T S_o = W^T
    rng = np.random.default_rng(0)
    Da = 6
    sym = rand_mirror(rng, Da, cdims[0][0], A)
    So = np.zeros((Da, Da)); So[np.arange(Da), sym["obs_perm"]] = sym["obs_sign"]
    Sa = np.zeros((A, A)); Sa[np.arange(A), sym["act_perm"]] = sym["act_sign"]
    W0 = rng.normal(size=(Da, A))
    W = 0.5 * (W0 + So.T @ W0 @ Sa.T)        # then mu(S_o o) = S_a mu(o) for a bias-free linear map
    params = {"actor": [(W, np.zeros(A))], "critic": p["critic"], "log_std": np.zeros(A)}
    b2 = dict(batch); b2["obs_actor"] = rng.normal(size=(batch["obs_actor"].shape[0], Da))
    s2, _ = O.ppo_loss_and_grads(params, b2, h, sym)
    assert s2["sym_loss"] == pytest.approx(0.0, abs=1e-25)
    assert np.allclose(O.mirror(O.mirror(b2["obs_actor"], sym["obs_perm"], sym["obs_sign"]),
                                sym["obs_perm"], sym["obs_sign"]), b2["obs_actor"])


def test_kl_hand_values():
    # 1-D: KL(N(0,1) || N(1,2)) = ln 2 + (1 + 1) / 8 - 1/2
    theta, dims, batch = small_problem(0, B=1, A=1, Da=2, hidden_a=(2,))
    adims, cdims, A = dims
    p = O.unpack_params(theta, adims, cdims, A)
    p["log_std"] = np.array([math.log(2.0)])
    mu, _ = O.mlp_forward(batch["obs_actor"], p["actor"], 1.0)
    batch.update(mu_old=mu - 1.0, sigma_old=np.ones((1, 1)))
    st, _ = O.ppo_loss_and_grads(p, batch, hp())
    assert st["kl"] == pytest.approx(math.log(2.0) + 2.0 / 8.0 - 0.5, rel=1e-13)


# --------------------------------------------------------------------------------------
# optimiser
# --------------------------------------------------------------------------------------
def test_clip_coefficient():
    assert O.clip_coefficient(0.5, 1.0) == 1.0
    assert O.clip_coefficient(4.0, 1.0) == pytest.approx(1.0 / (4.0 + 1e-6))
    g = torch.tensor([3.0, 4.0], dtype=torch.float64, requires_grad=True)
    g.grad = g.detach().clone()
    torch.nn.utils.clip_grad_norm_([g], 1.0)
    assert np.allclose(g.grad.numpy(), np.array([3.0, 4.0]) * O.clip_coefficient(5.0, 1.0), rtol=1e-14)


def test_adaptive_lr_rule():
    h = hp()
    assert O.adaptive_lr(1e-3, 0.0, h) == pytest.approx(1.5e-3)
    assert O.adaptive_lr(1e-3, 0.0025, h) == pytest.approx(1.5e-3)      # d/4 < d/2
    assert O.adaptive_lr(1e-3, 0.01, h) == 1e-3                          # d: hold
    assert O.adaptive_lr(1e-3, 0.03, h) == pytest.approx(1e-3 / 1.5)     # 3d > 2d
    assert O.adaptive_lr(1.2e-5, 0.03, h) == 1e-5                        # clamp below
    assert O.adaptive_lr(9e-3, 0.0, h) == 1e-2                           # clamp above
    assert O.adaptive_lr(1e-3, 0.03, hp(adaptive_lr=False)) == 1e-3


def test_adam_first_step_by_hand_and_against_torch():
    g = np.array([0.5, -2.0, 1e-3, 0.0])
    th = np.array([1.0, 2.0, 3.0, 4.0])
    t1, m, v = O.adam_step(th, g, np.zeros(4), np.zeros(4), 1, 0.01, 0.9, 0.999, 1e-8)
    # first step: m_hat = g, v_hat = g^2 -> theta - lr * g / (|g| + eps)
    assert np.allclose(t1, th - 0.01 * g / (np.abs(g) + 1e-8), rtol=1e-15)
    assert np.allclose(m, 0.1 * g) and np.allclose(v, 0.001 * g * g)
    rng = np.random.default_rng(0)
    p = torch.tensor(th, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=0.01, betas=(0.9, 0.999), eps=1e-8)
    th2, m, v = th.copy(), np.zeros(4), np.zeros(4)
    for s in range(1, 8):
        gs = rng.normal(size=4)
        p.grad = torch.tensor(gs)
        opt.step()
        th2, m, v = O.adam_step(th2, gs, m, v, s, 0.01, 0.9, 0.999, 1e-8)
        assert np.allclose(th2, p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_update_loop_matches_torch_reference_loop():
    """ppo_update's ordering -- permutation chunks, lr adapted before the step, clip, Adam,
    state carried across minibatches and epochs -- against an autograd + torch.optim loop."""
    w = WL.TINY.scaled(16, epochs=2, minibatches=2)
    dims = (w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)
    theta0 = WL.make_params(w).astype(np.float64)
    inp = WL.make_rollout_inputs(w)
    storage = O.rollout(theta0, dims, inp, w, seed=w.seed)
    state = O.OptimState(theta0, w.lr)
    steps = O.ppo_update(state, dims, storage, w, seed=w.seed, iteration=0)
    assert len(steps) == 4 and state.step == 4

    p = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=w.lr)
    lr = w.lr
    B = w.batch
    for e in range(2):
        perm = O.feistel_permutation(w.seed, 0, e, B)
        for k in range(2):
            rows = perm[k * (B // 2):(k + 1) * (B // 2)]
            batch = O.gather_minibatch(storage, rows)
            opt.zero_grad()
            L, parts = torch_loss(p, dims, batch, w)
            L.backward()
            kl = parts["kl"].item()
            if kl > 2 * w.desired_kl:
                lr = max(1e-5, lr / 1.5)
            elif kl < w.desired_kl / 2:
                lr = min(1e-2, lr * 1.5)
            for gr in opt.param_groups:
                gr["lr"] = lr
            torch.nn.utils.clip_grad_norm_([p], w.max_grad_norm)
            opt.step()
            st = steps[e * 2 + k]
            assert st["loss"] == pytest.approx(L.item(), rel=1e-9)
            assert st["lr"] == pytest.approx(lr, rel=1e-15)
    assert np.allclose(state.theta, p.detach().numpy(), rtol=1e-9, atol=1e-12)
    # every transition is visited exactly once per epoch
    assert np.array_equal(np.sort(O.feistel_permutation(w.seed, 0, 0, B)), np.arange(B))


def test_rollout_storage_shapes_and_normalised_advantages():
    w = WL.TINY
    dims = (w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)
    st = O.rollout(WL.make_params(w), dims, WL.make_rollout_inputs(w), w, seed=0)
    T, N, A = w.num_steps, w.num_envs, w.num_actions
    assert st["actions"].shape == (T, N, A) and st["sigma"].shape == (T, A)
    assert st["values"].shape == (T, N) and st["last_values"].shape == (N,)
    a = st["advantages"]
    assert abs(a.mean()) < 1e-12 and a.std(ddof=1) == pytest.approx(1.0, rel=1e-6)
    assert np.allclose(st["returns"], st["advantages_raw"] + st["values"])


# --------------------------------------------------------------------------------------
# distillation (paper, "Algorithms": behaviour cloning similar to DAgger)
# --------------------------------------------------------------------------------------
def _distill_problem(seed=3, B=30):
    theta, dims, batch = small_problem(seed, B=B)
    rng = np.random.default_rng(seed + 100)
    target = rng.normal(size=batch["actions"].shape)
    return theta, dims, batch["obs_actor"], target


def test_distill_loss_matches_torch_mse_and_autograd():
    theta, dims, obs, target = _distill_problem()
    adims, cdims, A = dims
    h = hp()
    stats, grads = O.distill_loss_and_grads(O.unpack_params(theta, adims, cdims, A), obs, target, h)
    p = torch.tensor(theta, dtype=torch.float64, requires_grad=True)
    off, x = 0, torch.as_tensor(obs, dtype=torch.float64)
    for li, (fi, fo) in enumerate(adims):
        W = p[off:off + fi * fo].reshape(fi, fo); off += fi * fo
        b = p[off:off + fo]; off += fo
        x = x @ W + b
        if li < len(adims) - 1:
            x = torch.nn.functional.elu(x, alpha=h.elu_alpha)
    L = torch.nn.functional.mse_loss(x, torch.as_tensor(target, dtype=torch.float64))
    L.backward()
    assert stats["loss"] == pytest.approx(L.item(), rel=1e-12)
    g = O.pack_grads(grads)
    assert np.allclose(g, p.grad.numpy(), rtol=1e-9, atol=1e-13)
    # log_std and the critic take no part
    n_actor = sum(i * o + o for i, o in adims)
    assert np.all(g[n_actor:] == 0.0)


def test_distill_gradient_matches_central_finite_differences():
    theta, dims, obs, target = _distill_problem(5, B=16)
    adims, cdims, A = dims
    h = hp()
    loss = lambda th: O.distill_loss_and_grads(O.unpack_params(th, adims, cdims, A), obs, target, h)[0]["loss"]
    g = O.pack_grads(O.distill_loss_and_grads(O.unpack_params(theta, adims, cdims, A), obs, target, h)[1])
    n_actor = sum(i * o + o for i, o in adims)
    rng = np.random.default_rng(2)
    for i in rng.integers(0, n_actor, 40):
        e = np.zeros_like(theta); e[i] = 1e-6
        fd = (loss(theta + e) - loss(theta - e)) / 2e-6
        assert g[i] == pytest.approx(fd, rel=2e-5, abs=1e-9), i


def test_distill_zero_when_the_student_already_matches_and_quadratic_in_the_error():
    theta, dims, obs, _ = _distill_problem(9)
    adims, cdims, A = dims
    h = hp()
    params = O.unpack_params(theta, adims, cdims, A)
    mu, _ = O.mlp_forward(obs, params["actor"], h.elu_alpha)
    stats, grads = O.distill_loss_and_grads(params, obs, mu, h)
    assert stats["loss"] == 0.0 and np.all(O.pack_grads(grads) == 0.0)
    d = np.random.default_rng(0).normal(size=mu.shape)
    l1 = O.distill_loss_and_grads(params, obs, mu + d, h)[0]["loss"]
    l2 = O.distill_loss_and_grads(params, obs, mu + 2 * d, h)[0]["loss"]
    assert l1 == pytest.approx((d ** 2).mean(), rel=1e-12) and l2 == pytest.approx(4 * l1, rel=1e-12)


def test_distill_update_loop_matches_torch_reference_loop():
    """Same shuffle and chunks as the PPO update, clip, Adam with a fixed learning rate."""
    w = WL.TINY.scaled(16, epochs=2, minibatches=2)
    dims = (w.layer_dims("actor"), w.layer_dims("critic"), w.num_actions)
    theta0 = WL.make_params(w).astype(np.float64)
    inp = WL.make_rollout_inputs(w)
    T, N, A = w.num_steps, w.num_envs, w.num_actions
    expert = np.random.default_rng(4).normal(size=(T, N, A))
    state = O.OptimState(theta0, w.lr)
    steps = O.distill_update(state, dims, inp["obs_actor"], expert, w, seed=w.seed, iteration=3)
    assert len(steps) == 4 and state.step == 4 and state.lr == w.lr

    adims = dims[0]
    p = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=w.lr)
    B = T * N
    obs = torch.as_tensor(inp["obs_actor"][:T].reshape(B, -1), dtype=torch.float64)
    tgt = torch.as_tensor(expert.reshape(B, A))
    for e in range(2):
        perm = O.feistel_permutation(w.seed, 3, e, B)
        for k in range(2):
            rows = torch.as_tensor(perm[k * (B // 2):(k + 1) * (B // 2)].astype(np.int64))
            opt.zero_grad()
            off, x = 0, obs[rows]
            for li, (fi, fo) in enumerate(adims):
                W = p[off:off + fi * fo].reshape(fi, fo); off += fi * fo
                b = p[off:off + fo]; off += fo
                x = x @ W + b
                if li < len(adims) - 1:
                    x = torch.nn.functional.elu(x, alpha=w.elu_alpha)
            L = torch.nn.functional.mse_loss(x, tgt[rows])
            L.backward()
            torch.nn.utils.clip_grad_norm_([p], w.max_grad_norm)
            opt.step()
            assert steps[e * 2 + k]["loss"] == pytest.approx(L.item(), rel=1e-9)
    assert np.allclose(state.theta, p.detach().numpy(), rtol=1e-9, atol=1e-12)


# --------------------------------------------------------------------------------------
# random network distillation on a state subset (paper, "Auxiliary Techniques")
# --------------------------------------------------------------------------------------
def _rnd_problem(seed=11, B=28, D=9, idx=(7, 1, 4, 2), hidden=(6, 5), E=3):
    rng = np.random.default_rng(seed)
    dims = list(zip([len(idx), *hidden], [*hidden, E]))
    P = sum(i * o + o for i, o in dims)
    return rng.normal(0, 0.6, P), rng.normal(0, 0.6, P), dims, rng.normal(size=(B, D)), np.array(idx)


def _torch_mlp(p, dims, x, alpha):
    off = 0
    for li, (fi, fo) in enumerate(dims):
        W = p[off:off + fi * fo].reshape(fi, fo); off += fi * fo
        b = p[off:off + fo]; off += fo
        x = x @ W + b
        if li < len(dims) - 1:
            x = torch.nn.functional.elu(x, alpha=alpha)
    return x


def test_rnd_reward_and_gradient_match_torch():
    tf, tg, dims, obs, idx = _rnd_problem()
    r, f, g, _ = O.rnd_reward(tf, tg, dims, obs, idx, 1.0)
    p = torch.tensor(tf, dtype=torch.float64, requires_grad=True)
    s = torch.as_tensor(obs[:, idx])
    ft = _torch_mlp(p, dims, s, 1.0)
    gt = _torch_mlp(torch.as_tensor(tg), dims, s, 1.0)
    rt = ((ft - gt) ** 2).mean(dim=1)
    assert np.allclose(r, rt.detach().numpy(), rtol=1e-12, atol=1e-15)
    L, grad = O.rnd_loss_and_grads(tf, tg, dims, obs, idx, 1.0)
    rt.mean().backward()
    assert L == pytest.approx(rt.mean().item(), rel=1e-12)
    assert np.allclose(grad, p.grad.numpy(), rtol=1e-9, atol=1e-13)


def test_rnd_reads_only_the_subset_and_vanishes_for_equal_nets():
    tf, tg, dims, obs, idx = _rnd_problem(13)
    r0 = O.rnd_reward(tf, tg, dims, obs, idx, 1.0)[0]
    other = [c for c in range(obs.shape[1]) if c not in idx]
    obs2 = obs.copy(); obs2[:, other] += 5.0               # columns outside the subset do not matter
    assert np.array_equal(O.rnd_reward(tf, tg, dims, obs2, idx, 1.0)[0], r0)
    obs3 = obs.copy(); obs3[:, idx[0]] += 0.5              # one inside does
    assert not np.allclose(O.rnd_reward(tf, tg, dims, obs3, idx, 1.0)[0], r0)
    assert np.all(r0 >= 0.0)
    L, grad = O.rnd_loss_and_grads(tf, tf, dims, obs, idx, 1.0)     # predictor == target
    assert L == 0.0 and np.all(grad == 0.0)


def test_rnd_gradient_matches_central_finite_differences():
    tf, tg, dims, obs, idx = _rnd_problem(17, B=12)
    _, grad = O.rnd_loss_and_grads(tf, tg, dims, obs, idx, 1.0)
    for i in np.random.default_rng(1).integers(0, tf.size, 30):
        e = np.zeros_like(tf); e[i] = 1e-6
        fd = (O.rnd_loss_and_grads(tf + e, tg, dims, obs, idx, 1.0)[0] - O.rnd_loss_and_grads(tf - e, tg, dims, obs, idx, 1.0)[0]) / 2e-6
        assert grad[i] == pytest.approx(fd, rel=2e-5, abs=1e-9), i


def test_rnd_update_loop_matches_torch_reference_loop():
    tf, tg, dims, obs, idx = _rnd_problem(19, B=32)
    h = hp(epochs=2, minibatches=4, lr=3e-3)
    state = O.OptimState(tf.copy(), h.lr)
    steps = O.rnd_update(state, tg, dims, obs, idx, h, seed=5, iteration=2)
    assert len(steps) == 8 and state.step == 8
    p = torch.tensor(tf, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=h.lr)
    s_all = torch.as_tensor(obs[:, idx]); tgt = torch.as_tensor(tg)
    k = 0
    for e in range(2):
        perm = O.feistel_permutation(5, 2, e, 32)
        for c in range(4):
            rows = torch.as_tensor(perm[c * 8:(c + 1) * 8].astype(np.int64))
            opt.zero_grad()
            L = ((_torch_mlp(p, dims, s_all[rows], 1.0) - _torch_mlp(tgt, dims, s_all[rows], 1.0)) ** 2).mean()
            L.backward(); opt.step()
            assert steps[k]["loss"] == pytest.approx(L.item(), rel=1e-9); k += 1
    assert np.allclose(state.theta, p.detach().numpy(), rtol=1e-9, atol=1e-12)
