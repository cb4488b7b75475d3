"""GPU parity of random network distillation on a state subset (rslrl_rnd_*) against the FP64 oracle:
intrinsic reward per row, reward mixing, the first predictor step (loss, gradient, parameters) and the whole
epoch x minibatch training loop on the same keyed minibatches.

The CUDA path computes in FP32; tolerance 1e-4 (relative to the element plus the array's rms), as for
the FP32 mode of the PPO update.  The intrinsic reward is a mean of squared differences of two nets that start
far apart (the target is drawn four times wider), so it carries no cancellation at these inputs."""
from types import SimpleNamespace

import numpy as np
import pytest

from oracle import ppo_oracle as O
from paper_2509_10771_b200 import workloads as WL

from parity_utils import assert_close, rel_l2

pytestmark = pytest.mark.gpu

CASES = {
    # name: (workload for the observation recipe, rows, RND net keywords, minibatches, epochs)
    "tiny": (WL.TINY, 8 * 64, dict(num_idx=5, hidden=(16,), embed_dim=3), 2, 1),
    "flat": (WL.FLAT, 24 * 300, dict(num_idx=12, hidden=(128, 64), embed_dim=32), 4, 2),
    "rough": (WL.ROUGH, 24 * 257, dict(num_idx=48, hidden=(256, 128, 64), embed_dim=50), 8, 2),   # ragged rows
}


def _setup(case, lr=1e-3, precision=0):
    import torch
    from paper_2509_10771_b200 import binding
    w, rows, kw, mbs, epochs = CASES[case]
    envs = rows // w.num_steps
    ws = w.scaled(envs)
    obs = WL.make_rollout_inputs(ws)["obs_actor"][:w.num_steps].reshape(rows, w.actor_obs_dim)
    setup = WL.make_rnd_setup(ws, **kw)
    rnd = binding.Rnd(w.actor_obs_dim, setup["idx"], setup["hidden"], setup["embed_dim"], max_rows=rows, lr=lr, max_batch=rows,
                      precision=precision)
    rnd.set_params(setup["predictor"], setup["target"])
    d_obs = torch.from_numpy(obs).to("cuda")
    return w, rows, setup, rnd, obs, d_obs, mbs, epochs


@pytest.mark.parametrize("case", ["tiny", "flat", "rough"])
def test_intrinsic_reward_matches_oracle(case):
    import torch
    w, rows, setup, rnd, obs, d_obs, _, _ = _setup(case)
    ref, _, _, _ = O.rnd_reward(setup["predictor"], setup["target"], setup["dims"], obs, setup["idx"], 1.0)
    rng = np.random.default_rng(1)
    r_ext = rng.standard_normal(rows).astype(np.float32)
    d_rew = torch.from_numpy(r_ext.copy()).to("cuda")
    d_int = torch.full((rows,), -1.0, device="cuda")
    rnd.reward(d_obs, rows, w.actor_obs_dim, weight=0.25, d_rewards_inout=d_rew, d_r_int_out=d_int)
    torch.cuda.synchronize()
    assert_close(d_int.cpu().numpy(), ref, 1e-4, "r_int")
    assert_close(d_rew.cpu().numpy(), r_ext.astype(np.float64) + 0.25 * ref, 1e-4, "mixed reward")
    # a prefix of the rows, and a wider row stride, give the same rewards
    wide = torch.zeros((rows, w.actor_obs_dim + 5), device="cuda")
    wide[:, :w.actor_obs_dim] = d_obs
    d_int2 = torch.full((rows,), -1.0, device="cuda")
    rnd.reward(wide, rows // 3, w.actor_obs_dim + 5, d_r_int_out=d_int2)
    torch.cuda.synchronize()
    assert torch.equal(d_int2[:rows // 3], d_int[:rows // 3])
    assert bool((d_int2[rows // 3:] == -1.0).all())
    rnd.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough"])
def test_reward_and_first_step_match_oracle_tf32(case):
    """RSLRL_TF32: the products of both nets see TF32 operands (11 significant bits).  The reward of untrained nets and
    the loss at the mode's tolerance 5e-3, the gradient at twice that per element and at 5e-3 in relative L2; the
    parameters after Adam's first step (lr * sign(g)) as in the FP32 test."""
    import torch
    w, rows, setup, rnd, obs, d_obs, mbs, epochs = _setup(case, precision=WL.PRECISION_TF32)
    ref_r, _, _, _ = O.rnd_reward(setup["predictor"], setup["target"], setup["dims"], obs, setup["idx"], 1.0)
    d_int = torch.full((rows,), -1.0, device="cuda")
    rnd.reward(d_obs, rows, w.actor_obs_dim, d_r_int_out=d_int)
    torch.cuda.synchronize()
    got_r = d_int.cpu().numpy()
    assert_close(got_r, ref_r, 5e-3, "r_int")
    fp32 = _setup(case)
    d_int32 = torch.full((rows,), -1.0, device="cuda")
    fp32[3].reward(d_obs, rows, w.actor_obs_dim, d_r_int_out=d_int32)
    torch.cuda.synchronize()
    assert not np.array_equal(got_r, d_int32.cpu().numpy())          # the tensor cores did see TF32 operands
    fp32[3].destroy()
    hp = SimpleNamespace(epochs=epochs, minibatches=mbs, elu_alpha=1.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8)
    out = rnd.update(d_obs, rows, w.actor_obs_dim, epochs, mbs, seed=7, iteration=3, max_steps=1)
    state = O.OptimState(setup["predictor"], 1e-3)
    ref = O.rnd_update(state, setup["target"], setup["dims"], obs, setup["idx"], hp, seed=7, iteration=3, max_steps=1)
    assert_close(out["first_loss"], ref[0]["loss"], 5e-3, "loss")
    g = rnd.get_grads()
    assert_close(g, ref[0]["grad"], 1e-2, "grad")
    assert rel_l2(g, ref[0]["grad"]) < 5e-3
    assert_close(rnd.get_params(), state.theta, 1e-4, "params", max_outlier_frac=2e-2, outlier_abs=2.05e-3)
    rnd.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough"])
def test_first_predictor_step_matches_oracle(case):
    w, rows, setup, rnd, obs, d_obs, mbs, epochs = _setup(case)
    hp = SimpleNamespace(epochs=epochs, minibatches=mbs, elu_alpha=1.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8)
    out = rnd.update(d_obs, rows, w.actor_obs_dim, epochs, mbs, seed=7, iteration=3, max_steps=1)
    state = O.OptimState(setup["predictor"], 1e-3)
    ref = O.rnd_update(state, setup["target"], setup["dims"], obs, setup["idx"], hp, seed=7, iteration=3, max_steps=1)
    assert_close(out["first_loss"], ref[0]["loss"], 1e-4, "loss")
    assert_close(rnd.get_grads(), ref[0]["grad"], 1e-4, "grad")
    # Adam's first step moves every entry by lr * sign(g): entries whose gradient is zero to rounding may differ
    assert_close(rnd.get_params(), state.theta, 1e-4, "params", max_outlier_frac=2e-3, outlier_abs=2.05e-3)
    rnd.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough"])
def test_predictor_training_tracks_oracle(case):
    import torch
    w, rows, setup, rnd, obs, d_obs, mbs, epochs = _setup(case)
    hp = SimpleNamespace(epochs=epochs, minibatches=mbs, elu_alpha=1.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8)
    out = rnd.update(d_obs, rows, w.actor_obs_dim, epochs, mbs, seed=11, iteration=0)
    state = O.OptimState(setup["predictor"], 1e-3)
    ref = O.rnd_update(state, setup["target"], setup["dims"], obs, setup["idx"], hp, seed=11, iteration=0)
    assert len(ref) == epochs * mbs
    assert_close(out["first_loss"], ref[0]["loss"], 1e-4, "first loss")
    assert_close(out["mean_loss"], float(np.mean([r["loss"] for r in ref])), 1e-4, "mean loss")
    assert rel_l2(rnd.get_params(), state.theta) < 1e-4
    assert rel_l2(rnd.get_grads(), ref[-1]["grad"]) < 1e-3
    # training lowers the intrinsic reward of the rows it was trained on
    d_int = torch.empty((rows,), device="cuda")
    rnd.reward(d_obs, rows, w.actor_obs_dim, d_r_int_out=d_int)
    before, _, _, _ = O.rnd_reward(setup["predictor"], setup["target"], setup["dims"], obs, setup["idx"], 1.0)
    after, _, _, _ = O.rnd_reward(state.theta, setup["target"], setup["dims"], obs, setup["idx"], 1.0)
    assert after.mean() < before.mean()
    assert_close(d_int.cpu().numpy(), after, 2e-4, "r_int after training")
    rnd.destroy()


def test_rnd_argument_checks():
    import torch
    from paper_2509_10771_b200 import binding
    with pytest.raises(binding.RslrlError) as e:
        binding.Rnd(8, [0, 9], (4,), 2, max_rows=16)                # index out of range
    assert e.value.status == 1
    rnd = binding.Rnd(8, [0, 3, 5], (4,), 2, max_rows=16)
    n = rnd.num_params
    assert n == 3 * 4 + 4 + 4 * 2 + 2
    rnd.set_params(np.zeros(n, np.float32), np.ones(n, np.float32))
    d_obs = torch.zeros((64, 8), device="cuda")
    with pytest.raises(binding.RslrlError) as e:
        rnd.reward(d_obs, 17, 8, d_r_int_out=torch.zeros(17, device="cuda"))
    assert e.value.status == 5
    with pytest.raises(binding.RslrlError) as e:
        rnd.update(d_obs, 30, 8, 1, 4, seed=0, iteration=0)          # 30 rows do not divide into 4
    assert e.value.status == 2
    with pytest.raises(binding.RslrlError) as e:
        rnd.update(d_obs, 64, 8, 1, 2, seed=0, iteration=0)          # 32 rows per minibatch > max_rows
    assert e.value.status == 5
    small = binding.Rnd(8, [0, 3, 5], (4,), 2, max_rows=16, max_batch=32, max_epochs=2, max_minibatches=4)
    small.set_params(np.zeros(n, np.float32), np.ones(n, np.float32))
    for batch, epochs, mbs in ((64, 1, 4), (32, 3, 4), (32, 1, 8)):  # beyond max_batch, max_epochs, max_minibatches
        with pytest.raises(binding.RslrlError) as e:
            small.update(d_obs, batch, 8, epochs, mbs, seed=0, iteration=0)
        assert e.value.status == 5
    free0 = torch.cuda.mem_get_info()[0]
    small.update(d_obs, 32, 8, 2, 4, seed=0, iteration=0)            # at the limits: runs, and allocates nothing
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    small.destroy()
    with pytest.raises(binding.RslrlError) as e:
        binding.Rnd(8, [0, 3, 5], (4,), 2, max_rows=16, max_epochs=0)
    assert e.value.status == 1
    with pytest.raises(binding.RslrlError) as e:
        rnd.set_params(np.zeros(n + 1, np.float32), np.zeros(n + 1, np.float32))
    assert e.value.status == 2
    # zero observations, zero predictor, target of ones: g = bias path only, reward is finite and equal on all rows
    d_int = torch.empty(16, device="cuda")
    rnd.reward(d_obs, 16, 8, d_r_int_out=d_int)
    torch.cuda.synchronize()
    v = d_int.cpu().numpy()
    assert np.all(v == v[0]) and np.isfinite(v[0]) and v[0] > 0
    rnd.destroy()


def test_intrinsic_reward_enters_gae_like_the_oracle():
    """The place of the reward in the learn iteration: r_t + w * r_int(o_t) is what record_step stores and what
    the advantage estimator sees.  The oracle's rollout runs on the mixed rewards computed by the oracle."""
    import torch
    from paper_2509_10771_b200 import binding
    from parity_utils import oracle_rollout, read_storage
    w = WL.ROUGH.scaled(300, minibatches=4)
    T, N, Da = w.num_steps, w.num_envs, w.actor_obs_dim
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    setup = WL.make_rnd_setup(w, num_idx=20, hidden=(64, 32), embed_dim=16)
    weight = 0.05
    ctx = binding.Context(w, precision=WL.PRECISION_FP32)
    ctx.set_params(theta)
    rnd = binding.Rnd(Da, setup["idx"], setup["hidden"], setup["embed_dim"], max_rows=N, max_batch=N)
    rnd.set_params(setup["predictor"], setup["target"])
    dev = torch.device("cuda")
    oa = torch.from_numpy(inputs["obs_actor"]).to(dev)
    rew = torch.from_numpy(inputs["rewards"]).to(dev)
    dn = torch.from_numpy(inputs["dones"]).to(dev)
    to = torch.from_numpy(inputs["timeouts"]).to(dev)
    for t in range(T):
        ctx.act(oa[t])
        r = rew[t].clone()
        rnd.reward(oa[t], N, Da, weight=weight, d_rewards_inout=r)
        ctx.record_step(r, dn[t], to[t])
    ctx.gae(oa[T])
    torch.cuda.synchronize()
    got = read_storage(ctx, w)
    r_int, _, _, _ = O.rnd_reward(setup["predictor"], setup["target"], setup["dims"],
                                  inputs["obs_actor"][:T].reshape(T * N, Da), setup["idx"], 1.0)
    mixed = dict(inputs)
    mixed["rewards"] = inputs["rewards"].astype(np.float64) + weight * r_int.reshape(T, N)
    want = oracle_rollout(w, theta, mixed)
    assert float(np.abs(weight * r_int).mean()) > 0.1 * float(np.abs(inputs["rewards"]).mean())   # the term matters here
    assert_close(got["rewards"], mixed["rewards"], 1e-4, "rewards")
    for k in ("returns", "advantages"):
        assert_close(got[k], want[k], 1e-4, k)
    rnd.destroy()
    ctx.destroy()


def test_full_size_reward_and_first_step_match_oracle():
    """The size the benchmark's distillation-reward task runs: 98,304 rows of rough_terrain observations, 48 selected
    entries, nets 48-256-128-64-32; the reward of every row and the first predictor step (24,576-row minibatch)."""
    import torch
    from paper_2509_10771_b200 import binding
    w = WL.ROUGH
    T, N, Da = w.num_steps, w.num_envs, w.actor_obs_dim
    B = T * N
    setup = WL.make_rnd_setup(w, num_idx=48, hidden=(256, 128, 64), embed_dim=32)
    obs = WL.make_rollout_inputs(w)["obs_actor"][:T].reshape(B, Da)
    d_obs = torch.from_numpy(obs).to("cuda")
    rnd = binding.Rnd(Da, setup["idx"], setup["hidden"], setup["embed_dim"], max_rows=B, max_batch=B)
    rnd.set_params(setup["predictor"], setup["target"])
    d_int = torch.empty(B, device="cuda")
    rnd.reward(d_obs, B, Da, d_r_int_out=d_int)
    torch.cuda.synchronize()
    ref, _, _, _ = O.rnd_reward(setup["predictor"], setup["target"], setup["dims"], obs, setup["idx"], 1.0)
    assert_close(d_int.cpu().numpy(), ref, 1e-4, "r_int")
    hp = SimpleNamespace(epochs=w.epochs, minibatches=w.minibatches, elu_alpha=1.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8)
    out = rnd.update(d_obs, B, Da, w.epochs, w.minibatches, seed=w.seed, iteration=0, max_steps=1)
    state = O.OptimState(setup["predictor"], 1e-3)
    r = O.rnd_update(state, setup["target"], setup["dims"], obs, setup["idx"], hp, seed=w.seed, iteration=0, max_steps=1)
    assert_close(out["first_loss"], r[0]["loss"], 1e-4, "loss")
    assert_close(rnd.get_grads(), r[0]["grad"], 1e-4, "grad")
    rnd.destroy()


def test_degenerate_sizes():
    """No rows, one row, one minibatch of an odd number of rows, a single selected entry and a one-wide embedding."""
    import torch
    from paper_2509_10771_b200 import binding
    rng = np.random.default_rng(3)
    obs = rng.standard_normal((37, 6)).astype(np.float32)
    idx = np.array([4], dtype=np.int32)
    dims = WL.rnd_layer_dims(1, (5,), 1)
    n = sum(i * o + o for i, o in dims)
    f, g = (rng.standard_normal(n) * 0.7).astype(np.float32), (rng.standard_normal(n) * 0.7).astype(np.float32)
    rnd = binding.Rnd(6, idx, (5,), 1, max_rows=37, lr=1e-2)
    rnd.set_params(f, g)
    d_obs = torch.from_numpy(obs).to("cuda")
    d_int = torch.full((37,), -1.0, device="cuda")
    rnd.reward(d_obs, 0, 6, d_r_int_out=d_int)                      # nothing to do, nothing written
    rnd.reward(d_obs, 1, 6, d_r_int_out=d_int)
    torch.cuda.synchronize()
    ref, _, _, _ = O.rnd_reward(f, g, dims, obs, idx, 1.0)
    got = d_int.cpu().numpy()
    assert_close(got[:1], ref[:1], 1e-4, "one row") ; assert np.all(got[1:] == -1.0)
    hp = SimpleNamespace(epochs=3, minibatches=1, elu_alpha=1.0, adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8)
    out = rnd.update(d_obs, 37, 6, 3, 1, seed=5, iteration=2)
    state = O.OptimState(f, 1e-2)
    r = O.rnd_update(state, g, dims, obs, idx, hp, seed=5, iteration=2)
    assert_close(out["mean_loss"], float(np.mean([x["loss"] for x in r])), 1e-4, "mean loss")
    assert_close(rnd.get_params(), state.theta, 2e-4, "params")
    rnd.destroy()
