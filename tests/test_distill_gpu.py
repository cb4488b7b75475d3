"""GPU parity of the distillation step (rslrl_distill_update) against the FP64 oracle: the student
(the context's actor net) is rolled out through the C ABI, its transitions are relabelled with
seeded stand-in expert actions, and the first optimiser step (loss, gradient, parameters, Adam
moments) and the whole epoch x minibatch loop are compared.

Tolerances as for the PPO update: 1e-4 (FP32 mode), 1e-2 (BF16 operands)."""
import numpy as np
import pytest

from oracle import ppo_oracle as O
from paper_2509_10771_b200 import workloads as WL

from parity_utils import assert_close, dims_of, rel_l2

pytestmark = pytest.mark.gpu

FP32, BF16 = WL.PRECISION_FP32, WL.PRECISION_BF16

CASES = {
    "tiny": WL.TINY,
    "flat": WL.FLAT.scaled(500, minibatches=4),
    "rough": WL.ROUGH.scaled(300, minibatches=4),
    "humanoid": WL.HUMANOID.scaled(200, minibatches=8),
}


def _student_rollout(ctx, w, inputs):
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


def _expert_on_device(ctx, w, expert):
    import torch
    s = ctx.storage_view()
    padded = np.zeros((w.num_steps, w.num_envs, s.act_stride), dtype=np.float32)
    padded[..., :w.num_actions] = expert
    return torch.from_numpy(padded).to("cuda")


def _run(case, precision, max_steps):
    from paper_2509_10771_b200 import binding
    w = CASES[case]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    expert = WL.make_expert_actions(w)
    ctx = binding.Context(w, precision=precision)
    ctx.set_params(theta)
    _student_rollout(ctx, w, inputs)
    d_expert = _expert_on_device(ctx, w, expert)
    stats = ctx.distill_update(d_expert, max_steps=max_steps)
    state = O.OptimState(theta, w.lr)
    ref = O.distill_update(state, dims_of(w), inputs["obs_actor"], expert, w, seed=w.seed, iteration=0,
                           max_steps=max_steps if max_steps > 0 else None)
    return w, ctx, stats, state, ref


@pytest.mark.parametrize("precision", [FP32, BF16])
@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid"])
def test_first_distillation_step_matches_oracle(case, precision):
    w, ctx, stats, state, ref = _run(case, precision, max_steps=1)
    tol = 1e-4 if precision == FP32 else 1e-2
    assert_close(stats["first_surrogate"], ref[0]["loss"], tol, "loss")
    assert_close(stats["first_grad_norm"], ref[0]["grad_norm"], tol, "grad_norm")
    assert stats["lr"] == pytest.approx(w.lr, rel=1e-6)          # no learning-rate rule in this step
    assert stats["first_kl"] == 0.0 and stats["first_value_loss"] == 0.0
    g = ctx.get_grads()
    n_actor = sum(i * o + o for i, o in w.layer_dims("actor"))
    assert np.all(g[n_actor:] == 0.0)                            # log_std and the critic take no part
    if precision == FP32:
        assert_close(g, ref[0]["grad"], tol, "grad")
    else:
        for name, off, shape in WL.param_layout(w):
            n = int(np.prod(shape))
            if off + n <= n_actor:
                assert rel_l2(g[off:off + n], ref[0]["grad"][off:off + n]) < 3e-2, name
        assert rel_l2(g, ref[0]["grad"]) < 1e-2
    frac = 2e-3 if precision == FP32 else 5e-2
    assert_close(ctx.get_params(), state.theta, tol, "params", max_outlier_frac=frac, outlier_abs=2.05 * w.lr)
    c = ctx.get_counters()
    assert c.adam_step == 1 and c.iteration == 1
    ctx.destroy()


@pytest.mark.parametrize("case,precision", [("tiny", FP32), ("flat", FP32), ("rough", BF16)])
def test_whole_distillation_update_tracks_oracle(case, precision):
    w, ctx, stats, state, ref = _run(case, precision, max_steps=0)
    assert stats["steps"] == w.epochs * w.minibatches == len(ref)
    mean_loss = float(np.mean([r["loss"] for r in ref]))
    assert_close(stats["surrogate"], mean_loss, 1e-3 if precision == FP32 else 2e-2, "mean loss")
    assert_close(stats["last_grad_norm"], ref[-1]["grad_norm"], 1e-2 if precision == FP32 else 5e-2, "last grad norm")
    assert rel_l2(ctx.get_params(), state.theta) < (1e-4 if precision == FP32 else 1e-2)
    ctx.destroy()


def test_distillation_call_order_and_arguments():
    import torch
    from paper_2509_10771_b200 import binding
    w = CASES["tiny"]
    ctx = binding.Context(w, precision=FP32)
    ctx.set_params(WL.make_params(w))
    d_expert = _expert_on_device(ctx, w, WL.make_expert_actions(w))
    with pytest.raises(binding.RslrlError) as e:                 # no rollout yet
        ctx.distill_update(d_expert)
    assert e.value.status == 4
    _student_rollout(ctx, w, WL.make_rollout_inputs(w))
    with pytest.raises(binding.RslrlError) as e:
        ctx.distill_update(None)
    assert e.value.status == 1
    ctx.distill_update(d_expert)                                  # now it runs, and starts a new rollout
    assert ctx.storage_view().step == 0
    ctx.destroy()
    torch.cuda.synchronize()


@pytest.mark.parametrize("precision", [FP32, BF16])
def test_distillation_after_a_ppo_update_leaves_the_critic_alone(precision):
    """A PPO iteration first (it leaves critic gradients in the work buffers), then a distillation step
    from the optimiser state the PPO update ended with: the critic's gradient must be exactly zero and the
    step must match the oracle started from the same state."""
    import torch
    from paper_2509_10771_b200 import binding
    from parity_utils import gpu_rollout
    w = CASES["rough"]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    ctx = binding.Context(w, precision=precision)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    ctx.ppo_update()
    theta1 = ctx.get_params().astype(np.float64)
    m1, v1 = ctx.get_adam()
    c1 = ctx.get_counters()
    inputs2 = WL.make_rollout_inputs(w, seed=w.seed + 1)
    expert = WL.make_expert_actions(w, seed=w.seed + 1)
    _student_rollout(ctx, w, inputs2)
    stats = ctx.distill_update(_expert_on_device(ctx, w, expert), max_steps=1)
    state = O.OptimState(theta1, float(c1.lr))
    state.m, state.v, state.step = m1.astype(np.float64), v1.astype(np.float64), int(c1.adam_step)
    ref = O.distill_update(state, dims_of(w), inputs2["obs_actor"], expert, w, seed=w.seed, iteration=int(c1.iteration),
                           max_steps=1)
    tol = 1e-4 if precision == FP32 else 1e-2
    assert_close(stats["first_surrogate"], ref[0]["loss"], tol, "loss")
    g = ctx.get_grads()
    n_actor = sum(i * o + o for i, o in w.layer_dims("actor"))
    assert np.all(g[n_actor:] == 0.0)
    assert rel_l2(g, ref[0]["grad"]) < (1e-4 if precision == FP32 else 1e-2)
    ctx.destroy()
    torch.cuda.synchronize()
