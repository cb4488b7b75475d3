"""GPU parity: the CUDA path, called through the C ABI, against the FP64 oracle on the same
seeded synthetic inputs.

Tolerances (|x - y| <= tol |y| + tol rms(y), element by element):
  FP32 mode  actions / mu / log-probs / values 1e-5; returns / advantages 1e-5;
             losses, gradient and parameters after one optimiser step 1e-4.
  TF32 mode  5e-3 for the act outputs and for losses / parameters after one step.
  BF16 mode  2e-2 for the act outputs, 1e-2 for losses / parameters after one step.
Integer work (shuffle indices, stored flags) is compared bit for bit.
"""
import numpy as np
import pytest

from oracle import ppo_oracle as O
from paper_2509_10771_b200 import workloads as WL

from parity_utils import (assert_close, dims_of, gpu_rollout, oracle_rollout, read_storage, rel_l2, write_storage)

pytestmark = pytest.mark.gpu

FP32, TF32, BF16 = WL.PRECISION_FP32, WL.PRECISION_TF32, WL.PRECISION_BF16

# parity-sized versions of the five workloads (the oracle finishes each in seconds); row
# counts are chosen ragged on purpose: not multiples of the 128-row tiles
CASES = {
    "tiny": WL.TINY,
    "flat": WL.FLAT.scaled(500, minibatches=4),
    "rough": WL.ROUGH.scaled(300, minibatches=4),
    "humanoid": WL.HUMANOID.scaled(200, minibatches=8),
    "rough_sym": WL.ROUGH_SYM.scaled(150, minibatches=16, precision=FP32),
    # full sizes: rough_terrain is the configuration bench.py times (4096 envs x 24 steps, 24,576-row minibatches)
    "flat_full": WL.FLAT,
    "rough_full": WL.ROUGH,
    "humanoid_full": WL.HUMANOID,
    # 65,536 envs x 32 steps, minibatches of 131,072 rows doubled by the mirror to 262,144, BF16 operands
    "rough_sym_full": WL.ROUGH_SYM,
}


def make_ctx(w, precision=None, mirror=None):
    from paper_2509_10771_b200 import binding
    return binding.Context(w, precision=precision, mirror=mirror)


def mirror_of(w):
    return WL.make_mirror(w) if w.sym_enable else None


# --------------------------------------------------------------------------------------
# (1) act + (2) gae
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid"])
def test_rollout_and_gae_match_oracle_fp32(case):
    w = CASES[case]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    ctx = make_ctx(w, FP32)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    got = read_storage(ctx, w)
    want = oracle_rollout(w, theta, inputs)
    for k in ("actions", "mu", "sigma", "logp", "values"):
        assert_close(got[k], want[k], 1e-5, f"{case}.{k}")
    for k in ("returns", "advantages"):
        assert_close(got[k], want[k], 1e-5, f"{case}.{k}")
    assert np.array_equal(got["obs_actor"], inputs["obs_actor"][:w.num_steps])
    assert np.array_equal(got["obs_critic"], inputs["obs_critic"][:w.num_steps])
    assert np.array_equal(got["dones"], inputs["dones"]) and np.array_equal(got["timeouts"], inputs["timeouts"])
    assert np.array_equal(got["rewards"], inputs["rewards"])
    ctx.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid"])
def test_rollout_and_gae_match_oracle_bf16(case):
    w = CASES[case]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    ctx = make_ctx(w, BF16)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    got = read_storage(ctx, w)
    want = oracle_rollout(w, theta, inputs)
    for k in ("actions", "mu", "values"):
        assert_close(got[k], want[k], 2e-2, f"{case}.{k}")
    # the log-density of a = mu + sigma eps under (mu, sigma) depends on eps alone
    assert_close(got["logp"], want["logp"], 1e-5, f"{case}.logp")
    assert_close(got["sigma"], want["sigma"], 1e-6, f"{case}.sigma")
    for k in ("returns", "advantages"):
        assert_close(got[k], want[k], 2e-2, f"{case}.{k}")
    assert np.array_equal(got["obs_actor"], inputs["obs_actor"][:w.num_steps])
    ctx.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid"])
def test_rollout_and_gae_match_oracle_tf32(case):
    """TF32 operands in the hidden-layer products (FP32 storage, accumulation and heads): 5e-3."""
    w = CASES[case]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    ctx = make_ctx(w, TF32)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    got = read_storage(ctx, w)
    want = oracle_rollout(w, theta, inputs)
    for k in ("actions", "mu", "values", "returns", "advantages"):
        assert_close(got[k], want[k], 5e-3, f"{case}.{k}")
    assert_close(got["logp"], want["logp"], 1e-5, f"{case}.logp")
    assert_close(got["sigma"], want["sigma"], 1e-6, f"{case}.sigma")
    assert np.array_equal(got["obs_actor"], inputs["obs_actor"][:w.num_steps])
    # the tensor cores did see TF32 operands: the result is not the FP32 mode's
    ctx32 = make_ctx(w, FP32)
    ctx32.set_params(theta)
    gpu_rollout(ctx32, w, inputs)
    assert np.abs(read_storage(ctx32, w)["mu"] - got["mu"]).max() > 0.0
    ctx32.destroy()
    ctx.destroy()


@pytest.mark.parametrize("case", ["flat_full", "rough_full", "humanoid_full"])
def test_full_size_workloads_bf16(case):
    """The flat, rough (the benchmarked one) and humanoid workloads at full size, BF16: every stored rollout
    output and the first minibatch step against the oracle (which needs some seconds at these sizes)."""
    _first_step(case, BF16, from_oracle_storage=True, check_rollout=True)


def test_symmetry_workload_at_full_size_bf16():
    """The massive-parallel symmetry workload as stated: 65,536 environments x 32 steps, 16 minibatches of
    131,072 rows doubled by the mirror, BF16 operands.  Every stored rollout output (2,097,152 transitions), the
    advantages and returns, and the first minibatch step (losses, symmetry loss, gradient block by block and
    element by element, parameters) against the oracle, which needs a few minutes of host time at this size."""
    _first_step("rough_sym_full", BF16, from_oracle_storage=True, check_rollout=True)


def test_noise_is_the_shared_philox_stream():
    """(a - mu) / sigma recovers the oracle's Gaussian noise for the right (env, step) counters."""
    w = CASES["flat"]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    off = [o for name, o, _ in WL.param_layout(w) if name == "actor.log_std"][0]
    theta[off:off + w.num_actions] = np.linspace(-0.5, 0.3, w.num_actions, dtype=np.float32)
    ctx = make_ctx(w, FP32)
    ctx.set_params(theta)
    ctx.set_counters(lr=w.lr, adam_step=0, global_step=1000, iteration=0)
    gpu_rollout(ctx, w, inputs)
    got = read_storage(ctx, w)
    for t in (0, 7, w.num_steps - 1):
        eps = (got["actions"][t] - got["mu"][t]) / got["sigma"][t]
        want = O.gaussian_noise(w.seed, 1000 + t, w.num_envs, w.num_actions)
        assert np.abs(eps - want).max() < 2e-5
    ctx.destroy()


# --------------------------------------------------------------------------------------
# (3) update
# --------------------------------------------------------------------------------------
def _first_step(case, precision, from_oracle_storage, check_rollout=False):
    w = CASES[case]
    theta, inputs, mir = WL.make_params(w), WL.make_rollout_inputs(w), mirror_of(w)
    ctx = make_ctx(w, precision, mir)
    ctx.set_params(theta)
    want_st = oracle_rollout(w, theta, inputs)
    gpu_rollout(ctx, w, inputs)
    if check_rollout:
        got = read_storage(ctx, w, with_obs=False)
        # beyond ten million elements the tail of the BF16 rounding error (a sum of many independent roundings,
        # about a quarter of the bound in spread) crosses the bound for a few elements per ten million: one per
        # million may, by at most half the bound
        many = got["mu"].size > 10_000_000
        for k in ("actions", "mu", "values", "returns", "advantages"):
            assert_close(got[k], want_st[k], 2e-2, f"{case}.{k}", max_outlier_frac=1e-6 if many else 0.0,
                         outlier_factor=1.5 if many else 0.0)
        assert_close(got["logp"], want_st["logp"], 1e-5, f"{case}.logp")
        del got
    if from_oracle_storage:
        write_storage(ctx, w, want_st)
    stats = ctx.ppo_update(max_steps=1)
    state = O.OptimState(theta, w.lr)
    ref = O.ppo_update(state, dims_of(w), want_st, w, seed=w.seed, iteration=0, sym=mir, max_steps=1)[0]
    tol = {FP32: 1e-4, TF32: 5e-3, BF16: 1e-2}[precision]
    if case.endswith("_full"):
        # the surrogate is a mean of -A r over the minibatch with A normalised (mean 0, |A| ~ 1) and r ~ 1:
        # over 24,576 rows it cancels to ~1e-4, so the bound is relative to the size of the terms, mean |A|
        scale = float(np.abs(want_st["advantages"]).mean())
        assert abs(stats["first_surrogate"] - ref["surrogate"]) <= tol * (abs(ref["surrogate"]) + scale), "surrogate"
    else:
        assert_close(stats["first_surrogate"], ref["surrogate"], tol, "surrogate")
    assert_close(stats["first_value_loss"], ref["value_loss"], tol, "value_loss")
    assert_close(stats["entropy"], ref["entropy"], tol, "entropy")
    assert abs(stats["first_kl"] - ref["kl"]) < (1e-6 if precision == FP32 else 1e-4)   # the exact value is 0
    assert_close(stats["first_grad_norm"], ref["grad_norm"], tol, "grad_norm")
    assert_close(stats["lr"], ref["lr"], 1e-6, "lr")
    if w.sym_enable:
        assert_close(stats["first_sym_loss"], ref["sym_loss"], tol, "sym_loss")
    g = ctx.get_grads()
    blocks = [(name, off, int(np.prod(shape))) for name, off, shape in WL.param_layout(w)]
    if precision == FP32:
        assert_close(g, ref["grad"], tol, "grad")
    elif precision == TF32:
        # every product of the step saw TF32 operands (11 significant bits): each term of a weight-gradient sum
        # carries two operand roundings of 2^-11, and the sum over the minibatch rows cancels (the advantages have
        # mean zero), so the error relative to the result is a few times that of a term: element by element at
        # twice the mode's tolerance per block, the whole gradient in relative L2 at the mode's tolerance itself
        for name, off, n in blocks:
            assert_close(g[off:off + n], ref["grad"][off:off + n], 1e-2, f"grad {name}")
        assert rel_l2(g, ref["grad"]) < tol
    else:
        # every parameter block on its own, so a wrong layer cannot hide behind a large one: element by element
        # (a BF16-rounded operand perturbs every product of a three-layer chain: 5e-2 of |y| + rms of the block;
        # the largest ratio seen on these workloads is 3.2e-2), and in relative L2
        for name, off, n in blocks:
            assert_close(g[off:off + n], ref["grad"][off:off + n], 5e-2, f"grad {name}")
            assert rel_l2(g[off:off + n], ref["grad"][off:off + n]) < 3e-2, name
        assert rel_l2(g, ref["grad"]) < 1e-2
    # Adam's first step is lr * g / (|g| + eps), i.e. lr * sign(g): discontinuous where a gradient entry is zero to
    # rounding.  The parameters are therefore compared at the plain tolerance on the entries whose gradient is
    # clearly non-zero, |g| >= thr * rms(g of the block) (about 95 % of them); the others can differ by up to
    # 2 lr whatever the implementation, which is only asserted as a sanity bound.
    thr = 1e-2 if precision == FP32 else 5e-2
    sure = np.zeros(ref["grad"].shape, dtype=bool)
    for name, off, n in blocks:
        b = ref["grad"][off:off + n]
        sure[off:off + n] = np.abs(b) >= thr * np.sqrt(np.mean(b * b))
    assert sure.mean() > 0.8
    got_p = ctx.get_params().astype(np.float64)
    rms_p = float(np.sqrt(np.mean(state.theta ** 2)))
    err_p = np.abs(got_p - state.theta)
    assert np.all(err_p[sure] <= tol * (np.abs(state.theta[sure]) + rms_p)), "params"
    assert err_p.max() <= 2.05 * ref["lr"]
    m, v = ctx.get_adam()
    if precision == FP32:
        assert_close(m, state.m, tol, "adam_m")
        assert_close(v, state.v, 2 * tol, "adam_v")
    else:
        assert rel_l2(m, state.m) < (tol if precision == TF32 else 1e-2)
    c = ctx.get_counters()
    assert c.adam_step == 1 and c.iteration == 1
    ctx.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid", "rough_sym"])
def test_first_update_step_matches_oracle_fp32(case):
    _first_step(case, FP32, from_oracle_storage=False)


@pytest.mark.parametrize("case", ["tiny", "rough_sym"])
def test_first_update_step_from_oracle_storage(case):
    _first_step(case, FP32, from_oracle_storage=True)


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid", "rough_sym"])
def test_first_update_step_matches_oracle_bf16(case):
    _first_step(case, BF16, from_oracle_storage=True)


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid", "rough_sym"])
def test_first_update_step_matches_oracle_tf32(case):
    _first_step(case, TF32, from_oracle_storage=True)


@pytest.mark.parametrize("case,precision", [("tiny", FP32), ("flat", FP32), ("rough_sym", FP32), ("rough", BF16), ("rough", TF32)])
def test_full_update_tracks_oracle(case, precision):
    """All E*M steps: the trajectories stay together (looser: Adam amplifies rounding)."""
    w = CASES[case]
    theta, inputs, mir = WL.make_params(w), WL.make_rollout_inputs(w), mirror_of(w)
    ctx = make_ctx(w, precision, mir)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    stats = ctx.ppo_update()
    state = O.OptimState(theta, w.lr)
    ref = O.ppo_update(state, dims_of(w), oracle_rollout(w, theta, inputs), w, seed=w.seed, iteration=0, sym=mir)
    assert stats["steps"] == len(ref) == w.epochs * w.minibatches
    loose = {FP32: 2e-3, TF32: 2e-2, BF16: 5e-2}[precision]
    assert_close(stats["surrogate"], np.mean([r["surrogate"] for r in ref]), loose, "mean surrogate")
    assert_close(stats["value_loss"], np.mean([r["value_loss"] for r in ref]), loose, "mean value loss")
    assert_close(stats["kl"], np.mean([r["kl"] for r in ref]), 10 * loose, "mean kl")
    if precision == FP32:
        assert_close(stats["lr"], ref[-1]["lr"], 1e-6, "final lr")
    assert rel_l2(ctx.get_params(), state.theta) < loose
    ctx.destroy()


def test_two_iterations_advance_noise_and_shuffle_counters():
    w = CASES["tiny"]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    ctx = make_ctx(w, FP32)
    ctx.set_params(theta)
    state = O.OptimState(theta, w.lr)
    for it in range(2):
        gpu_rollout(ctx, w, inputs)
        got = read_storage(ctx, w)
        want = O.rollout(state.theta, dims_of(w), inputs, w, seed=w.seed, first_global_step=it * w.num_steps)
        assert_close(got["actions"], want["actions"], 1e-4, f"actions it{it}")
        ctx.ppo_update()
        O.ppo_update(state, dims_of(w), want, w, seed=w.seed, iteration=it)
    assert rel_l2(ctx.get_params(), state.theta) < 2e-3
    c = ctx.get_counters()
    assert c.global_step == 2 * w.num_steps and c.iteration == 2 and c.adam_step == 2 * w.epochs * w.minibatches
    ctx.destroy()


@pytest.mark.parametrize("precision", [FP32, BF16])
def test_update_is_bitwise_deterministic_and_resumable(precision):
    w = CASES["flat"]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    outs = []
    for _ in range(2):
        ctx = make_ctx(w, precision)
        ctx.set_params(theta)
        gpu_rollout(ctx, w, inputs)
        ctx.ppo_update()
        outs.append((ctx.get_params(), ctx.get_grads(), *ctx.get_adam()))
        ctx.destroy()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)
    # checkpoint after the first iteration, resume in a fresh context, run a second iteration
    ctx = make_ctx(w, precision)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    ctx.ppo_update()
    snap = (ctx.get_params(), *ctx.get_adam(), ctx.get_counters())
    gpu_rollout(ctx, w, inputs)
    ctx.ppo_update()
    want = ctx.get_params()
    ctx.destroy()
    ctx = make_ctx(w, precision)
    ctx.set_params(snap[0]); ctx.set_adam(snap[1], snap[2])
    ctx.set_counters(snap[3].lr, snap[3].adam_step, snap[3].global_step, snap[3].iteration)
    gpu_rollout(ctx, w, inputs)
    ctx.ppo_update()
    assert np.array_equal(ctx.get_params(), want)
    ctx.destroy()


# --------------------------------------------------------------------------------------
# stand-alone pieces at full size, edge cases
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("T,N", [(1, 1), (8, 64), (24, 4096), (5, 130), (32, 65536), (24, 100001)])
@pytest.mark.parametrize("normalize", [True, False])
def test_gae_scan_matches_oracle(T, N, normalize):
    import torch
    from paper_2509_10771_b200 import binding
    rng = np.random.default_rng(T * 1000003 + N)
    r = rng.normal(0, 0.5, (T, N)).astype(np.float32)
    v = rng.normal(0, 1.0, (T, N)).astype(np.float32)
    lv = rng.normal(0, 1.0, N).astype(np.float32)
    d = (rng.random((T, N)) < 0.02).astype(np.uint8)
    to = (d & (rng.random((T, N)) < 0.5)).astype(np.uint8)
    dev = lambda x: torch.from_numpy(x).cuda()
    ret = torch.empty((T, N), device="cuda"); adv = torch.empty((T, N), device="cuda")
    scratch = torch.empty(max(binding.gae_scratch_bytes(T, N), 16), dtype=torch.uint8, device="cuda")
    binding.gae_scan(dev(r), dev(v), dev(d), dev(to), dev(lv), ret, adv, T, N, 0.99, 0.95, normalize, True, 1e-8,
                     scratch)
    torch.cuda.synchronize()
    wret, wadv = O.gae(r, v, d, to, lv, 0.99, 0.95)
    if normalize and T * N > 1:
        wadv = O.normalize_advantages(wadv, 1e-8, True)
    assert_close(ret.cpu().numpy(), wret, 1e-5, "returns")
    if T * N > 1 or not normalize:
        assert_close(adv.cpu().numpy(), wadv, 1e-5, "advantages")


def test_gae_scan_degenerate_flags():
    import torch
    from paper_2509_10771_b200 import binding
    T, N = 6, 257
    rng = np.random.default_rng(0)
    r = rng.normal(size=(T, N)).astype(np.float32); v = rng.normal(size=(T, N)).astype(np.float32)
    lv = rng.normal(size=N).astype(np.float32)
    dev = lambda x: torch.from_numpy(x).cuda()
    for d, to in ((np.ones((T, N), np.uint8), np.zeros((T, N), np.uint8)),
                  (np.ones((T, N), np.uint8), np.ones((T, N), np.uint8)),
                  (np.zeros((T, N), np.uint8), np.zeros((T, N), np.uint8))):
        ret = torch.empty((T, N), device="cuda"); adv = torch.empty((T, N), device="cuda")
        scratch = torch.empty(binding.gae_scratch_bytes(T, N), dtype=torch.uint8, device="cuda")
        binding.gae_scan(dev(r), dev(v), dev(d), dev(to), dev(lv), ret, adv, T, N, 0.99, 0.95, False, True, 1e-8, scratch)
        wret, wadv = O.gae(r, v, d, to, lv, 0.99, 0.95)
        assert_close(adv.cpu().numpy(), wadv, 1e-5, "adv"); assert_close(ret.cpu().numpy(), wret, 1e-5, "ret")
    # empty inputs are a no-op
    binding.gae_scan(None, None, None, None, None, None, None, 0, 0, 0.99, 0.95, True, True, 1e-8, None)


@pytest.mark.parametrize("batch,mb", [(512, 2), (98304, 4), (196608, 8), (2097152, 16), (1000, 1), (7, 7), (3 * 5 * 7 * 11, 5)])
def test_minibatch_indices_bit_exact(batch, mb):
    import torch
    from paper_2509_10771_b200 import binding
    seed, it, ep = 0x1234567890ABCDEF, 3, 2
    want = O.feistel_permutation(seed, it, ep, batch)
    rows = batch // mb
    out = torch.empty(rows, dtype=torch.int32, device="cuda")
    for k in sorted({0, mb // 2, mb - 1}):
        binding.minibatch_indices(seed, it, ep, batch, mb, k, out)
        assert np.array_equal(out.cpu().numpy().astype(np.int64), want[k * rows:(k + 1) * rows])


# --------------------------------------------------------------------------------------
# boundary behaviour on a live device
# --------------------------------------------------------------------------------------
def test_call_order_and_argument_errors():
    import torch
    from paper_2509_10771_b200 import binding
    w = WL.TINY
    ctx = make_ctx(w, FP32)
    ctx.set_params(WL.make_params(w))
    obs = torch.zeros((w.num_envs, w.actor_obs_dim), device="cuda")
    rew = torch.zeros(w.num_envs, device="cuda"); flags = torch.zeros(w.num_envs, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.RslrlError) as e:
        ctx.gae(obs)
    assert e.value.status == 4
    with pytest.raises(binding.RslrlError) as e:
        ctx.ppo_update()
    assert e.value.status == 4
    with pytest.raises(binding.RslrlError) as e:
        ctx.record_step(rew, flags, flags)
    assert e.value.status == 4
    ctx.act(obs)
    with pytest.raises(binding.RslrlError) as e:
        ctx.act(obs)
    assert e.value.status == 4
    ctx.record_step(rew, flags, flags)
    with pytest.raises(binding.RslrlError) as e:
        ctx.act(obs.data_ptr() + 2)                  # misaligned device pointer
    assert e.value.status == 3
    with pytest.raises(binding.RslrlError) as e:
        ctx.set_params(np.zeros(3, np.float32))
    assert e.value.status == 2
    for _ in range(w.num_steps - 1):
        ctx.act(obs); ctx.record_step(rew, flags, flags)
    with pytest.raises(binding.RslrlError) as e:
        ctx.act(obs)
    assert e.value.status == 4
    ctx.gae(obs)
    st = ctx.ppo_update()
    assert st["steps"] == w.epochs * w.minibatches and st["nonfinite"] == 0
    ctx.destroy()
    with pytest.raises(binding.RslrlError) as e:
        make_ctx(WL.TINY.scaled(64, minibatches=7))
    assert e.value.status == 2


def test_host_buffer_variants_match_device_calls():
    w = CASES["tiny"]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    a = make_ctx(w, FP32); a.set_params(theta)
    gpu_rollout(a, w, inputs)
    want = read_storage(a, w)
    b = make_ctx(w, FP32); b.set_params(theta)
    acts = np.empty((w.num_envs, w.num_actions), np.float32)
    for t in range(w.num_steps):
        b.act_host(inputs["obs_actor"][t], None, acts)
        assert np.array_equal(acts, want["actions"][t])
        b.record_step_host(inputs["rewards"][t], inputs["dones"][t], inputs["timeouts"][t])
    b.gae_host(inputs["obs_critic"][w.num_steps])
    got = read_storage(b, w)
    for k in ("actions", "logp", "values", "returns", "advantages"):
        assert np.array_equal(got[k], want[k]), k
    a.destroy(); b.destroy()


def test_kernels_were_launched_by_this_library():
    from paper_2509_10771_b200 import binding
    before = binding.kernel_launch_count()
    w = WL.TINY
    ctx = make_ctx(w, FP32)
    ctx.set_params(WL.make_params(w))
    gpu_rollout(ctx, w, WL.make_rollout_inputs(w))
    ctx.ppo_update()
    ctx.destroy()
    assert binding.kernel_launch_count() - before > 3 * w.num_steps


@pytest.mark.parametrize("precision", [FP32, BF16])
def test_non_finite_step_is_skipped_and_reported(precision):
    """A NaN among the parameters (set from the host; nothing faults on the device) makes every loss of the
    update non-finite: each optimiser step is skipped, rslrl_ppo_update returns RSLRL_ERR_NONFINITE with
    nonfinite = 1 in the statistics, and parameters, Adam moments and the step count are what they were."""
    import ctypes as C
    from paper_2509_10771_b200 import binding
    w = CASES["flat"]
    theta, inputs = WL.make_params(w), WL.make_rollout_inputs(w)
    theta[3] = np.nan                                  # an entry of the actor's first weight matrix
    ctx = make_ctx(w, precision)
    ctx.set_params(theta)
    gpu_rollout(ctx, w, inputs)
    st = binding.UpdateStats()
    rc = ctx.lib.rslrl_ppo_update(ctx.handle, C.byref(st))
    assert rc == 7 and st.nonfinite == 1               # RSLRL_ERR_NONFINITE
    assert "not finite" in ctx.lib.rslrl_last_error(ctx.handle).decode()
    with pytest.raises(binding.RslrlError) as e:       # the binding turns the status into an exception
        gpu_rollout(ctx, w, inputs)
        ctx.ppo_update()
    assert e.value.status == 7
    got = ctx.get_params()
    assert np.isnan(got[3]) and np.array_equal(np.delete(got, 3), np.delete(theta, 3))
    m, v = ctx.get_adam()
    assert not m.any() and not v.any()
    assert ctx.get_counters().adam_step == 0
    ctx.destroy()
