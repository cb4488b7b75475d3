"""GPU parity of the recurrent memory layer (rslrl_gru_forward / rslrl_gru_backward) against the FP64 oracle:
hidden states of every step, gradients with respect to the inputs, the carried-in state and the parameters, on
rollouts with episode ends (state resets) including a raised done rate so that every environment is reset
several times.

The CUDA path computes in FP32.  Tolerances: states 2e-5, gradients 1e-4 (relative to the element plus the
array's rms): a gradient is a sum over up to T N products that back-propagation has passed through up to T
steps of FP32 gate arithmetic."""
import numpy as np
import pytest

from oracle import gru_oracle as G
from paper_2509_10771_b200 import workloads as WL

from parity_utils import assert_close

pytestmark = pytest.mark.gpu

CASES = {
    # name: (workload, hidden_dim, x_stride padding, done probability override)
    "tiny": (WL.TINY, 8, 0, 0.2),
    "flat": (WL.FLAT.scaled(130), 64, 0, 0.05),
    "rough": (WL.ROUGH.scaled(300), 128, 1, 0.1),          # D = 235 -> stride 236: ragged in every direction
    "humanoid": (WL.HUMANOID.scaled(257), 256, 5, 0.01),   # D = 123 -> stride 128; odd number of environments
}


def _run(case, want_dx=True, want_dh0=True, precision=0):
    import torch
    from paper_2509_10771_b200 import binding
    w0, H, pad, dp = CASES[case]
    from dataclasses import replace
    w = replace(w0, done_prob=dp)
    T, N, D = w.num_steps, w.num_envs, w.actor_obs_dim
    inputs = WL.make_rollout_inputs(w)
    setup = WL.make_gru_setup(w, hidden_dim=H)
    x = inputs["obs_actor"][:T]
    dones = inputs["dones"]
    stride = (D + 3) // 4 * 4 + (4 * ((pad + 3) // 4) if pad else 0)
    xp = np.full((T, N, stride), 7.0, dtype=np.float32)        # padding holds junk: it must not be read as data
    xp[..., :D] = x
    gru = binding.Gru(D, H, T, N, precision=precision)
    gru.set_params(setup["params"])
    dev = "cuda"
    d_x = torch.from_numpy(xp).to(dev)
    d_h0 = torch.from_numpy(setup["h0"]).to(dev)
    d_dn = torch.from_numpy(dones).to(dev)
    d_h = torch.empty((T, N, H), device=dev)
    gru.forward(d_x, stride, d_h0, d_dn, T, N, d_h)
    d_dh = torch.from_numpy(setup["dh"]).to(dev)
    d_dx = torch.full((T, N, stride), -3.0, device=dev) if want_dx else None
    d_dh0 = torch.empty((N, H), device=dev) if want_dh0 else None
    gru.backward(d_dh, d_dx, stride, d_dh0)
    torch.cuda.synchronize()
    p = G.unpack_gru(setup["params"], D, H)
    c = G.gru_sequence_forward(p, x, setup["h0"], dones)
    g = G.gru_sequence_backward(p, c, setup["dh"])
    got = {"h": d_h.cpu().numpy(), "dx": d_dx.cpu().numpy() if want_dx else None,
           "dh0": d_dh0.cpu().numpy() if want_dh0 else None, "grad": gru.get_grads()}
    return w, D, H, dones, c, g, got, gru


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid"])
def test_states_and_gradients_match_oracle(case):
    w, D, H, dones, c, g, got, gru = _run(case)
    assert dones[:-1].any()                                        # resets take part
    assert_close(got["h"], c["h"], 2e-5, f"{case}.h")
    assert_close(got["dx"][..., :D], g["x"], 1e-4, f"{case}.dx")
    assert_close(got["dh0"], g["h0"], 1e-4, f"{case}.dh0")
    ref = G.flat_grads(g)
    o = np.cumsum([0, D * 3 * H, 3 * H, H * 3 * H, 3 * H])
    for name, a, b in zip(("W_i", "b_i", "W_h", "b_h"), o[:-1], o[1:]):
        assert_close(got["grad"][a:b], ref[a:b], 1e-4, f"{case}.d{name}")
    # columns of dx between D and D rounded up to 4 are written as zero, the rest of the padding is left alone
    d4 = (D + 3) // 4 * 4
    assert np.all(got["dx"][..., D:d4] == 0.0) and np.all(got["dx"][..., d4:] == -3.0)
    gru.destroy()


@pytest.mark.parametrize("case", ["tiny", "flat", "rough", "humanoid"])
def test_states_and_gradients_match_oracle_tf32(case):
    """RSLRL_TF32: every matrix product of the layer sees TF32 operands (11 significant bits).  States at the mode's
    tolerance 5e-3; gradients, which back-propagation passes through up to T such products, at twice that."""
    w, D, H, dones, c, g, got, gru = _run(case, precision=WL.PRECISION_TF32)
    assert_close(got["h"], c["h"], 5e-3, f"{case}.h")
    assert not np.array_equal(got["h"], _run(case)[6]["h"])        # the tensor cores did see TF32 operands
    assert_close(got["dx"][..., :D], g["x"], 1e-2, f"{case}.dx")
    assert_close(got["dh0"], g["h0"], 1e-2, f"{case}.dh0")
    ref = G.flat_grads(g)
    o = np.cumsum([0, D * 3 * H, 3 * H, H * 3 * H, 3 * H])
    for name, a, b in zip(("W_i", "b_i", "W_h", "b_h"), o[:-1], o[1:]):
        assert_close(got["grad"][a:b], ref[a:b], 1e-2, f"{case}.d{name}")
    d4 = (D + 3) // 4 * 4
    assert np.all(got["dx"][..., D:d4] == 0.0) and np.all(got["dx"][..., d4:] == -3.0)
    gru.destroy()


def test_environments_reset_at_every_step_see_only_the_current_input():
    """done everywhere: every step starts from the zero state, so h(t) is a function of x(t) alone and no
    gradient reaches h0 from steps after the first."""
    import torch
    from paper_2509_10771_b200 import binding
    w = WL.TINY
    T, N, D, H = w.num_steps, w.num_envs, w.actor_obs_dim, 8
    setup = WL.make_gru_setup(w, hidden_dim=H)
    x = WL.make_rollout_inputs(w)["obs_actor"][:T]
    dones = np.ones((T, N), dtype=np.uint8)
    gru = binding.Gru(D, H, T, N)
    gru.set_params(setup["params"])
    d_h = torch.empty((T, N, H), device="cuda")
    d_x, d_h0, d_dones = torch.from_numpy(x).to("cuda"), torch.from_numpy(setup["h0"]).to("cuda"), torch.from_numpy(dones).to("cuda")
    gru.forward(d_x, D, d_h0, d_dones, T, N, d_h)
    dh = setup["dh"].copy(); dh[0] = 0.0
    d_dh, d_dh0 = torch.from_numpy(dh).to("cuda"), torch.full((N, H), 5.0, device="cuda")
    gru.backward(d_dh, None, 0, d_dh0)
    torch.cuda.synchronize()
    p = G.unpack_gru(setup["params"], D, H)
    zero = np.zeros((N, H))
    for t in range(1, T):
        one = G.gru_sequence_forward(p, x[t:t + 1], zero, np.zeros((1, N), np.uint8))["h"][0]
        assert_close(d_h[t].cpu().numpy(), one, 2e-5, f"h[{t}]")
    assert np.all(d_dh0.cpu().numpy() == 0.0)
    gru.destroy()


def test_gru_argument_checks():
    import torch
    from paper_2509_10771_b200 import binding
    with pytest.raises(binding.RslrlError) as e:
        binding.Gru(16, 6, 4, 8)                                   # hidden_dim not a multiple of 4
    assert e.value.status == 1
    gru = binding.Gru(6, 8, 4, 8)
    assert gru.num_params == 6 * 24 + 24 + 8 * 24 + 24
    gru.set_params(np.zeros(gru.num_params, np.float32))
    x = torch.zeros((4, 8, 8), device="cuda"); h0 = torch.zeros((8, 8), device="cuda")
    dn = torch.zeros((4, 8), dtype=torch.uint8, device="cuda"); h = torch.empty((4, 8, 8), device="cuda")
    with pytest.raises(binding.RslrlError) as e:
        gru.backward(h)                                            # no forward yet
    assert e.value.status == 4
    with pytest.raises(binding.RslrlError) as e:
        gru.forward(x, 6, h0, dn, 4, 8, h)                         # stride not a multiple of 4
    assert e.value.status == 2
    with pytest.raises(binding.RslrlError) as e:
        gru.forward(x, 8, h0, dn, 5, 8, h)                         # more steps than max_steps
    assert e.value.status == 5
    gru.forward(x, 8, h0, dn, 4, 8, h)
    torch.cuda.synchronize()
    assert np.all(h.cpu().numpy() == 0.0)                          # zero weights, zero state: n = tanh(0) = 0, h stays 0
    gru.backward(h)
    with pytest.raises(binding.RslrlError) as e:
        gru.backward(h)                                            # one backward per forward
    assert e.value.status == 4
    with pytest.raises(binding.RslrlError) as e:
        gru.set_params(np.zeros(3, np.float32))
    assert e.value.status == 2
    gru.destroy()


def test_full_size_rollout_matches_oracle():
    """The size the benchmark's recurrent task runs: 24 steps x 4096 environments of 235 observations, H = 256,
    the workload's own done rate.  Every state and every gradient entry is compared."""
    import torch
    from paper_2509_10771_b200 import binding
    w = WL.ROUGH
    T, N, D, H = w.num_steps, w.num_envs, w.actor_obs_dim, 256
    inputs = WL.make_rollout_inputs(w)
    setup = WL.make_gru_setup(w, hidden_dim=H)
    stride = (D + 3) // 4 * 4
    xp = np.zeros((T, N, stride), dtype=np.float32)
    xp[..., :D] = inputs["obs_actor"][:T]
    gru = binding.Gru(D, H, T, N)
    gru.set_params(setup["params"])
    d_x, d_h0 = torch.from_numpy(xp).to("cuda"), torch.from_numpy(setup["h0"]).to("cuda")
    d_dn, d_dh = torch.from_numpy(inputs["dones"]).to("cuda"), torch.from_numpy(setup["dh"]).to("cuda")
    d_h, d_dx, d_dh0 = torch.empty((T, N, H), device="cuda"), torch.empty((T, N, stride), device="cuda"), torch.empty((N, H), device="cuda")
    gru.forward(d_x, stride, d_h0, d_dn, T, N, d_h)
    gru.backward(d_dh, d_dx, stride, d_dh0)
    torch.cuda.synchronize()
    p = G.unpack_gru(setup["params"], D, H)
    c = G.gru_sequence_forward(p, inputs["obs_actor"][:T], setup["h0"], inputs["dones"])
    g = G.gru_sequence_backward(p, c, setup["dh"])
    assert_close(d_h.cpu().numpy(), c["h"], 2e-5, "h")
    assert_close(d_dx.cpu().numpy()[..., :D], g["x"], 1e-4, "dx")
    assert_close(d_dh0.cpu().numpy(), g["h0"], 1e-4, "dh0")
    assert_close(gru.get_grads(), G.flat_grads(g), 1e-4, "grad")
    gru.destroy()


def test_rollout_taken_step_by_step_equals_the_rollout_taken_at_once():
    """Acting uses the layer one step per call: the state comes back in with the previous step's done flags as the
    reset vector.  The states equal those of the single T-step call up to FP32 rounding (the input product runs
    with a different tile shape when all steps are batched), the flagged form matches the oracle, and the gradient with respect to a flagged carried-in state is exactly zero."""
    import torch
    from dataclasses import replace
    from paper_2509_10771_b200 import binding
    w = replace(WL.FLAT.scaled(130), done_prob=0.1)
    T, N, D, H = w.num_steps, w.num_envs, w.actor_obs_dim, 64
    inputs = WL.make_rollout_inputs(w)
    setup = WL.make_gru_setup(w, hidden_dim=H)
    x, dones = inputs["obs_actor"][:T], inputs["dones"]
    gru = binding.Gru(D, H, T, N)
    gru.set_params(setup["params"])
    d_x, d_dn = torch.from_numpy(x).to("cuda"), torch.from_numpy(dones).to("cuda")
    d_h0 = torch.from_numpy(setup["h0"]).to("cuda")
    whole = torch.empty((T, N, H), device="cuda")
    gru.forward(d_x, D, d_h0, d_dn, T, N, whole)
    steps = torch.empty((T, N, H), device="cuda")
    for t in range(T):
        gru.forward(d_x[t], D, d_h0 if t == 0 else steps[t - 1], d_dn[t], 1, N, steps[t],
                    d_h0_reset=None if t == 0 else d_dn[t - 1])
    torch.cuda.synchronize()
    assert float((whole - steps).abs().max()) <= 2e-6
    flags = (np.arange(N) % 3 == 0).astype(np.uint8)
    d_flags = torch.from_numpy(flags).to("cuda")
    d_h, d_dh0 = torch.empty((T, N, H), device="cuda"), torch.empty((N, H), device="cuda")
    gru.forward(d_x, D, d_h0, d_dn, T, N, d_h, d_h0_reset=d_flags)
    gru.backward(torch.from_numpy(setup["dh"]).to("cuda"), None, 0, d_dh0)
    torch.cuda.synchronize()
    p = G.unpack_gru(setup["params"], D, H)
    c = G.gru_sequence_forward(p, x, setup["h0"], dones, h0_reset=flags)
    g = G.gru_sequence_backward(p, c, setup["dh"])
    assert_close(d_h.cpu().numpy(), c["h"], 2e-5, "h")
    assert_close(d_dh0.cpu().numpy(), g["h0"], 1e-4, "dh0")
    assert np.all(d_dh0.cpu().numpy()[flags == 1] == 0.0)
    assert_close(gru.get_grads(), G.flat_grads(g), 1e-4, "grad")
    gru.destroy()


@pytest.mark.parametrize("T,N,D,H", [(1, 1, 1, 4), (3, 5, 7, 12), (32, 33, 9, 20)])
def test_smallest_and_odd_shapes(T, N, D, H):
    """One step of one environment with one input, and shapes that are multiples of nothing."""
    import torch
    from paper_2509_10771_b200 import binding
    rng = np.random.default_rng(T * 100 + N)
    n = D * 3 * H + 3 * H + H * 3 * H + 3 * H
    params = (rng.standard_normal(n) * 0.4).astype(np.float32)
    stride = (D + 3) // 4 * 4
    x = rng.standard_normal((T, N, D)).astype(np.float32)
    xp = np.zeros((T, N, stride), np.float32); xp[..., :D] = x
    h0 = rng.standard_normal((N, H)).astype(np.float32)
    dones = (rng.random((T, N)) < 0.3).astype(np.uint8)
    dh = rng.standard_normal((T, N, H)).astype(np.float32)
    gru = binding.Gru(D, H, T, N)
    gru.set_params(params)
    d_x, d_h0, d_dn, d_dh = (torch.from_numpy(a).to("cuda") for a in (xp, h0, dones, dh))
    d_h, d_dx, d_dh0 = torch.empty((T, N, H), device="cuda"), torch.zeros((T, N, stride), device="cuda"), torch.empty((N, H), device="cuda")
    gru.forward(d_x, stride, d_h0, d_dn, T, N, d_h)
    gru.backward(d_dh, d_dx, stride, d_dh0)
    torch.cuda.synchronize()
    p = G.unpack_gru(params, D, H)
    c = G.gru_sequence_forward(p, x, h0, dones)
    g = G.gru_sequence_backward(p, c, dh)
    assert_close(d_h.cpu().numpy(), c["h"], 2e-5, "h")
    assert_close(d_dx.cpu().numpy()[..., :D], g["x"], 1e-4, "dx")
    assert_close(d_dh0.cpu().numpy(), g["h0"], 1e-4, "dh0")
    assert_close(gru.get_grads(), G.flat_grads(g), 1e-4, "grad")
    gru.destroy()
