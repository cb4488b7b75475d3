"""Pins of the recurrent-layer oracle (oracle/gru_oracle.py) against things other than itself: torch.nn.GRU
(forward and autograd) where no state is reset, a torch GRUCell loop with masked states under autograd where
some are, central finite differences, the one-step closed form, and the independence of what follows a reset
from what came before it."""
import numpy as np
import pytest
import torch

from oracle import gru_oracle as G


def problem(seed=0, T=6, N=5, D=4, H=3, done_prob=0.3):
    rng = np.random.default_rng(seed)
    flat = rng.standard_normal(D * 3 * H + 3 * H + H * 3 * H + 3 * H) * 0.5
    x = rng.standard_normal((T, N, D))
    h0 = rng.standard_normal((N, H))
    dones = (rng.random((T, N)) < done_prob).astype(np.uint8)
    dh = rng.standard_normal((T, N, H))
    return flat, x, h0, dones, dh


def torch_cell(flat, D, H):
    p = G.unpack_gru(flat, D, H)
    cell = torch.nn.GRUCell(D, H).double()
    with torch.no_grad():
        cell.weight_ih.copy_(torch.from_numpy(p["W_i"].T.copy()))
        cell.weight_hh.copy_(torch.from_numpy(p["W_h"].T.copy()))
        cell.bias_ih.copy_(torch.from_numpy(p["b_i"].copy()))
        cell.bias_hh.copy_(torch.from_numpy(p["b_h"].copy()))
    return cell


def test_forward_and_gradients_match_torch_gru_without_resets():
    flat, x, h0, dones, dh = problem(done_prob=0.0)
    T, N, D = x.shape; H = h0.shape[1]
    p = G.unpack_gru(flat, D, H)
    gru = torch.nn.GRU(D, H).double()
    with torch.no_grad():
        gru.weight_ih_l0.copy_(torch.from_numpy(p["W_i"].T.copy())); gru.weight_hh_l0.copy_(torch.from_numpy(p["W_h"].T.copy()))
        gru.bias_ih_l0.copy_(torch.from_numpy(p["b_i"].copy())); gru.bias_hh_l0.copy_(torch.from_numpy(p["b_h"].copy()))
    xt = torch.from_numpy(x).requires_grad_(True)
    ht = torch.from_numpy(h0).requires_grad_(True)
    out, _ = gru(xt, ht[None])
    (out * torch.from_numpy(dh)).sum().backward()
    c = G.gru_sequence_forward(p, x, h0, dones)
    g = G.gru_sequence_backward(p, c, dh)
    np.testing.assert_allclose(c["h"], out.detach().numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["x"], xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["h0"], ht.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["W_i"], gru.weight_ih_l0.grad.numpy().T, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["W_h"], gru.weight_hh_l0.grad.numpy().T, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["b_i"], gru.bias_ih_l0.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["b_h"], gru.bias_hh_l0.grad.numpy(), rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("seed", [1, 2])
def test_resets_match_a_masked_cell_loop_under_autograd(seed):
    flat, x, h0, dones, dh = problem(seed=seed, T=7, N=6, D=5, H=4, done_prob=0.35)
    T, N, D = x.shape; H = h0.shape[1]
    assert dones[:-1].any()
    cell = torch_cell(flat, D, H)
    xt = torch.from_numpy(x).requires_grad_(True)
    ht = torch.from_numpy(h0).requires_grad_(True)
    h, outs = ht, []
    for t in range(T):
        if t > 0:
            h = h * torch.from_numpy(1.0 - dones[t - 1].astype(np.float64))[:, None]
        h = cell(xt[t], h)
        outs.append(h)
    out = torch.stack(outs)
    (out * torch.from_numpy(dh)).sum().backward()
    p = G.unpack_gru(flat, D, H)
    c = G.gru_sequence_forward(p, x, h0, dones)
    g = G.gru_sequence_backward(p, c, dh)
    np.testing.assert_allclose(c["h"], out.detach().numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(g["x"], xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["h0"], ht.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["W_i"], cell.weight_ih.grad.numpy().T, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["W_h"], cell.weight_hh.grad.numpy().T, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["b_i"], cell.bias_ih.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["b_h"], cell.bias_hh.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_gradients_match_finite_differences():
    flat, x, h0, dones, dh = problem(seed=3, T=4, N=3, D=3, H=2, done_prob=0.3)
    D, H = x.shape[2], h0.shape[1]

    def loss(flat_, x_, h0_):
        c = G.gru_sequence_forward(G.unpack_gru(flat_, D, H), x_, h0_, dones)
        return float((c["h"] * dh).sum())

    p = G.unpack_gru(flat, D, H)
    g = G.gru_sequence_backward(p, G.gru_sequence_forward(p, x, h0, dones), dh)
    gf = G.flat_grads(g)
    eps = 1e-6
    for i in range(flat.size):
        e = np.zeros_like(flat); e[i] = eps
        fd = (loss(flat + e, x, h0) - loss(flat - e, x, h0)) / (2 * eps)
        assert abs(fd - gf[i]) <= 1e-7 * (1 + abs(fd)), (i, fd, gf[i])
    for idx in np.ndindex(*x.shape):
        e = np.zeros_like(x); e[idx] = eps
        fd = (loss(flat, x + e, h0) - loss(flat, x - e, h0)) / (2 * eps)
        assert abs(fd - g["x"][idx]) <= 1e-7 * (1 + abs(fd)), (idx, fd)
    for idx in np.ndindex(*h0.shape):
        e = np.zeros_like(h0); e[idx] = eps
        fd = (loss(flat, x, h0 + e) - loss(flat, x, h0 - e)) / (2 * eps)
        assert abs(fd - g["h0"][idx]) <= 1e-7 * (1 + abs(fd)), (idx, fd)


def test_one_step_closed_form():
    """D = H = 1, one step, scalars: the gate equations typed out with math functions."""
    import math
    wir, wiz, win, bir, biz, bin_, whr, whz, whn, bhr, bhz, bhn = 0.3, -0.2, 0.7, 0.1, 0.05, -0.3, 0.4, 0.6, -0.5, 0.02, -0.04, 0.08
    flat = np.array([wir, wiz, win, bir, biz, bin_, whr, whz, whn, bhr, bhz, bhn])
    xv, hv = 0.9, -0.6
    r = 1 / (1 + math.exp(-(xv * wir + bir + hv * whr + bhr)))
    z = 1 / (1 + math.exp(-(xv * wiz + biz + hv * whz + bhz)))
    n = math.tanh(xv * win + bin_ + r * (hv * whn + bhn))
    want = (1 - z) * n + z * hv
    c = G.gru_sequence_forward(G.unpack_gru(flat, 1, 1), np.array([[[xv]]]), np.array([[hv]]), np.zeros((1, 1), np.uint8))
    assert c["h"][0, 0, 0] == pytest.approx(want, rel=1e-14)


def test_nothing_crosses_a_reset():
    """Environment 0 is done at step 2: its states from step 3 on do not depend on its inputs at steps 0..2 or on
    h0, and no gradient flows from dh at steps >= 3 to x at steps <= 2 or to h0; a done at the last step has no
    effect inside the rollout."""
    flat, x, h0, dones, dh = problem(seed=5, T=6, N=2, D=3, H=3, done_prob=0.0)
    D, H = 3, 3
    p = G.unpack_gru(flat, D, H)
    dones[2, 0] = 1
    a = G.gru_sequence_forward(p, x, h0, dones)
    x2, h02 = x.copy(), h0.copy()
    x2[:3, 0] += 1.0; h02[0] -= 2.0
    b = G.gru_sequence_forward(p, x2, h02, dones)
    assert np.array_equal(a["h"][3:, 0], b["h"][3:, 0]) and not np.allclose(a["h"][:3, 0], b["h"][:3, 0])
    assert np.array_equal(a["h"][:, 1], b["h"][:, 1])
    dh_late = dh.copy(); dh_late[:3] = 0.0
    g = G.gru_sequence_backward(p, a, dh_late)
    assert np.all(g["x"][:3, 0] == 0.0) and np.all(g["h0"][0] == 0.0)
    assert np.any(g["x"][:3, 1] != 0.0) and np.any(g["h0"][1] != 0.0)
    d_last = dones.copy(); d_last[-1, :] = 1
    c = G.gru_sequence_forward(p, x, h0, d_last)
    assert np.array_equal(c["h"], a["h"])


def test_a_rollout_taken_step_by_step_equals_the_rollout_taken_at_once():
    """T calls of one step each, every call carrying the previous state in and flagging the environments whose
    previous step was done, give the states of the single T-step call; and the gradient with respect to a
    flagged carried-in state is zero."""
    flat, x, h0, dones, dh = problem(seed=7, T=6, N=5, D=4, H=3, done_prob=0.4)
    D, H = 4, 3
    p = G.unpack_gru(flat, D, H)
    whole = G.gru_sequence_forward(p, x, h0, dones)
    h, prev_done = h0, np.zeros(5, np.uint8)
    for t in range(6):
        c = G.gru_sequence_forward(p, x[t:t + 1], h, dones[t:t + 1], h0_reset=prev_done)
        h, prev_done = c["h"][0], dones[t]
        np.testing.assert_allclose(h, whole["h"][t], rtol=1e-13, atol=1e-14)
    flags = np.array([1, 0, 0, 1, 0], np.uint8)
    c = G.gru_sequence_forward(p, x, h0, dones, h0_reset=flags)
    g = G.gru_sequence_backward(p, c, dh)
    assert np.all(g["h0"][flags == 1] == 0.0) and np.all(np.abs(g["h0"][flags == 0]).sum(axis=1) > 0)
    h0z = h0.copy(); h0z[flags == 1] = 0.0
    np.testing.assert_array_equal(c["h"], G.gru_sequence_forward(p, x, h0z, dones)["h"])
