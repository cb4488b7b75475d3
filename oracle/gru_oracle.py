"""CPU oracle of a recurrent (GRU) memory layer over a rollout with explicit hidden-state management and
back-propagation through time (paper: "Implementation Details", recurrent networks for the RL and the
distillation setting).  Test infrastructure only: plain numpy in float64, one time step after the other,
written from the gate equations below; nothing of the CUDA path is imported and nothing here is used by
the product path.

The paper names the feature but neither the cell nor the reset rule, so the reading is:

  * the cell is a GRU (Cho et al. 2014) in the common gate convention
        r = sigmoid(x W_ir + b_ir + h W_hr + b_hr)
        z = sigmoid(x W_iz + b_iz + h W_hz + b_hz)
        n = tanh   (x W_in + b_in + r * (h W_hn + b_hn))
        h' = (1 - z) * n + z * h
    with W_i = [W_ir | W_iz | W_in] of shape [D][3H] and W_h = [W_hr | W_hz | W_hn] of shape [H][3H];
  * sequences are time-major, x[T][N][D]; the state entering step 0 is h0[N][H] (carried over from the
    previous rollout by the caller); with same-step resets an environment that reports done at step t
    starts step t + 1 from the zero state: h_in(t) = (1 - done[t-1]) * h(t-1) for t >= 1; the same rule at
    the seam between two calls is an optional flag vector that zeroes carried-in states;
  * back-propagation runs through all T steps of the rollout and stops where the state was reset
    (the factor (1 - done) carries that), and it returns the gradient with respect to h0.

Pins (tests/test_gru_oracle.py): torch.nn.GRU forward and autograd without resets (library routine),
a torch GRUCell loop with masked states under autograd with resets, central finite differences, the
one-step closed form, and independence of everything after a reset from everything before it.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

F64 = np.float64


def sigmoid(a: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-a))


def unpack_gru(flat: np.ndarray, D: int, H: int) -> Dict[str, np.ndarray]:
    """W_i[D][3H], b_i[3H], W_h[H][3H], b_h[3H] from the flat order W_i, b_i, W_h, b_h (gate order r, z, n)."""
    flat = np.asarray(flat, dtype=F64)
    sizes = [D * 3 * H, 3 * H, H * 3 * H, 3 * H]
    assert flat.size == sum(sizes), (flat.size, sum(sizes))
    o = np.cumsum([0] + sizes)
    return {"W_i": flat[o[0]:o[1]].reshape(D, 3 * H), "b_i": flat[o[1]:o[2]],
            "W_h": flat[o[2]:o[3]].reshape(H, 3 * H), "b_h": flat[o[3]:o[4]]}


def gru_sequence_forward(p: Dict[str, np.ndarray], x: np.ndarray, h0: np.ndarray, dones: np.ndarray,
                         h0_reset: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """h[T][N][H] (the state after every step) and what the backward pass needs.  ``h0_reset[N]`` (optional) marks
    environments whose step before this sequence reported done: their carried-in state is replaced by zero, which
    is what makes a rollout taken one step per call equal to the same rollout taken in one call."""
    x = np.asarray(x, dtype=F64); h0 = np.asarray(h0, dtype=F64)
    T, N, _ = x.shape
    H = h0.shape[1]
    keep = 1.0 - np.asarray(dones, dtype=F64)                    # [T][N]
    keep0 = np.ones(N) if h0_reset is None else 1.0 - np.asarray(h0_reset, dtype=F64)
    h0 = keep0[:, None] * h0
    out = {k: np.zeros((T, N, H)) for k in ("h", "h_in", "r", "z", "n", "gh_n")}
    h = h0
    for t in range(T):
        h_in = h if t == 0 else keep[t - 1][:, None] * h
        gi = x[t] @ p["W_i"] + p["b_i"]
        gh = h_in @ p["W_h"] + p["b_h"]
        r = sigmoid(gi[:, :H] + gh[:, :H])
        z = sigmoid(gi[:, H:2 * H] + gh[:, H:2 * H])
        n = np.tanh(gi[:, 2 * H:] + r * gh[:, 2 * H:])
        h = (1.0 - z) * n + z * h_in
        for k, v in (("h", h), ("h_in", h_in), ("r", r), ("z", z), ("n", n), ("gh_n", gh[:, 2 * H:])):
            out[k][t] = v
    out["x"] = x
    out["keep"] = keep
    out["keep0"] = keep0
    return out


def gru_sequence_backward(p: Dict[str, np.ndarray], c: Dict[str, np.ndarray], dh_seq: np.ndarray) -> Dict[str, np.ndarray]:
    """Gradients of L = sum_t <dh_seq[t], h[t]> with respect to x, h0 and the four parameter arrays."""
    dh_seq = np.asarray(dh_seq, dtype=F64)
    T, N, H = dh_seq.shape
    x = c["x"]
    g = {"W_i": np.zeros_like(p["W_i"]), "b_i": np.zeros_like(p["b_i"]), "W_h": np.zeros_like(p["W_h"]),
         "b_h": np.zeros_like(p["b_h"]), "x": np.zeros_like(x)}
    carry = np.zeros((N, H))                                     # dL/dh(t) arriving from step t + 1
    for t in range(T - 1, -1, -1):
        dh = dh_seq[t] + carry
        r, z, n, gh_n, h_in = c["r"][t], c["z"][t], c["n"][t], c["gh_n"][t], c["h_in"][t]
        da_n = dh * (1.0 - z) * (1.0 - n * n)
        da_z = dh * (h_in - n) * z * (1.0 - z)
        da_r = da_n * gh_n * r * (1.0 - r)
        dgi = np.concatenate([da_r, da_z, da_n], axis=1)
        dgh = np.concatenate([da_r, da_z, da_n * r], axis=1)
        g["W_i"] += x[t].T @ dgi; g["b_i"] += dgi.sum(axis=0)
        g["W_h"] += h_in.T @ dgh; g["b_h"] += dgh.sum(axis=0)
        g["x"][t] = dgi @ p["W_i"].T
        dh_in = dh * z + dgh @ p["W_h"].T
        carry = dh_in if t == 0 else c["keep"][t - 1][:, None] * dh_in
    g["h0"] = c["keep0"][:, None] * carry
    return g


def flat_grads(g: Dict[str, np.ndarray]) -> np.ndarray:
    return np.concatenate([g["W_i"].ravel(), g["b_i"], g["W_h"].ravel(), g["b_h"]])
