"""ctypes binding of librslrl_b200.so: the same names as include/rslrl_b200.h, argument
marshalling only.  Every step of the path runs in the library's CUDA kernels; there is no
CPU fallback -- a missing library raises."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

from . import workloads as WL

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "librslrl_b200.so")
LIB_PATH_DEBUG = os.path.join(HERE, "librslrl_b200_debug.so")

RSLRL_MAX_HIDDEN = 8

STATUS = {0: "RSLRL_OK", 1: "RSLRL_ERR_INVALID_ARG", 2: "RSLRL_ERR_SHAPE", 3: "RSLRL_ERR_ALIGNMENT",
          4: "RSLRL_ERR_STATE", 5: "RSLRL_ERR_UNSUPPORTED", 6: "RSLRL_ERR_CUDA", 7: "RSLRL_ERR_NONFINITE",
          8: "RSLRL_ERR_TIMEOUT"}


class RslrlError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status


class ModelCfg(C.Structure):
    _fields_ = [("num_envs", C.c_int32), ("num_steps", C.c_int32), ("actor_obs_dim", C.c_int32),
                ("critic_obs_dim", C.c_int32), ("num_actions", C.c_int32), ("shared_obs", C.c_int32),
                ("num_actor_hidden", C.c_int32), ("actor_hidden", C.c_int32 * RSLRL_MAX_HIDDEN),
                ("num_critic_hidden", C.c_int32), ("critic_hidden", C.c_int32 * RSLRL_MAX_HIDDEN),
                ("elu_alpha", C.c_float), ("precision", C.c_int32)]


class PpoCfg(C.Structure):
    _fields_ = [("gamma", C.c_float), ("lam", C.c_float), ("clip", C.c_float), ("value_clip", C.c_float),
                ("value_coef", C.c_float), ("entropy_coef", C.c_float),
                ("use_clipped_value_loss", C.c_int32), ("epochs", C.c_int32), ("minibatches", C.c_int32),
                ("lr", C.c_float), ("lr_min", C.c_float), ("lr_max", C.c_float), ("lr_factor", C.c_float),
                ("desired_kl", C.c_float), ("adaptive_lr", C.c_int32), ("max_grad_norm", C.c_float),
                ("adam_b1", C.c_float), ("adam_b2", C.c_float), ("adam_eps", C.c_float),
                ("normalize_adv", C.c_int32), ("adv_std_unbiased", C.c_int32), ("adv_eps", C.c_float),
                ("sym_enable", C.c_int32), ("sym_coef", C.c_float),
                ("h_sym_obs_perm", C.c_void_p), ("h_sym_obs_sign", C.c_void_p),
                ("h_sym_cobs_perm", C.c_void_p), ("h_sym_cobs_sign", C.c_void_p),
                ("h_sym_act_perm", C.c_void_p), ("h_sym_act_sign", C.c_void_p),
                ("seed", C.c_uint64)]


class Storage(C.Structure):
    _fields_ = [("T", C.c_int32), ("N", C.c_int32), ("step", C.c_int32), ("obs_a_stride", C.c_int32),
                ("obs_c_stride", C.c_int32), ("act_stride", C.c_int32),
                ("obs_actor", C.c_void_p), ("obs_critic", C.c_void_p), ("actions", C.c_void_p),
                ("mu", C.c_void_p), ("sigma", C.c_void_p), ("logp", C.c_void_p), ("values", C.c_void_p),
                ("rewards", C.c_void_p), ("returns", C.c_void_p), ("advantages", C.c_void_p),
                ("dones", C.c_void_p), ("timeouts", C.c_void_p)]


class UpdateStats(C.Structure):
    _fields_ = [("surrogate", C.c_float), ("value_loss", C.c_float), ("entropy", C.c_float),
                ("sym_loss", C.c_float), ("kl", C.c_float), ("first_surrogate", C.c_float),
                ("first_value_loss", C.c_float), ("first_kl", C.c_float), ("first_sym_loss", C.c_float),
                ("first_grad_norm", C.c_float), ("last_grad_norm", C.c_float), ("lr", C.c_float),
                ("steps", C.c_int32), ("nonfinite", C.c_int32)]

    def as_dict(self) -> Dict[str, float]:
        return {n: getattr(self, n) for n, _ in self._fields_}


class RndCfg(C.Structure):
    _fields_ = [("obs_dim", C.c_int32), ("num_idx", C.c_int32), ("h_idx", C.c_void_p), ("num_hidden", C.c_int32),
                ("hidden", C.c_int32 * 8), ("embed_dim", C.c_int32), ("elu_alpha", C.c_float), ("max_rows", C.c_int32),
                ("lr", C.c_float), ("adam_b1", C.c_float), ("adam_b2", C.c_float), ("adam_eps", C.c_float),
                ("max_batch", C.c_int32), ("max_epochs", C.c_int32), ("max_minibatches", C.c_int32),
                ("precision", C.c_int32)]


class GruCfg(C.Structure):
    _fields_ = [("input_dim", C.c_int32), ("hidden_dim", C.c_int32), ("max_steps", C.c_int32), ("max_envs", C.c_int32),
                ("precision", C.c_int32)]


class Counters(C.Structure):
    _fields_ = [("lr", C.c_float), ("adam_step", C.c_int32), ("global_step", C.c_uint32),
                ("iteration", C.c_uint32)]


EXPORTS = [
    "rslrl_num_params", "rslrl_create", "rslrl_destroy", "rslrl_last_error", "rslrl_storage_view",
    "rslrl_set_params", "rslrl_get_params", "rslrl_get_grads", "rslrl_get_adam", "rslrl_set_adam",
    "rslrl_get_counters", "rslrl_set_counters", "rslrl_act", "rslrl_record_step", "rslrl_gae",
    "rslrl_ppo_update", "rslrl_ppo_update_steps", "rslrl_distill_update", "rslrl_distill_update_steps", "rslrl_act_host", "rslrl_record_step_host",
    "rslrl_gae_host", "rslrl_gae_scratch_bytes", "rslrl_gae_scan", "rslrl_minibatch_indices",
    "rslrl_kernel_launch_count", "rslrl_profile_enable", "rslrl_profile_report", "rslrl_gae_scan_static",
    "rslrl_debug_report",
    "rslrl_rnd_num_params", "rslrl_rnd_create", "rslrl_rnd_destroy", "rslrl_rnd_last_error", "rslrl_rnd_set_params",
    "rslrl_rnd_get_params", "rslrl_rnd_get_grads", "rslrl_rnd_reward", "rslrl_rnd_update",
    "rslrl_gru_num_params", "rslrl_gru_create", "rslrl_gru_destroy", "rslrl_gru_last_error", "rslrl_gru_set_params",
    "rslrl_gru_get_grads", "rslrl_gru_forward", "rslrl_gru_backward",
]

_lib = None


def load_library() -> C.CDLL:
    """Load the CUDA library; fail loudly when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    # RSLRL_B200_DEBUG_LIBRARY=1 selects the checking build (python -m paper_2509_10771_b200.build --debug)
    path = LIB_PATH_DEBUG if os.environ.get("RSLRL_B200_DEBUG_LIBRARY") == "1" else LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run `python -m paper_2509_10771_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(path)
    vp, i32, u32, u64, f32, sz = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_float, C.c_size_t
    sig = {
        "rslrl_num_params": (sz, [C.POINTER(ModelCfg)]),
        "rslrl_debug_report": (i32, [C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]),
        "rslrl_create": (i32, [C.POINTER(ModelCfg), C.POINTER(PpoCfg), vp, C.POINTER(vp)]),
        "rslrl_destroy": (i32, [vp]),
        "rslrl_last_error": (C.c_char_p, [vp]),
        "rslrl_storage_view": (i32, [vp, C.POINTER(Storage)]),
        "rslrl_set_params": (i32, [vp, vp, sz]),
        "rslrl_get_params": (i32, [vp, vp, sz]),
        "rslrl_get_grads": (i32, [vp, vp, sz]),
        "rslrl_get_adam": (i32, [vp, vp, vp, sz]),
        "rslrl_set_adam": (i32, [vp, vp, vp, sz]),
        "rslrl_get_counters": (i32, [vp, C.POINTER(Counters)]),
        "rslrl_set_counters": (i32, [vp, C.POINTER(Counters)]),
        "rslrl_act": (i32, [vp, vp, vp, vp]),
        "rslrl_record_step": (i32, [vp, vp, vp, vp]),
        "rslrl_gae": (i32, [vp, vp]),
        "rslrl_ppo_update": (i32, [vp, C.POINTER(UpdateStats)]),
        "rslrl_ppo_update_steps": (i32, [vp, i32, C.POINTER(UpdateStats)]),
        "rslrl_distill_update": (i32, [vp, vp, C.POINTER(UpdateStats)]),
        "rslrl_distill_update_steps": (i32, [vp, vp, i32, C.POINTER(UpdateStats)]),
        "rslrl_act_host": (i32, [vp, vp, vp, vp]),
        "rslrl_record_step_host": (i32, [vp, vp, vp, vp]),
        "rslrl_gae_host": (i32, [vp, vp]),
        "rslrl_gae_scratch_bytes": (sz, [i32, i32]),
        "rslrl_gae_scan": (i32, [vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, i32, i32, f32, vp, vp]),
        "rslrl_minibatch_indices": (i32, [u64, u32, u32, i32, i32, i32, vp, vp]),
        "rslrl_gae_scan_static": (i32, [vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, i32, i32, f32, vp]),
        "rslrl_kernel_launch_count": (u64, []),
        "rslrl_profile_enable": (i32, [i32]),
        "rslrl_profile_report": (i32, [C.c_char_p, sz]),
        "rslrl_rnd_num_params": (sz, [C.POINTER(RndCfg)]),
        "rslrl_rnd_create": (i32, [C.POINTER(RndCfg), vp, C.POINTER(vp)]),
        "rslrl_rnd_destroy": (i32, [vp]),
        "rslrl_rnd_last_error": (C.c_char_p, [vp]),
        "rslrl_rnd_set_params": (i32, [vp, vp, vp, sz]),
        "rslrl_rnd_get_params": (i32, [vp, vp, sz]),
        "rslrl_rnd_get_grads": (i32, [vp, vp, sz]),
        "rslrl_rnd_reward": (i32, [vp, vp, i32, i32, f32, vp, vp]),
        "rslrl_rnd_update": (i32, [vp, vp, i32, i32, i32, i32, u64, u32, i32, C.POINTER(f32), C.POINTER(f32)]),
        "rslrl_gru_num_params": (sz, [C.POINTER(GruCfg)]),
        "rslrl_gru_create": (i32, [C.POINTER(GruCfg), vp, C.POINTER(vp)]),
        "rslrl_gru_destroy": (i32, [vp]),
        "rslrl_gru_last_error": (C.c_char_p, [vp]),
        "rslrl_gru_set_params": (i32, [vp, vp, sz]),
        "rslrl_gru_get_grads": (i32, [vp, vp, sz]),
        "rslrl_gru_forward": (i32, [vp, vp, i32, vp, vp, vp, i32, i32, vp]),
        "rslrl_gru_backward": (i32, [vp, vp, vp, i32, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    """Device pointer of a torch tensor, host pointer of a numpy array, an int, or None."""
    if x is None:
        return None
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    if isinstance(x, int):
        return x
    assert x.is_contiguous()
    return x.data_ptr()


def model_cfg(w: WL.Workload, precision: Optional[int] = None) -> ModelCfg:
    m = ModelCfg()
    m.num_envs, m.num_steps = w.num_envs, w.num_steps
    m.actor_obs_dim, m.critic_obs_dim, m.num_actions = w.actor_obs_dim, w.critic_obs_dim, w.num_actions
    m.shared_obs = int(w.shared_obs)
    m.num_actor_hidden, m.num_critic_hidden = len(w.actor_hidden), len(w.critic_hidden)
    for i, h in enumerate(w.actor_hidden):
        m.actor_hidden[i] = h
    for i, h in enumerate(w.critic_hidden):
        m.critic_hidden[i] = h
    m.elu_alpha = w.elu_alpha
    m.precision = w.precision if precision is None else precision
    return m


def ppo_cfg(w: WL.Workload, mirror: Optional[Dict[str, np.ndarray]] = None, keep=None) -> PpoCfg:
    p = PpoCfg()
    for name in ("gamma", "lam", "clip", "value_clip", "value_coef", "entropy_coef", "epochs", "minibatches",
                 "lr", "lr_min", "lr_max", "lr_factor", "desired_kl", "max_grad_norm", "adam_b1", "adam_b2",
                 "adam_eps", "adv_eps", "sym_coef"):
        setattr(p, name, getattr(w, name))
    p.use_clipped_value_loss = int(w.use_clipped_value_loss)
    p.adaptive_lr = int(w.adaptive_lr)
    p.normalize_adv = int(w.normalize_adv)
    p.adv_std_unbiased = int(w.adv_std_unbiased)
    p.sym_enable = int(w.sym_enable)
    p.seed = w.seed
    if w.sym_enable:
        assert mirror is not None
        for key, field, dt in (("obs_perm", "h_sym_obs_perm", np.int32), ("obs_sign", "h_sym_obs_sign", np.float32),
                               ("cobs_perm", "h_sym_cobs_perm", np.int32), ("cobs_sign", "h_sym_cobs_sign", np.float32),
                               ("act_perm", "h_sym_act_perm", np.int32), ("act_sign", "h_sym_act_sign", np.float32)):
            arr = np.ascontiguousarray(mirror[key], dtype=dt)
            if keep is not None:
                keep.append(arr)
            setattr(p, field, arr.ctypes.data)
    return p


class Context:
    """One rslrl_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, w: WL.Workload, precision: Optional[int] = None, mirror=None, stream: int = 0):
        self.lib = load_library()
        self.w = w
        self._keep = []
        self.mc = model_cfg(w, precision)
        self.pc = ppo_cfg(w, mirror, self._keep)
        self.handle = C.c_void_p()
        st = self.lib.rslrl_create(C.byref(self.mc), C.byref(self.pc), C.c_void_p(stream), C.byref(self.handle))
        if st != 0:
            raise RslrlError(st, self.lib.rslrl_last_error(None).decode())
        self.num_params = int(self.lib.rslrl_num_params(C.byref(self.mc)))

    def _check(self, st: int):
        if st != 0:
            raise RslrlError(st, self.lib.rslrl_last_error(self.handle).decode())

    def destroy(self):
        if self.handle:
            self.lib.rslrl_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # ---- state -------------------------------------------------------------------------
    def storage_view(self) -> Storage:
        s = Storage()
        self._check(self.lib.rslrl_storage_view(self.handle, C.byref(s)))
        return s

    def set_params(self, flat: np.ndarray):
        flat = np.ascontiguousarray(flat, dtype=np.float32)
        self._check(self.lib.rslrl_set_params(self.handle, flat.ctypes.data, flat.size))

    def _get(self, fn) -> np.ndarray:
        out = np.empty(self.num_params, dtype=np.float32)
        self._check(fn(self.handle, out.ctypes.data, out.size))
        return out

    def get_params(self) -> np.ndarray:
        return self._get(self.lib.rslrl_get_params)

    def get_grads(self) -> np.ndarray:
        return self._get(self.lib.rslrl_get_grads)

    def get_adam(self):
        m = np.empty(self.num_params, dtype=np.float32)
        v = np.empty(self.num_params, dtype=np.float32)
        self._check(self.lib.rslrl_get_adam(self.handle, m.ctypes.data, v.ctypes.data, m.size))
        return m, v

    def set_adam(self, m: np.ndarray, v: np.ndarray):
        m = np.ascontiguousarray(m, dtype=np.float32)
        v = np.ascontiguousarray(v, dtype=np.float32)
        self._check(self.lib.rslrl_set_adam(self.handle, m.ctypes.data, v.ctypes.data, m.size))

    def get_counters(self) -> Counters:
        c = Counters()
        self._check(self.lib.rslrl_get_counters(self.handle, C.byref(c)))
        return c

    def set_counters(self, lr: float, adam_step: int, global_step: int, iteration: int):
        c = Counters(lr, adam_step, global_step, iteration)
        self._check(self.lib.rslrl_set_counters(self.handle, C.byref(c)))

    # ---- the path ------------------------------------------------------------------------
    def act(self, d_actor_obs, d_critic_obs=None, d_actions_out=None):
        self._check(self.lib.rslrl_act(self.handle, _ptr(d_actor_obs), _ptr(d_critic_obs), _ptr(d_actions_out)))

    def record_step(self, d_rewards, d_dones, d_timeouts):
        self._check(self.lib.rslrl_record_step(self.handle, _ptr(d_rewards), _ptr(d_dones), _ptr(d_timeouts)))

    def gae(self, d_last_critic_obs):
        self._check(self.lib.rslrl_gae(self.handle, _ptr(d_last_critic_obs)))

    def ppo_update(self, want_stats: bool = True, max_steps: int = 0) -> Optional[Dict[str, float]]:
        st = UpdateStats()
        ref = C.byref(st) if want_stats else None
        if max_steps > 0:
            self._check(self.lib.rslrl_ppo_update_steps(self.handle, max_steps, ref))
        else:
            self._check(self.lib.rslrl_ppo_update(self.handle, ref))
        return st.as_dict() if want_stats else None

    def distill_update(self, d_expert_actions, want_stats: bool = True, max_steps: int = 0) -> Optional[Dict[str, float]]:
        """rslrl_distill_update: the student's mean regressed on d_expert_actions [T][N][act_stride]."""
        st = UpdateStats()
        ref = C.byref(st) if want_stats else None
        self._check(self.lib.rslrl_distill_update_steps(self.handle, _ptr(d_expert_actions), max_steps, ref))
        return st.as_dict() if want_stats else None

    def act_host(self, h_actor_obs: np.ndarray, h_critic_obs=None, h_actions_out=None):
        self._check(self.lib.rslrl_act_host(self.handle, _ptr(h_actor_obs), _ptr(h_critic_obs), _ptr(h_actions_out)))

    def record_step_host(self, h_rewards, h_dones, h_timeouts):
        self._check(self.lib.rslrl_record_step_host(self.handle, _ptr(h_rewards), _ptr(h_dones), _ptr(h_timeouts)))

    def gae_host(self, h_last_critic_obs):
        self._check(self.lib.rslrl_gae_host(self.handle, _ptr(h_last_critic_obs)))


class Rnd:
    """One rslrl_rnd: target and predictor MLPs on the entries ``idx`` of an observation row."""

    def __init__(self, obs_dim: int, idx, hidden, embed_dim: int, max_rows: int, lr: float = 1e-3, elu_alpha: float = 1.0,
                 adam_b1: float = 0.9, adam_b2: float = 0.999, adam_eps: float = 1e-8, stream: int = 0,
                 max_batch: int = 0, max_epochs: int = 8, max_minibatches: int = 16, precision: int = 0):
        # max_batch = 0: room for max_minibatches minibatches of max_rows rows
        self.lib = load_library()
        self.handle = None
        self._idx = np.ascontiguousarray(idx, dtype=np.int32)
        cfg = RndCfg()
        cfg.obs_dim, cfg.num_idx, cfg.h_idx = obs_dim, self._idx.size, self._idx.ctypes.data
        cfg.num_hidden = len(hidden)
        for i, h in enumerate(hidden):
            cfg.hidden[i] = h
        cfg.embed_dim, cfg.elu_alpha, cfg.max_rows = embed_dim, elu_alpha, max_rows
        cfg.lr, cfg.adam_b1, cfg.adam_b2, cfg.adam_eps = lr, adam_b1, adam_b2, adam_eps
        cfg.max_batch = max_batch if max_batch > 0 else max_rows * max_minibatches
        cfg.max_epochs, cfg.max_minibatches = max_epochs, max_minibatches
        cfg.precision = precision
        self.num_params = int(self.lib.rslrl_rnd_num_params(C.byref(cfg)))
        h = C.c_void_p()
        st = self.lib.rslrl_rnd_create(C.byref(cfg), stream, C.byref(h))
        if st != 0:
            raise RslrlError(st, (self.lib.rslrl_rnd_last_error(None) or b"").decode())
        self.handle = h

    def _check(self, st: int):
        if st != 0:
            raise RslrlError(st, (self.lib.rslrl_rnd_last_error(self.handle) or b"").decode())

    def destroy(self):
        if self.handle is not None:
            self.lib.rslrl_rnd_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def set_params(self, predictor: np.ndarray, target: np.ndarray):
        f = np.ascontiguousarray(predictor, dtype=np.float32)
        g = np.ascontiguousarray(target, dtype=np.float32)
        self._check(self.lib.rslrl_rnd_set_params(self.handle, f.ctypes.data, g.ctypes.data, f.size))

    def get_params(self) -> np.ndarray:
        out = np.empty(self.num_params, dtype=np.float32)
        self._check(self.lib.rslrl_rnd_get_params(self.handle, out.ctypes.data, out.size))
        return out

    def get_grads(self) -> np.ndarray:
        out = np.empty(self.num_params, dtype=np.float32)
        self._check(self.lib.rslrl_rnd_get_grads(self.handle, out.ctypes.data, out.size))
        return out

    def reward(self, d_obs, rows: int, obs_stride: int, weight: float = 0.0, d_rewards_inout=None, d_r_int_out=None):
        self._check(self.lib.rslrl_rnd_reward(self.handle, _ptr(d_obs), rows, obs_stride, weight, _ptr(d_rewards_inout),
                                              _ptr(d_r_int_out)))

    def update(self, d_obs, batch: int, obs_stride: int, epochs: int, minibatches: int, seed: int, iteration: int,
               max_steps: int = 0, want_loss: bool = True):
        mean, first = C.c_float(0), C.c_float(0)
        self._check(self.lib.rslrl_rnd_update(self.handle, _ptr(d_obs), batch, obs_stride, epochs, minibatches, seed,
                                              iteration, max_steps, C.byref(mean) if want_loss else None,
                                              C.byref(first) if want_loss else None))
        return {"mean_loss": mean.value, "first_loss": first.value} if want_loss else None


class Gru:
    """One rslrl_gru: a GRU memory layer over time-major rollouts with state resets and BPTT."""

    def __init__(self, input_dim: int, hidden_dim: int, max_steps: int, max_envs: int, stream: int = 0,
                 precision: int = 0):
        self.lib = load_library()
        self.handle = None
        cfg = GruCfg(input_dim, hidden_dim, max_steps, max_envs, precision)
        self.num_params = int(self.lib.rslrl_gru_num_params(C.byref(cfg)))
        h = C.c_void_p()
        st = self.lib.rslrl_gru_create(C.byref(cfg), stream, C.byref(h))
        if st != 0:
            raise RslrlError(st, (self.lib.rslrl_gru_last_error(None) or b"").decode())
        self.handle = h

    def _check(self, st: int):
        if st != 0:
            raise RslrlError(st, (self.lib.rslrl_gru_last_error(self.handle) or b"").decode())

    def destroy(self):
        if self.handle is not None:
            self.lib.rslrl_gru_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def set_params(self, flat: np.ndarray):
        f = np.ascontiguousarray(flat, dtype=np.float32)
        self._check(self.lib.rslrl_gru_set_params(self.handle, f.ctypes.data, f.size))

    def get_grads(self) -> np.ndarray:
        out = np.empty(self.num_params, dtype=np.float32)
        self._check(self.lib.rslrl_gru_get_grads(self.handle, out.ctypes.data, out.size))
        return out

    def forward(self, d_x, x_stride: int, d_h0, d_dones, T: int, N: int, d_h_out, d_h0_reset=None):
        self._check(self.lib.rslrl_gru_forward(self.handle, _ptr(d_x), x_stride, _ptr(d_h0), _ptr(d_h0_reset), _ptr(d_dones),
                                               T, N, _ptr(d_h_out)))

    def backward(self, d_dh, d_dx=None, dx_stride: int = 0, d_dh0=None):
        self._check(self.lib.rslrl_gru_backward(self.handle, _ptr(d_dh), _ptr(d_dx), dx_stride, _ptr(d_dh0)))


def gae_scan(d_rewards, d_values, d_dones, d_timeouts, d_last_values, d_returns, d_advantages, T: int, N: int,
             gamma: float, lam: float, normalize: bool, unbiased: bool, adv_eps: float, d_scratch, stream: int = 0):
    lib = load_library()
    st = lib.rslrl_gae_scan(_ptr(d_rewards), _ptr(d_values), _ptr(d_dones), _ptr(d_timeouts), _ptr(d_last_values),
                            _ptr(d_returns), _ptr(d_advantages), T, N, gamma, lam, int(normalize), int(unbiased),
                            adv_eps, _ptr(d_scratch), C.c_void_p(stream))
    if st != 0:
        raise RslrlError(st, "rslrl_gae_scan")


def debug_report():
    """(is the checking build loaded, damaged guard regions, worst index-fault code); synchronises the device."""
    lib = load_library()
    a, b, c = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    st = lib.rslrl_debug_report(C.byref(a), C.byref(b), C.byref(c))
    if st != 0:
        raise RslrlError(st, "rslrl_debug_report")
    return bool(a.value), int(b.value), int(c.value)


GAE_STATIC_MAX_ENVS = 1048576


def gae_scan_static(d_rewards, d_values, d_dones, d_timeouts, d_last_values, d_returns, d_advantages, T: int, N: int,
                    gamma: float, lam: float, normalize: bool, unbiased: bool, adv_eps: float, stream: int = 0):
    """rslrl_gae_scan_static: the GAE scan with its scratch inside the library, for callers that
    cannot allocate device memory.  At most GAE_STATIC_MAX_ENVS environments."""
    lib = load_library()
    st = lib.rslrl_gae_scan_static(_ptr(d_rewards), _ptr(d_values), _ptr(d_dones), _ptr(d_timeouts),
                                   _ptr(d_last_values), _ptr(d_returns), _ptr(d_advantages), T, N, gamma, lam,
                                   int(normalize), int(unbiased), adv_eps, C.c_void_p(stream))
    if st != 0:
        raise RslrlError(st, lib.rslrl_last_error(None).decode() or "rslrl_gae_scan_static")


def gae_scratch_bytes(T: int, N: int) -> int:
    return int(load_library().rslrl_gae_scratch_bytes(T, N))


def minibatch_indices(seed: int, iteration: int, epoch: int, batch: int, minibatches: int, k: int, d_rows_out,
                      stream: int = 0):
    st = load_library().rslrl_minibatch_indices(seed, iteration, epoch, batch, minibatches, k, _ptr(d_rows_out),
                                                C.c_void_p(stream))
    if st != 0:
        raise RslrlError(st, "rslrl_minibatch_indices")


def kernel_launch_count() -> int:
    return int(load_library().rslrl_kernel_launch_count())


def profile_enable(on: bool):
    load_library().rslrl_profile_enable(int(on))


def profile_report() -> Dict[str, Dict[str, float]]:
    """{kernel family: {"launches": n, "ms": total}} of the launches recorded since the last report."""
    buf = C.create_string_buffer(1 << 16)
    st = load_library().rslrl_profile_report(buf, len(buf))
    if st != 0:
        raise RslrlError(st, "rslrl_profile_report")
    out = {}
    for line in buf.value.decode().splitlines():
        name, n, ms = line.split()
        out[name] = {"launches": int(n), "ms": float(ms)}
    return out
