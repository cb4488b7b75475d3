"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rslrl_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rslrl_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_path():
    names = declared_functions()
    for must in ("rslrl_create", "rslrl_destroy", "rslrl_act", "rslrl_record_step", "rslrl_gae", "rslrl_ppo_update"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2509_10771_b200 import binding, build
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in include/rslrl_b200.h but not exported"
    assert sorted(binding.EXPORTS) == declared_functions()


def test_binding_structs_match_header_sizes():
    from paper_2509_10771_b200 import binding
    assert ctypes.sizeof(binding.ModelCfg) == 4 * (6 + 1 + 8 + 1 + 8 + 1 + 1)
    assert ctypes.sizeof(binding.Counters) == 16
    assert ctypes.sizeof(binding.UpdateStats) == 4 * 14
    assert ctypes.sizeof(binding.Storage) == 4 * 6 + 8 * 12
    assert binding.PpoCfg.seed.offset % 8 == 0


def test_num_params_and_config_validation_without_a_device():
    from paper_2509_10771_b200 import binding, build, workloads as WL
    build.build()
    lib = binding.load_library()
    for w in WL.CONFIGS:
        mc = binding.model_cfg(w)
        assert lib.rslrl_num_params(ctypes.byref(mc)) == w.num_params()
    bad = binding.model_cfg(WL.TINY)
    bad.num_actions = 0
    assert lib.rslrl_num_params(ctypes.byref(bad)) == 0
    # argument errors are reported before any CUDA call
    handle = ctypes.c_void_p()
    pc = binding.ppo_cfg(WL.TINY)
    assert lib.rslrl_create(ctypes.byref(bad), ctypes.byref(pc), None, ctypes.byref(handle)) == 1
    assert b"num_actions" in lib.rslrl_last_error(None)
    pc.minibatches = 7
    assert lib.rslrl_create(ctypes.byref(binding.model_cfg(WL.TINY)), ctypes.byref(pc), None, ctypes.byref(handle)) == 2
    assert lib.rslrl_gae_scan(None, None, None, None, None, None, None, 0, 0, 0.99, 0.95, 1, 1, 1e-8, None, None) == 0
    assert lib.rslrl_gae_scan(None, None, None, None, None, None, None, 4, 4, 0.99, 0.95, 1, 1, 1e-8, None, None) == 1
    assert lib.rslrl_minibatch_indices(0, 0, 0, 10, 3, 0, None, None) == 2


def test_rnd_and_gru_configs_without_a_device():
    """Parameter counts and config validation of the two side objects are host-only code."""
    import numpy as np
    from paper_2509_10771_b200 import binding, build
    build.build()
    lib = binding.load_library()
    idx = np.array([0, 3, 5], dtype=np.int32)
    cfg = binding.RndCfg()
    cfg.obs_dim, cfg.num_idx, cfg.h_idx, cfg.num_hidden = 8, 3, idx.ctypes.data, 2
    cfg.hidden[0], cfg.hidden[1] = 16, 8
    cfg.embed_dim, cfg.elu_alpha, cfg.max_rows = 4, 1.0, 64
    cfg.lr, cfg.adam_b1, cfg.adam_b2, cfg.adam_eps = 1e-3, 0.9, 0.999, 1e-8
    assert lib.rslrl_rnd_num_params(ctypes.byref(cfg)) == 0       # the update's limits are not set yet
    cfg.max_batch, cfg.max_epochs, cfg.max_minibatches = 256, 5, 4
    assert lib.rslrl_rnd_num_params(ctypes.byref(cfg)) == 3 * 16 + 16 + 16 * 8 + 8 + 8 * 4 + 4
    cfg.num_idx = 9                                    # more selected entries than the observation has
    assert lib.rslrl_rnd_num_params(ctypes.byref(cfg)) == 0
    cfg.num_idx, cfg.lr = 3, 0.0
    assert lib.rslrl_rnd_num_params(ctypes.byref(cfg)) == 0
    cfg.max_epochs, cfg.max_minibatches = 1 << 11, 1 << 10          # more steps than one call may take
    assert lib.rslrl_rnd_num_params(ctypes.byref(cfg)) == 0
    assert ctypes.sizeof(binding.RndCfg) == 4 + 4 + 8 + 4 + 32 + 4 + 4 + 4 + 16 + 12 + 4 and binding.RndCfg.h_idx.offset == 8
    assert binding.RndCfg.max_batch.offset == 80 and binding.RndCfg.precision.offset == 92
    cfg.max_epochs, cfg.max_minibatches, cfg.precision = 5, 4, 7
    assert lib.rslrl_rnd_num_params(ctypes.byref(cfg)) == 0        # no such precision
    g = binding.GruCfg(235, 256, 24, 4096)
    assert lib.rslrl_gru_num_params(ctypes.byref(g)) == 235 * 768 + 768 + 256 * 768 + 768
    assert lib.rslrl_gru_num_params(ctypes.byref(binding.GruCfg(235, 250, 24, 4096))) == 0     # H not a multiple of 4
    assert lib.rslrl_gru_num_params(ctypes.byref(binding.GruCfg(235, 256, 1 << 15, 1 << 15))) == 0   # T * N too large
    assert ctypes.sizeof(binding.GruCfg) == 20 and binding.GruCfg.precision.offset == 16
    assert lib.rslrl_gru_num_params(ctypes.byref(binding.GruCfg(235, 256, 24, 4096, 3))) == 0          # no such precision


def test_side_objects_refuse_the_bf16_mode_without_a_device():
    """The recurrent layer and random network distillation have FP32 and TF32 modes; asking for BF16 is refused by the
    host code before any device call."""
    import numpy as np
    from paper_2509_10771_b200 import binding, build
    build.build()
    lib = binding.load_library()
    h = ctypes.c_void_p()
    g = binding.GruCfg(16, 8, 4, 32, 2)
    assert lib.rslrl_gru_create(ctypes.byref(g), None, ctypes.byref(h)) == 5 and not h.value
    idx = np.array([0, 1], dtype=np.int32)
    cfg = binding.RndCfg()
    cfg.obs_dim, cfg.num_idx, cfg.h_idx, cfg.num_hidden = 4, 2, idx.ctypes.data, 1
    cfg.hidden[0] = 8
    cfg.embed_dim, cfg.elu_alpha, cfg.max_rows = 4, 1.0, 16
    cfg.lr, cfg.adam_b1, cfg.adam_b2, cfg.adam_eps = 1e-3, 0.9, 0.999, 1e-8
    cfg.max_batch, cfg.max_epochs, cfg.max_minibatches, cfg.precision = 16, 1, 1, 2
    assert lib.rslrl_rnd_create(ctypes.byref(cfg), None, ctypes.byref(h)) == 5 and not h.value

