"""rslrl_gae_scan_static -- the allocation-free GAE entry point -- against rslrl_gae_scan and
against the oracle.

The static variant exists for hosts that cannot get device memory while they run (see the
header).  It runs the same scan, so on the same inputs it must reproduce the regular entry
point, and like it the oracle's GAE and advantage normalisation; calls in a row check that what
one call leaves in the shared scratch array does not leak into the next, and that a call after
the first leaves the amount of free device memory as it found it.  This file sorts last on purpose: it exercises an optional
addition, and a run that stops at the first failure should have seen every other test first.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _inputs(T, N, seed):
    rng = np.random.default_rng(seed)
    r = rng.normal(0, 0.5, (T, N)).astype(np.float32)
    v = rng.normal(0, 1.0, (T, N)).astype(np.float32)
    lv = rng.normal(0, 1.0, N).astype(np.float32)
    d = (rng.random((T, N)) < 0.02).astype(np.uint8)
    to = (d & (rng.random((T, N)) < 0.5)).astype(np.uint8)
    return r, v, d, to, lv


def test_static_gae_matches_regular_entry_point_on_two_calls_in_a_row():
    import torch
    from oracle import ppo_oracle as O
    from paper_2509_10771_b200 import binding
    from parity_utils import assert_close

    dev = lambda x: torch.from_numpy(x).cuda()
    binding.gae_scan_static(None, None, None, None, None, None, None, 0, 0, 0.99, 0.95, True, True, 1e-8)   # start-up call
    # a large call first, then a smaller one with other data: stale triples of the first call
    # sit beyond the blocks the second call uses and must not influence it
    for T, N, seed, normalize in ((24, 40000, 1, True), (8, 1000, 2, True), (5, 130, 3, False)):
        host = _inputs(T, N, seed)
        r, v, d, to, lv = (dev(x) for x in host)
        ret_a = torch.empty((T, N), device="cuda"); adv_a = torch.empty((T, N), device="cuda")
        ret_b = torch.empty((T, N), device="cuda"); adv_b = torch.empty((T, N), device="cuda")
        scratch = torch.empty(binding.gae_scratch_bytes(T, N), dtype=torch.uint8, device="cuda")
        binding.gae_scan(r, v, d, to, lv, ret_a, adv_a, T, N, 0.99, 0.95, normalize, True, 1e-8, scratch)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        binding.gae_scan_static(r, v, d, to, lv, ret_b, adv_b, T, N, 0.99, 0.95, normalize, True, 1e-8)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before          # the call took no device memory
        assert_close(ret_b.cpu().numpy(), ret_a.cpu().numpy(), 1e-5, "returns")
        assert_close(adv_b.cpu().numpy(), adv_a.cpu().numpy(), 1e-5, "advantages")
        want_ret, want_adv = O.gae(host[0], host[1], host[2], host[3], host[4], 0.99, 0.95)
        if normalize:
            want_adv = O.normalize_advantages(want_adv, 1e-8, True)
        assert_close(ret_b.cpu().numpy(), want_ret, 1e-5, "returns vs oracle")
        assert_close(adv_b.cpu().numpy(), want_adv, 1e-5, "advantages vs oracle")


def test_static_gae_at_its_largest_size():
    """One step over RSLRL_GAE_STATIC_MAX_ENVS environments: the last slot of the scratch array is in use."""
    import torch
    from oracle import ppo_oracle as O
    from paper_2509_10771_b200 import binding
    from parity_utils import assert_close

    T, N = 1, binding.GAE_STATIC_MAX_ENVS
    host = _inputs(T, N, 4)
    r, v, d, to, lv = (torch.from_numpy(x).cuda() for x in host)
    ret = torch.empty((T, N), device="cuda"); adv = torch.empty((T, N), device="cuda")
    binding.gae_scan_static(r, v, d, to, lv, ret, adv, T, N, 0.99, 0.95, True, True, 1e-8)
    torch.cuda.synchronize()
    want_ret, want_adv = O.gae(host[0], host[1], host[2], host[3], host[4], 0.99, 0.95)
    assert_close(ret.cpu().numpy(), want_ret, 1e-5, "returns vs oracle")
    assert_close(adv.cpu().numpy(), O.normalize_advantages(want_adv, 1e-8, True), 1e-5, "advantages vs oracle")


def test_static_gae_rejects_sizes_beyond_its_limit():
    from paper_2509_10771_b200 import binding
    with pytest.raises(binding.RslrlError) as e:
        binding.gae_scan_static(None, None, None, None, None, None, None, 4, binding.GAE_STATIC_MAX_ENVS + 1,
                                0.99, 0.95, True, True, 1e-8)
    assert e.value.status == 5 and "RSLRL_GAE_STATIC_MAX_ENVS" in str(e.value)
    # empty input: nothing to do, nothing launched
    binding.gae_scan_static(None, None, None, None, None, None, None, 0, 0, 0.99, 0.95, True, True, 1e-8)
