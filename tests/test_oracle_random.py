"""Pins for the oracle's counter-based random streams (no GPU)."""
import os

import numpy as np
import pytest

from oracle import ppo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[:4], w[4:6], w[6:]))
    return rows


def test_philox_known_answers():
    """Published known-answer vectors of Philox-4x32-10 (Salmon et al., SC'11)."""
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = O.philox4x32_10(np.array(ctr, dtype=np.uint64), key)
        assert [int(x) for x in got] == want


def test_philox_vectorised_matches_scalar():
    rng = np.random.default_rng(1)
    ctr = rng.integers(0, 2 ** 32, size=(5, 7, 4), dtype=np.uint64)
    out = O.philox4x32_10(ctr, (123, 456))
    for i in range(5):
        for j in range(7):
            assert np.array_equal(out[i, j], O.philox4x32_10(ctr[i, j], (123, 456)))


def test_philox_is_bijective_in_counter_word():
    """Distinct counters give distinct blocks (a Philox block function is a bijection)."""
    ctr = np.zeros((4096, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(4096)
    out = O.philox4x32_10(ctr, (0, 0))
    assert len({tuple(r) for r in out.tolist()}) == 4096


def test_uniform_open_interval_and_float32_exact():
    bits = np.array([0, 1, 511, 512, 2 ** 31, 2 ** 32 - 1], dtype=np.uint32)
    u = O.uniform_open01(bits)
    assert np.all(u > 0.0) and np.all(u < 1.0)
    assert u[0] == 2.0 ** -24 and u[-1] == 1.0 - 2.0 ** -24
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)


def test_gaussian_noise_is_box_muller_of_the_philox_words():
    """Invert the transform: radius^2 and angle recover the uniforms of the Philox block."""
    seed, step, N, A = 77, 5, 9, 6
    eps = O.gaussian_noise(seed, step, N, A)
    assert eps.shape == (N, A)
    for n in (0, 4, 8):
        for j in range(2):
            blk = O.philox4x32_10(np.array([n, step, j, 1], dtype=np.uint64), (seed, 0))
            u = ((blk >> np.uint32(9)).astype(np.float64) + 0.5) / 2 ** 23
            z0, z1 = eps[n, 4 * j], eps[n, 4 * j + 1]
            assert np.isclose(np.exp(-(z0 * z0 + z1 * z1) / 2.0), u[0], rtol=1e-12)
            ang = (np.arctan2(z1, z0) / (2 * np.pi)) % 1.0
            assert np.isclose(ang, u[1], atol=1e-12)
            if 4 * j + 3 < A:
                z2, z3 = eps[n, 4 * j + 2], eps[n, 4 * j + 3]
                assert np.isclose(np.exp(-(z2 * z2 + z3 * z3) / 2.0), u[2], rtol=1e-12)
                assert np.isclose((np.arctan2(z3, z2) / (2 * np.pi)) % 1.0, u[3], atol=1e-12)


def test_gaussian_noise_moments_and_independence_across_steps():
    e0 = O.gaussian_noise(0, 0, 20000, 12)
    e1 = O.gaussian_noise(0, 1, 20000, 12)
    x = e0.ravel()
    assert abs(x.mean()) < 0.01
    assert abs(x.var() - 1.0) < 0.02
    assert abs((x ** 4).mean() - 3.0) < 0.1          # Gaussian kurtosis
    assert abs(np.corrcoef(e0.ravel(), e1.ravel())[0, 1]) < 0.01
    assert abs(np.corrcoef(e0[:, 0], e0[:, 1])[0, 1]) < 0.03
    assert not np.array_equal(e0, O.gaussian_noise(1, 0, 20000, 12))


@pytest.mark.parametrize("size", list(range(1, 70)) + [255, 256, 257, 511, 512, 1000, 1024, 1025, 4096, 98304])
def test_permutation_is_a_bijection(size):
    p = O.feistel_permutation(3, 2, 1, size)
    assert p.shape == (size,)
    assert np.array_equal(np.sort(p), np.arange(size))


def test_permutation_changes_with_epoch_iteration_seed_and_mixes():
    B = 4096
    base = O.feistel_permutation(0, 0, 0, B)
    for other in (O.feistel_permutation(0, 0, 1, B), O.feistel_permutation(0, 1, 0, B),
                  O.feistel_permutation(1, 0, 0, B)):
        assert (base == other).mean() < 0.01
    # a shuffle, not a shift: neighbours are scattered and few fixed points remain
    assert (base == np.arange(B)).mean() < 0.01
    assert np.abs(np.diff(base)).mean() > B / 8
    assert O.feistel_permutation(0, 0, 0, 0).size == 0


def test_permutation_matches_per_index_brute_force():
    """Re-derive a few entries with scalar integer code, walking the cycle by hand."""
    seed, it, ep, B = 11, 3, 2, 1000
    p = O.feistel_permutation(seed, it, ep, B)
    bits = 10
    h = bits // 2
    mask = (1 << h) - 1

    def net(x):
        L, R = x >> h, x & mask
        for rnd in range(O.FEISTEL_ROUNDS):
            f = int(O.philox4x32_10(np.array([R, ep, it, 2 | (rnd << 8)], dtype=np.uint64), (seed, 0))[0]) & mask
            L, R = R, L ^ f
        return (L << h) | R

    for i in (0, 1, 17, 512, 999):
        x = net(i)
        while x >= B:
            x = net(x)
        assert x == p[i]
