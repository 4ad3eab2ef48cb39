"""Pins for the oracle's coordinate generators (random-k, block-random-k)."""
import numpy as np
import pytest

from oracle import sparsify_oracle as O


def test_mix64_known_structure():
    # SplitMix finaliser: 0 maps to 0, so mix64(a, b) with a + (b+1)*phi == 0 is 0
    phi = 0x9E3779B97F4A7C15
    assert O.mix64((-phi) & (2 ** 64 - 1), 0) == 0
    outs = {O.mix64(7, b) for b in range(1000)}
    assert len(outs) == 1000
    assert all(0 <= v < 2 ** 64 for v in outs)


def test_mix32_scalar_equals_array_and_is_bijective_on_sample():
    xs = np.arange(0, 200000, dtype=np.uint32) * np.uint32(2654435761)
    arr = O.mix32(xs)
    assert [O.mix32(int(x)) for x in xs[:500]] == arr[:500].tolist()
    assert len(np.unique(arr)) == len(xs)        # both multipliers are odd, xorshifts invertible


@pytest.mark.parametrize("seed", [0, 1, 0xDEADBEEFCAFE])
def test_permutation_is_a_bijection_for_every_small_n(seed):
    for n in list(range(1, 300)) + [1023, 1024, 1025, 2047, 2048, 4097, 65536, 65537]:
        pi = O.randk_permute(seed, n, np.arange(n, dtype=np.uint32))
        assert pi.min() >= 0 and pi.max() < n
        assert len(np.unique(pi)) == n, n


def test_feistel_is_invertible_on_full_domain():
    left, right, keys = O.feistel_params(5, 3000)
    dom = 1 << (left + right)
    y = O.feistel_once(np.arange(dom, dtype=np.uint32), left, right, keys)
    assert len(np.unique(y)) == dom and y.max() < dom


def test_randk_indices_distinct_sorted_prefix_property():
    n = 10007
    full = O.randk_permute(11, n, np.arange(n, dtype=np.uint32))
    for k in (0, 1, 100, 5000, n):
        idx = O.randk_indices(11, n, k)
        assert len(idx) == k
        assert np.all(np.diff(idx.astype(np.int64)) > 0)
        assert set(idx.tolist()) == set(full[:k].tolist())       # the first k images of pi


def test_randk_inclusion_frequency_is_uniform():
    """Each coordinate is kept with probability k/n.  Sampling is without
    replacement, so the chi-square statistic over coordinates has mean
    (n-1)(1-k/n) and we test against that."""
    n, k, trials = 1000, 100, 4000
    cnt = np.zeros(n)
    for s in range(trials):
        cnt[O.randk_indices(O.segment_seed(s, 0), n, k)] += 1
    exp = trials * k / n
    chi2 = ((cnt - exp) ** 2 / exp).sum()
    mean = (n - 1) * (1 - k / n)
    sd = np.sqrt(2 * (n - 1)) * (1 - k / n)
    assert abs(chi2 - mean) < 5 * sd, (chi2, mean, sd)


def test_randk_pairs_are_not_locked_together():
    """Two fixed coordinates are kept together about (k/n)^2 of the time."""
    n, k, trials = 64, 16, 6000
    both = 0
    for s in range(trials):
        S = set(O.randk_indices(O.segment_seed(s, 0), n, k).tolist())
        both += (3 in S) and (40 in S)
    p = (k / n) * ((k - 1) / (n - 1))
    assert abs(both / trials - p) < 5 * np.sqrt(p * (1 - p) / trials)


def test_block_start_range_and_limits():
    for n in (1, 2, 10, 1000, 2 ** 32 - 1):
        for k in {0, 1, n // 3, n}:
            for seed in range(20):
                a = O.block_start(seed, n, k)
                assert 0 <= a <= n - k
    assert O.block_start(123, 50, 50) == 0


def test_block_start_is_uniform():
    n, k, trials = 120, 21, 20000
    hist = np.zeros(n - k + 1)
    for s in range(trials):
        hist[O.block_start(O.segment_seed(s, 0), n, k)] += 1
    exp = trials / (n - k + 1)
    chi2 = ((hist - exp) ** 2 / exp).sum()
    dof = n - k
    assert abs(chi2 - dof) < 5 * np.sqrt(2 * dof)


def test_block_is_contiguous_and_shared_for_one_seed():
    rng = np.random.default_rng(0)
    n, k, W = 999, 77, 4
    grads = [rng.standard_normal(n).astype(np.float32) for _ in range(W)]
    res = [np.zeros(n, np.float32) for _ in range(W)]
    vals, idx, res2, out = O.step(O.RANDBLOCK, grads, res, [(0, n, k)], [5] * W)
    assert all(np.array_equal(i, idx[0]) for i in idx)
    assert np.array_equal(np.diff(idx[0].astype(np.int64)), np.ones(k - 1))
    a = int(idx[0][0])
    want = sum(g[a:a + k].astype(np.float64) for g in grads) / W
    assert np.allclose(out[a:a + k], want, rtol=1e-5, atol=1e-6)
    assert not out[:a].any() and not out[a + k:].any()
    # different seeds give different blocks somewhere
    _, idx_b, _, _ = O.step(O.RANDBLOCK, grads, res, [(0, n, k)], [5, 6, 7, 8])
    assert len({int(i[0]) for i in idx_b}) > 1


def test_randk_same_seed_same_coordinates():
    rng = np.random.default_rng(1)
    n, k, W = 5000, 50, 3
    grads = [rng.standard_normal(n).astype(np.float32) for _ in range(W)]
    res = [np.zeros(n, np.float32) for _ in range(W)]
    vals, idx, _, out = O.step(O.RANDK, grads, res, [(0, n, k)], [9] * W)
    assert all(np.array_equal(i, idx[0]) for i in idx)
    want = sum(g[idx[0]].astype(np.float64) for g in grads) / W
    assert np.allclose(out[idx[0]], want, rtol=1e-5, atol=1e-6)


def test_segment_seeds_differ():
    assert len({O.segment_seed(1, s) for s in range(200)}) == 200
