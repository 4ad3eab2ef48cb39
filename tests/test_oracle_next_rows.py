"""Pins for the oracle's wrap-around block scheme and its fused accumulate p = gamma * g + e.

Both are checked against something other than the oracle's own formula: exact rational
arithmetic for the fused multiply-add, and counting / enumeration for the block.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import sparsify_oracle as O


# ---------------------------------------------------------------------------------------------
# fused multiply-add: round(a * b + c) once, against exact arithmetic
# ---------------------------------------------------------------------------------------------
def round_fraction_to_f32(x: Fraction) -> np.float32:
    """Nearest fp32 to an exact rational, ties to even, by bracketing with neighbouring floats."""
    if x == 0:
        return np.float32(0.0)
    guess = np.float32(float(x))                       # within one ulp of the answer
    if np.isinf(guess):
        big = Fraction(float(np.finfo(np.float32).max))
        half_ulp = Fraction(2) ** 103                  # half the spacing at the top binade
        if abs(x) < big + half_ulp:
            return np.float32(np.sign(float(x))) * np.finfo(np.float32).max
        return guess
    cands = {guess, np.nextafter(guess, np.float32(np.inf)), np.nextafter(guess, np.float32(-np.inf))}
    cands = [c for c in cands if np.isfinite(c)]
    best = min(cands, key=lambda c: abs(Fraction(float(c)) - x))
    ties = [c for c in cands if abs(Fraction(float(c)) - x) == abs(Fraction(float(best)) - x)]
    if len(ties) == 2:                                 # exactly half way: the even mantissa wins
        best = [c for c in ties if (np.float32(c).view(np.uint32) & 1) == 0][0]
    return np.float32(best)


def exact_fma(a, b, c):
    return np.array([round_fraction_to_f32(Fraction(float(x)) * Fraction(float(y)) + Fraction(float(z)))
                     for x, y, z in zip(a, b, c)], np.float32)


def bits(x):
    return np.asarray(x, np.float32).view(np.uint32)


def test_fma_matches_exact_arithmetic_on_random_inputs():
    rng = np.random.default_rng(1)
    n = 4000
    a = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 6, n)).astype(np.float32)
    b = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 6, n)).astype(np.float32)
    c = (rng.standard_normal(n) * 10.0 ** rng.uniform(-12, 12, n)).astype(np.float32)
    # make a third of the addends nearly cancel the product (where double rounding would bite)
    c[::3] = -(a[::3].astype(np.float64) * b[::3].astype(np.float64)).astype(np.float32)
    got = O.fma32(a, b, c)
    want = exact_fma(a, b, c)
    assert np.array_equal(bits(got), bits(want))


def test_fma_halfway_cases_need_the_single_rounding():
    # a * b = 1 + 2^-23 + 2^-46 exactly (a = b = 1 + 2^-23 gives 1 + 2^-22 + 2^-46); pick c so that the exact
    # sum sits just above / just below a rounding boundary of fp32, where rounding the product first
    # (two roundings) gives the other neighbour.
    a = np.float32(1.0) + np.float32(2.0 ** -23)
    prod_exact = Fraction(float(a)) ** 2                       # 1 + 2^-22 + 2^-46
    c_vals = np.float32([2.0 ** -24, -(2.0 ** -24), 3 * 2.0 ** -24, 1.0, -1.0, 2.0 ** -47])
    got = O.fma32(np.full(c_vals.size, a), np.full(c_vals.size, a), c_vals)
    want = np.array([round_fraction_to_f32(prod_exact + Fraction(float(c))) for c in c_vals], np.float32)
    assert np.array_equal(bits(got), bits(want))
    two_step = (np.full(c_vals.size, a) * np.full(c_vals.size, a)) + c_vals
    assert not np.array_equal(bits(two_step), bits(want)), "the cases must separate one rounding from two"


def test_fma_special_values_and_unit_step():
    g = np.float32([1.5, -0.0, 0.0, np.inf, 1e-45, 3e38, -3e38, 1.0])
    e = np.float32([2.5, 0.0, -0.0, 1.0, 1e-45, 3e38, 3e38, np.nan])
    with np.errstate(over="ignore"):
        plain = g + e
        assert np.array_equal(bits(O.accumulate(g, e, 1.0)), bits(plain))
    one = O.fma32(np.float32(1.0), g, e)                       # fma(1, g, e) is the plain add, bit for bit
    both_nan = np.isnan(one) & np.isnan(plain)
    assert np.array_equal(bits(one)[~both_nan], bits(plain)[~both_nan])
    assert np.isinf(O.fma32(np.float32(2.0), np.float32([3e38]), np.float32([0.0])))[0]
    # denormal result, exact: 2^-149 * 0.5 + 2^-149 = 1.5 * 2^-149 -> ties to even -> 2 * 2^-149
    tiny = np.float32(2.0 ** -149)
    assert bits(O.fma32(np.float32(0.5), np.float32([tiny]), np.float32([tiny])))[0] == 2


def test_accumulate_with_step_size_feeds_the_compressor():
    rng = np.random.default_rng(5)
    g = rng.standard_normal(500).astype(np.float32)
    e = (rng.standard_normal(500) * 0.1).astype(np.float32)
    gamma = 0.05
    vals, idx, e_new = O.compress(O.TOPK, g, e, 25, seed=3, gamma=gamma)
    p = exact_fma(np.full(500, np.float32(gamma)), g, e)
    order = sorted(range(500), key=lambda i: (-abs(float(p[i])), i))[:25]
    assert sorted(order) == idx.tolist()
    assert np.array_equal(bits(vals), bits(p[idx]))
    rest = p.copy()
    rest[idx] = 0.0
    assert np.array_equal(bits(e_new), bits(rest))


# ---------------------------------------------------------------------------------------------
# wrap-around block
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n,k", [(1, 1), (7, 3), (50, 7), (64, 64), (100, 99), (33, 0)])
def test_wrap_block_is_a_cyclic_interval(n, k):
    p = np.zeros(n, np.float32)
    for seed in range(200):
        idx = O.select(O.RANDBLOCK_WRAP, p, k, seed).astype(np.int64)
        assert idx.size == k and np.all(np.diff(idx) > 0)
        if k == 0:
            continue
        a = O.block_start_wrap(seed, n)
        assert 0 <= a < n
        assert set(idx.tolist()) == {(a + j) % n for j in range(k)}
        if a + k <= n:                                         # no wrap: the plain block
            assert idx.tolist() == list(range(a, a + k))
        else:                                                  # head [0, a+k-n) then tail [a, n)
            assert idx.tolist() == list(range(0, a + k - n)) + list(range(a, n))


def test_wrap_block_keeps_every_coordinate_equally_often():
    n, k, trials = 40, 9, 40000
    p = np.zeros(n, np.float32)
    hits = np.zeros(n)
    starts = np.zeros(n)
    for seed in range(trials):
        s = O.segment_seed(seed, 0)
        hits[O.select(O.RANDBLOCK_WRAP, p, k, s)] += 1
        starts[O.block_start_wrap(s, n)] += 1
    expect = trials * k / n
    chi_hits = float(((hits - expect) ** 2 / expect).sum())
    chi_starts = float(((starts - trials / n) ** 2 / (trials / n)).sum())
    assert chi_starts < 80.0                                   # 39 degrees of freedom, p ~ 1e-4 at 80
    assert chi_hits < 80.0
    # the plain block (no wrap) does NOT have this property: its first coordinate is kept k times less often
    plain = np.zeros(n)
    for seed in range(4000):
        plain[O.select(O.RANDBLOCK, p, k, O.segment_seed(seed, 0))] += 1
    assert plain[0] < 0.4 * plain[n // 2]


def test_wrap_block_shared_seed_and_segments():
    rng = np.random.default_rng(2)
    g = [rng.standard_normal(300).astype(np.float32) for _ in range(3)]
    e = [np.zeros(300, np.float32) for _ in range(3)]
    segs = [(0, 100, 30), (100, 150, 149), (250, 50, 1)]
    vals, idx, res, avg = O.step(O.RANDBLOCK_WRAP, g, e, segs, [9, 9, 9])
    assert all(np.array_equal(idx[0], i) for i in idx)
    for w in range(3):
        full = g[w].copy()
        back = res[w].copy()
        back[idx[w]] += vals[w]
        assert np.array_equal(bits(back), bits(full))          # e' + q^w == p exactly (residual was zero)
    dense = np.zeros(300, np.float32)
    for w in range(3):
        dense[idx[w]] += vals[w]
    assert np.array_equal(bits(avg), bits(dense / np.float32(3)))
