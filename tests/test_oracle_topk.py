"""Pins for the oracle's top-k, residual and multi-step behaviour (CPU only)."""
import struct

import numpy as np
import pytest
import torch

from oracle import sparsify_oracle as O


def f32(x):
    return np.asarray(x, dtype=np.float32)


def brute_topk(p, k):
    """Definition by sorting python tuples: larger |p| bit pattern first, ties to
    the lower index.  Bit pattern taken with struct, independent of numpy views."""
    def key(i):
        bits = struct.unpack("<I", struct.pack("<f", float(p[i])))[0] if not np.isnan(p[i]) \
            else int(np.array(p[i], dtype=np.float32).view(np.uint32))
        return (-(bits & 0x7FFFFFFF), i)
    order = sorted(range(len(p)), key=key)
    return sorted(order[:k])


def adversarial_vectors(rng):
    yield f32([0.0] * 17)
    yield f32([1.0, -1.0] * 9)
    yield f32([0.0, -0.0, 0.0, -0.0, 1e-45, -1e-45, 1e-38, -1e-38])
    yield f32([np.inf, -np.inf, 3.0, -3.0, np.nan, 0.0, 2.0, 2.0, -2.0])
    yield f32(rng.integers(-3, 4, size=64))
    yield f32(rng.standard_normal(97))
    v = f32(rng.standard_normal(128))
    v[::3] = 0.0
    yield v
    yield f32([5.0])


def test_topk_matches_bruteforce_all_k():
    rng = np.random.default_rng(1)
    for p in adversarial_vectors(rng):
        for k in range(len(p) + 1):
            got = O.topk_indices(p, k).tolist()
            assert got == brute_topk(p, k), (p, k)


def test_topk_random_many_sizes():
    rng = np.random.default_rng(2)
    for n in (1, 2, 3, 31, 32, 33, 255, 1000, 4096):
        p = f32(rng.standard_normal(n) * 1e-3)
        p[rng.integers(0, n, size=n // 4)] = p[0]        # plant ties
        for k in sorted({0, 1, n // 100 + 1, n // 2, n - 1, n} & set(range(n + 1))):
            assert O.topk_indices(p, k).tolist() == brute_topk(p, k)


def test_topk_set_equals_torch_topk_on_distinct_magnitudes():
    g = torch.Generator().manual_seed(3)
    for n, k in ((1000, 10), (65536, 655), (300001, 3001)):
        mag = torch.randperm(n, generator=g).to(torch.float32) + 1.0     # all distinct
        sign = torch.randint(0, 2, (n,), generator=g).to(torch.float32) * 2 - 1
        p = (mag * sign * 1e-3).numpy()
        want = set(torch.topk(torch.from_numpy(p).abs(), k).indices.tolist())
        got = O.topk_indices(p, k)
        assert set(got.tolist()) == want
        assert np.all(np.diff(got.astype(np.int64)) > 0)


def test_topk_threshold_property_and_tie_prefix():
    rng = np.random.default_rng(4)
    n, k = 5000, 777
    p = f32(rng.integers(-20, 21, size=n))                # many ties
    S = O.topk_indices(p, k)
    assert len(S) == k
    key = np.abs(p)
    inside = np.zeros(n, bool)
    inside[S] = True
    T = key[inside].min()
    assert key[~inside].max() <= T
    tie = np.nonzero(key == T)[0]
    chosen = inside[tie]
    # among the ties the chosen ones are a prefix in index order
    assert not np.any(~chosen[:-1] & chosen[1:])


def test_k_limits():
    p = f32(np.arange(10) - 4.5)
    assert O.topk_indices(p, 0).size == 0
    assert O.topk_indices(p, 10).tolist() == list(range(10))


@pytest.mark.parametrize("scheme", [O.TOPK, O.RANDK, O.RANDBLOCK])
def test_residual_plus_sent_is_accumulated_gradient(scheme):
    rng = np.random.default_rng(5)
    n, k = 3001, 123
    g = f32(rng.standard_normal(n))
    e = f32(rng.standard_normal(n))
    vals, idx, e2 = O.compress(scheme, g, e, k, seed=99)
    p = g + e
    assert len(idx) == k and len(set(idx.tolist())) == k
    assert np.all(np.diff(idx.astype(np.int64)) > 0)
    q = np.zeros(n, np.float32)
    q[idx] = vals
    assert np.array_equal(e2 + q, p)                                     # e' + q^w == p
    assert np.array_equal(e2[idx].view(np.uint32), np.zeros(k, np.uint32))   # kept entries: +0.0 bits
    rest = np.ones(n, bool)
    rest[idx] = False
    assert np.array_equal(e2[rest].view(np.uint32), p[rest].view(np.uint32))
    assert np.array_equal(vals.view(np.uint32), p[idx].view(np.uint32))


def test_selected_inf_leaves_zero_residual():
    g = f32([np.inf, 1.0, -np.inf, 0.5])
    e = f32([0, 0, 0, 0])
    vals, idx, e2 = O.compress(O.TOPK, g, e, 2, seed=0)
    assert idx.tolist() == [0, 2]
    assert e2.tolist() == [0.0, 1.0, 0.0, 0.5]


def test_denormals_survive_the_add():
    ulp = np.array([1, 1, 0x80000003], np.uint32).view(np.float32)      # 1, 1, -3 denormal ulps
    e = np.array([1, 0, 0], np.uint32).view(np.float32)
    vals, idx, e2 = O.compress(O.TOPK, ulp, e, 1, seed=0)                # p = 2, 1, -3 ulps
    assert idx.tolist() == [2]
    assert vals.view(np.uint32).tolist() == [0x80000003]
    assert e2.view(np.uint32).tolist() == [2, 1, 0]
    vals, idx, e2 = O.compress(O.TOPK, ulp, e, 2, seed=0)
    assert idx.tolist() == [0, 2] and vals.view(np.uint32).tolist() == [2, 0x80000003]


@pytest.mark.parametrize("scheme", [O.TOPK, O.RANDK, O.RANDBLOCK])
def test_telescoping_sum_is_exact_on_integer_gradients(scheme):
    """With integer-valued gradients every fp32 add is exact, so after T steps
    sum_t q_t^w + e_T^w == sum_t g_t^w bit for bit: pins the residual carry."""
    rng = np.random.default_rng(6)
    n, k, T = 2000, 20, 40
    e = np.zeros(n, np.float32)
    sent = np.zeros(n, np.float64)
    total = np.zeros(n, np.float64)
    for t in range(T):
        g = f32(rng.integers(-1024, 1025, size=n))
        total += g
        vals, idx, e = O.compress(scheme, g, e, k, seed=1000 + t)
        sent[idx] += vals
    assert np.array_equal(sent + e, total)
    assert np.abs(e).max() > 0


def test_dense_limit_is_plain_averaging():
    """k = n: every worker sends everything; the step is standard synchronous SGD
    averaging and the residual is identically zero."""
    rng = np.random.default_rng(7)
    W, n = 5, 777
    grads = [f32(rng.standard_normal(n)) for _ in range(W)]
    res = [f32(rng.standard_normal(n)) for _ in range(W)]
    for scheme in (O.TOPK, O.RANDK, O.RANDBLOCK):
        vals, idx, res2, out = O.step(scheme, grads, res, [(0, n, n)], [3] * W)
        want = np.zeros(n, np.float32)
        for w in range(W):
            want = want + (grads[w] + res[w])
        want = want / np.float32(W)
        assert np.array_equal(out, want)
        assert all(not r.any() for r in res2)


def test_single_worker_roundtrip():
    rng = np.random.default_rng(8)
    n, k = 1234, 100
    g, e = f32(rng.standard_normal(n)), f32(rng.standard_normal(n))
    vals, idx, res2, out = O.step(O.TOPK, [g], [e], [(0, n, k)], [0])
    assert np.array_equal(out + res2[0], g + e)


def test_aggregate_bruteforce_and_order():
    rng = np.random.default_rng(9)
    W, n, k = 7, 500, 60
    idx = [np.sort(rng.choice(n, k, replace=False)).astype(np.uint32) for _ in range(W)]
    vals = [f32(rng.standard_normal(k) * 10 ** rng.uniform(-3, 3)) for _ in range(W)]
    out = O.aggregate(vals, idx, n)
    for i in range(n):
        acc = np.float32(0.0)
        for w in range(W):
            hit = np.nonzero(idx[w] == i)[0]
            if hit.size:
                acc = np.float32(acc + vals[w][hit[0]])
        assert out[i] == np.float32(acc / np.float32(W))
    # a lone -0.0 aggregates to +0.0, untouched entries are +0.0
    o2 = O.aggregate([f32([-0.0])], [np.array([1], np.uint32)], 3)
    assert o2.view(np.uint32).tolist() == [0, 0, 0]


def test_segments_layerwise_vs_manual():
    rng = np.random.default_rng(10)
    sizes = [5, 64, 1, 300, 33]
    segs, off = [], 0
    for s in sizes:
        segs.append((off, s, (s + 9) // 10))
        off += s
    g, e = f32(rng.standard_normal(off)), f32(rng.standard_normal(off))
    for scheme in (O.TOPK, O.RANDK, O.RANDBLOCK):
        vals, idx, e2 = O.compress_segments(scheme, g, e, segs, seed=42)
        pos = 0
        for s, (o, n_s, k_s) in enumerate(segs):
            p = g[o:o + n_s] + e[o:o + n_s]
            sel = O.select(scheme, p, k_s, O.segment_seed(42, s))
            assert idx[pos:pos + k_s].tolist() == (sel + o).tolist()
            assert np.array_equal(vals[pos:pos + k_s], p[sel])
            pos += k_s
        assert pos == len(idx)


def test_aggregate_apply_is_dense_subtraction_and_leaves_the_rest_alone():
    rng = np.random.default_rng(11)
    W, n, k = 6, 400, 37
    idx = [np.sort(rng.choice(n, k, replace=False)).astype(np.uint32) for _ in range(W)]
    vals = [f32(rng.standard_normal(k)) for _ in range(W)]
    x = f32(rng.standard_normal(n))
    x2 = O.aggregate_apply(x, vals, idx)
    touched = np.zeros(n, bool)
    for i in idx:
        touched[i] = True
    assert np.array_equal(x2[~touched].view(np.uint32), x[~touched].view(np.uint32))
    for i in np.nonzero(touched)[0][:50]:
        acc = np.float32(0)
        for w in range(W):
            hit = np.nonzero(idx[w] == i)[0]
            if hit.size:
                acc = np.float32(acc + vals[w][hit[0]])
        assert x2[i] == np.float32(x[i] - np.float32(acc / np.float32(W)))
