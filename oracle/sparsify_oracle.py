"""CPU oracle for the sparsified-SGD compressor and aggregator.  TEST INFRASTRUCTURE.

This file is a plain, slow, single-threaded numpy statement of what one step
of "Sparsified SGD with error-feedback" (Algorithm 1 of the paper) computes on
the path  p = g + e,  q^w = C(p),  e' = p - q^w,  q = (sum_w q^w) / W.
It exists so that the CUDA library can be checked against it.  Nothing in the
product imports it; only the tests, the smoke check and the benchmark's
CPU-baseline leg do.  It shares no code, constants or tables with the CUDA
path: both are written from the same prose specification (below).

Arithmetic: fp32, IEEE-754 round-to-nearest-even, denormals kept.  The paper's
implementation is fp32 PyTorch ("Experimental setup") and the GPU library must
agree bit for bit, so the oracle does NOT widen to fp64.

Readings of the paper where it is silent or garbled (all restated in the
project's design notes):
 * Algorithm 1, residual line: printed with the aggregate q_t; read as the
   worker's own message, e' = p - q^w, as the Methodology prose says: what a
   worker keeps is its own accumulated gradient minus what it sent, and the
   residual collects the entries that were left out of the message.
 * Algorithm 1, accumulate line: gamma*g + e.  The caller passes gamma*g as the
   gradient; one fp32 add happens here.
 * Aggregate: Algorithm 1 prints a sum, the abstract and introduction say the
   workers use the average.  The oracle sums in worker order 0..W-1 starting
   from +0.0 and then divides by float(W).
 * Top-k (Methodology item; the paper does not say how values are ranked):
   largest magnitude, compared on the
   bit pattern of |p| (so NaN > inf > finite, +0 == -0); ties go to the lowest
   index.
 * Message order: ascending coordinate, for every scheme.
 * Random-k: k DISTINCT coordinates, {pi(j) : j < k} for a keyed bijection pi
   of [0, n) (a Feistel network with cycle walking, specified below).
 * Block-random-k: the block does not wrap; its start is uniform on [0, n-k].
   Variant RANDBLOCK_WRAP: the start is uniform on [0, n) and the block wraps
   around the end of the segment, so every coordinate is kept with the same
   probability k/n (without the wrap the first and last k-1 coordinates are
   kept less often).
 * Step size: with gamma != 1 the accumulate line is evaluated as ONE fused
   multiply-add, p = round(gamma * g + e) (a single fp32 rounding); gamma = 1
   gives the plain add bit for bit.
 * Workers that share their seed state (Methodology, on reduce against gather):
   the seed is an argument; equal seeds give equal
   coordinates on every worker.
 * Scope (layer-wise or global): a segment table; segment s of a call uses the
   seed mix64(seed, s); global scope is a single segment (s = 0).

Parity pins (tests/test_oracle_*.py): brute-force ordering by Python tuples on
tiny inputs, set equality with torch.topk on distinct magnitudes, k = 0 / k = n
limits, e' + q == p, exact telescoping sums on integer-valued gradients, the
dense limit against a three-line loop, enumeration of pi for every small n,
chi-square tests of inclusion frequencies and block starts; the fused
multiply-add against exact rational arithmetic (fractions.Fraction) on random
and constructed halfway cases.
Parity unpinned: agreement of the random generator with the authors' own code
(the paper names no generator; the one below is this project's specification).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

TOPK, RANDK, RANDBLOCK, RANDBLOCK_WRAP = 0, 1, 2, 3
SCHEMES = {"topk": TOPK, "randk": RANDK, "randblock": RANDBLOCK, "randblock_wrap": RANDBLOCK_WRAP}

_M64 = (1 << 64) - 1
_M32 = (1 << 32) - 1


# ---------------------------------------------------------------------------
# Seed arithmetic (integer only).  This is the project's own specification of
# the random choice that the Methodology items Random-k and Block-random-k ask for.
# ---------------------------------------------------------------------------
def mix64(a: int, b: int) -> int:
    """64-bit finaliser of the SplitMix generator applied to a + (b+1)*phi."""
    z = (a + (b + 1) * 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def mix32(x):
    """xorshift-multiply hash on 32-bit words (python int or uint32 array)."""
    if isinstance(x, np.ndarray):
        x = x.astype(np.uint32, copy=True)
        x ^= x >> np.uint32(16)
        x *= np.uint32(0x6A09E667)
        x ^= x >> np.uint32(15)
        x *= np.uint32(0xBB67AE85)
        x ^= x >> np.uint32(16)
        return x
    x &= _M32
    x ^= x >> 16
    x = (x * 0x6A09E667) & _M32
    x ^= x >> 15
    x = (x * 0xBB67AE85) & _M32
    x ^= x >> 16
    return x


SALT_BLOCK = 0x626C6F636B          # "block"
SALT_RANDK = 0x72616E646B00        # "randk\0" + round number
FEISTEL_ROUNDS = 6


def segment_seed(seed: int, s: int) -> int:
    return mix64(seed & _M64, s)


def block_start(seed_s: int, n: int, k: int) -> int:
    """Start a of the kept block [a, a+k): floor(h * (n-k+1) / 2^64) for a
    64-bit hash h of the segment seed, so 0 <= a <= n-k (no wrap-around)."""
    h = mix64(seed_s, SALT_BLOCK)
    return (h * (n - k + 1)) >> 64


def block_start_wrap(seed_s: int, n: int) -> int:
    """Start a of the wrapping block {(a + j) mod n : j < k}: floor(h * n / 2^64)
    for the same 64-bit hash h, so 0 <= a < n (a = 0 for an empty segment)."""
    h = mix64(seed_s, SALT_BLOCK)
    return (h * n) >> 64


def feistel_params(seed_s: int, n: int) -> Tuple[int, int, List[int]]:
    """Bit widths (left, right) and the round keys of the permutation of
    [0, 2^b), b = max(2, ceil(log2 n))."""
    b = max(2, (n - 1).bit_length())
    left = b // 2
    right = b - left
    keys = [mix64(seed_s, SALT_RANDK + r) >> 32 for r in range(FEISTEL_ROUNDS)]
    return left, right, keys


def feistel_once(x: np.ndarray, left: int, right: int, keys: Sequence[int]) -> np.ndarray:
    """One application of the alternating Feistel network to uint32 values in
    [0, 2^(left+right)).  x = (L << right) | R.  Even rounds replace L by
    L xor mix32(R xor K_r) (masked to `left` bits); odd rounds replace R by
    R xor mix32(L xor K_r) (masked to `right` bits)."""
    mask_l = np.uint32((1 << left) - 1)
    mask_r = np.uint32((1 << right) - 1)
    L = (x >> np.uint32(right)) & mask_l
    R = x & mask_r
    for r, key in enumerate(keys):
        kk = np.uint32(key)
        if r % 2 == 0:
            L = L ^ (mix32(R ^ kk) & mask_l)
        else:
            R = R ^ (mix32(L ^ kk) & mask_r)
    return (L << np.uint32(right)) | R


def randk_permute(seed_s: int, n: int, j: np.ndarray) -> np.ndarray:
    """pi(j) for each j in the array (all j < n): apply the Feistel network
    until the value falls below n (cycle walking)."""
    left, right, keys = feistel_params(seed_s, n)
    x = feistel_once(j.astype(np.uint32), left, right, keys)
    todo = np.nonzero(x >= n)[0]
    while todo.size:
        x[todo] = feistel_once(x[todo], left, right, keys)
        todo = todo[x[todo] >= n]
    return x


def randk_indices(seed_s: int, n: int, k: int) -> np.ndarray:
    """The k distinct coordinates of random-k, ascending."""
    return np.sort(randk_permute(seed_s, n, np.arange(k, dtype=np.uint32)))


# ---------------------------------------------------------------------------
# Selection
# ---------------------------------------------------------------------------
def topk_indices(p: np.ndarray, k: int) -> np.ndarray:
    """Coordinates of the k first elements in the strict order
    "larger |p| bit pattern first, equal patterns: lower index first", ascending."""
    n = p.size
    if k == 0:
        return np.zeros(0, dtype=np.uint32)
    key = p.view(np.uint32) & np.uint32(0x7FFFFFFF)
    # one distinct 64-bit rank per element: larger rank = earlier in the order
    rank = (key.astype(np.uint64) << np.uint64(32)) | (np.uint64(_M32) - np.arange(n, dtype=np.uint64))
    if k < n:
        rank = np.partition(rank, n - k)[n - k:]          # the k largest ranks
    idx = (np.uint64(_M32) - (rank & np.uint64(_M32))).astype(np.uint32)
    return np.sort(idx)


def select(scheme: int, p: np.ndarray, k: int, seed_s: int) -> np.ndarray:
    n = p.size
    if not 0 <= k <= n:
        raise ValueError("k out of range")
    if scheme == TOPK:
        return topk_indices(p, k)
    if scheme == RANDK:
        return randk_indices(seed_s, n, k)
    if scheme == RANDBLOCK:
        a = block_start(seed_s, n, k)
        return np.arange(a, a + k, dtype=np.uint32)
    if scheme == RANDBLOCK_WRAP:
        if n == 0:
            return np.zeros(0, np.uint32)
        a = block_start_wrap(seed_s, n)
        return np.sort((a + np.arange(k, dtype=np.int64)) % n).astype(np.uint32)
    raise ValueError("unknown scheme")


# ---------------------------------------------------------------------------
# Algorithm 1, per worker: accumulate, compress, residual
# ---------------------------------------------------------------------------
def fma32(a: np.ndarray, b, c: np.ndarray) -> np.ndarray:
    """round_fp32(a * b + c) with a single rounding, elementwise on fp32 inputs.

    The product of two fp32 numbers is exact in fp64.  The fp64 sum s = prod + c
    is rounded once; its exact error follows from the classical two-sum identity.
    Replacing s by its round-to-odd neighbour when it is inexact (truncate towards
    zero, then set the last mantissa bit) makes the final fp64 -> fp32 rounding
    come out as if the exact sum had been rounded directly (fp64 carries more
    than 2 x 24 + 2 bits)."""
    a64 = np.asarray(a, np.float32).astype(np.float64)
    b64 = np.asarray(b, np.float32).astype(np.float64)
    c64 = np.asarray(c, np.float32).astype(np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        prod = a64 * b64
        s = prod + c64
        bb = s - prod
        err = (prod - (s - bb)) + (c64 - bb)
    inexact = np.isfinite(s) & np.isfinite(err) & (err != 0.0)
    bits = np.ascontiguousarray(s).view(np.int64).copy()
    sign = bits & np.int64(-0x8000000000000000)
    mag = bits & np.int64(0x7FFFFFFFFFFFFFFF)
    shrink = inexact & ((err > 0.0) != (s > 0.0))                   # |exact| < |s|: step towards zero
    mag = mag - shrink.astype(np.int64)
    mag = mag | inexact.astype(np.int64)
    s_odd = (sign | mag).view(np.float64)
    with np.errstate(over="ignore"):
        return s_odd.astype(np.float32)


def accumulate(grad: np.ndarray, residual: np.ndarray, gamma: float = 1.0) -> np.ndarray:
    """Algorithm 1, accumulate line: p = gamma * g + e.  gamma == 1: one fp32 add."""
    if np.float32(gamma) == np.float32(1.0):
        return grad + residual
    return fma32(np.float32(gamma), grad, residual)


def compress(scheme: int, grad: np.ndarray, residual: np.ndarray, k: int, seed: int,
             gamma: float = 1.0) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One worker, global scope.  Returns (vals[k], idx[k] ascending, new residual)."""
    vals, idx, e_new = compress_segments(scheme, grad, residual, [(0, grad.size, k)], seed, gamma)
    return vals, idx, e_new


def compress_segments(scheme: int, grad: np.ndarray, residual: np.ndarray,
                      segments: Sequence[Tuple[int, int, int]], seed: int,
                      gamma: float = 1.0) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One worker, a table of (offset, n_s, k_s).  Message slots of segment s
    follow those of segment s-1; coordinates are global (offset added)."""
    assert grad.dtype == np.float32 and residual.dtype == np.float32
    e_new = residual.copy()
    vals_all, idx_all = [], []
    for s, (off, n_s, k_s) in enumerate(segments):
        p = accumulate(grad[off:off + n_s], residual[off:off + n_s], gamma)   # p = gamma*g + e (one rounding)
        sel = select(scheme, p, k_s, segment_seed(seed, s))            # coordinates kept by C(p)
        vals_all.append(p[sel].copy())                                 # q^w on its support
        idx_all.append(sel.astype(np.uint32) + np.uint32(off))
        p_rest = p.copy()
        p_rest[sel] = np.float32(0.0)                                  # e' = p - q^w  (kept entries become +0)
        e_new[off:off + n_s] = p_rest
    vals = np.concatenate(vals_all) if vals_all else np.zeros(0, np.float32)
    idx = np.concatenate(idx_all) if idx_all else np.zeros(0, np.uint32)
    return vals, idx, e_new


# ---------------------------------------------------------------------------
# Algorithm 1, after the exchange: q = sum_w q^w, averaged
# ---------------------------------------------------------------------------
def aggregate(vals: Sequence[np.ndarray], idx: Sequence[np.ndarray], n: int) -> np.ndarray:
    """Dense fp32[n]: for every coordinate the sum over workers 0..W-1, in that
    order, starting from +0.0, then divided by float(W)."""
    W = len(vals)
    out = np.zeros(n, dtype=np.float32)
    for w in range(W):
        # coordinates are distinct within one message, so this is one add per touched entry
        out[idx[w]] = out[idx[w]] + vals[w]
    return out / np.float32(W)


def aggregate_apply(x: np.ndarray, vals: Sequence[np.ndarray], idx: Sequence[np.ndarray]) -> np.ndarray:
    """Algorithm 1, model-update line with the aggregate read as the average:
    x_{t+1} = x_t - q_t, q_t = aggregate(...).  Returns the new x (fp32)."""
    assert x.dtype == np.float32
    return x - aggregate(vals, idx, x.size)


def step(scheme: int, grads: Sequence[np.ndarray], residuals: Sequence[np.ndarray],
         segments: Sequence[Tuple[int, int, int]], seeds: Sequence[int], gamma: float = 1.0):
    """All W workers compress, then one aggregate.  Returns
    (vals list, idx list, new residual list, dense average)."""
    vals, idx, res = [], [], []
    for g, e, sd in zip(grads, residuals, seeds):
        v, i, r = compress_segments(scheme, g, e, segments, sd, gamma)
        vals.append(v), idx.append(i), res.append(r)
    return vals, idx, res, aggregate(vals, idx, grads[0].size)
