"""Randomised GPU parity: seeded random segment tables, kept counts, worker counts, seeds and
value distributions, every case compared bit for bit with the oracle through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2009_09271_b200 as sc
from parity_util import run_step_both

pytestmark = pytest.mark.gpu

BIG = 1 << 20


@pytest.fixture(scope="module")
def ctx():
    c = sc.Context(max_n=5 * BIG, max_W=6, max_segments=24)
    yield c
    c.close()


def _values(rng, n, kind):
    if kind == 0:
        v = rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 2)
    elif kind == 1:
        v = rng.standard_t(2, n) * 1e-3
    elif kind == 2:                                   # few distinct values: heavy ties
        v = rng.integers(-4, 5, n).astype(np.float64) * 0.5
    elif kind == 3:                                   # mostly exact zeros
        v = rng.standard_normal(n) * (rng.random(n) < 0.03)
    else:                                             # huge dynamic range, both signs, some denormals
        v = np.ldexp(rng.standard_normal(n), rng.integers(-140, 100, n))
    return torch.from_numpy(v.astype(np.float32))


def _table(rng, big):
    nseg = int(rng.integers(1, 9))
    sizes = []
    for _ in range(nseg):
        pick = rng.random()
        if pick < 0.4:
            sizes.append(int(rng.integers(1, 300)))
        elif pick < 0.8:
            sizes.append(int(rng.integers(300, 40_000)))
        else:
            sizes.append(int(rng.integers(40_000, 300_000)))
    if big:
        sizes[int(rng.integers(0, nseg))] = int(rng.integers(BIG, 2 * BIG + 5000))
    segs, off = [], 0
    for s in sizes:
        off += int(rng.integers(0, 6)) if rng.random() < 0.3 else 0          # occasional gap
        mode = rng.random()
        k = 0 if mode < 0.05 else s if mode < 0.1 else max(1, int(s * 10.0 ** rng.uniform(-4, -0.3)))
        segs.append((off, s, min(k, s)))
        off += s
    return segs, off + int(rng.integers(0, 4))


@pytest.mark.parametrize("case", range(36))
def test_random_case(ctx, case):
    rng = np.random.default_rng(1000 + case)
    scheme = [sc.SC_TOPK, sc.SC_RANDK, sc.SC_RANDBLOCK][case % 3]
    segs, n = _table(rng, big=(case % 4 == 0))
    W = int(rng.integers(1, 6))
    kind = int(rng.integers(0, 5))
    g = torch.stack([_values(rng, n, kind) for _ in range(W)])
    e = torch.stack([_values(rng, n, int(rng.integers(0, 5))) * 0.1 for _ in range(W)])
    shared = rng.random() < 0.5
    seeds = [int(rng.integers(0, 2 ** 62))] * W if shared else [int(x) for x in rng.integers(0, 2 ** 62, W)]
    use = ["step", "split", "host"][int(rng.integers(0, 3))]
    e = run_step_both(ctx, scheme, g, e, segs, seeds, use=use)
    run_step_both(ctx, scheme, g, e, segs, [s + 1 for s in seeds], use="step")      # second step on the carried residual


@pytest.mark.parametrize("case", range(12))
def test_random_case_wrap_block_and_step_size(ctx, case):
    """The same generator of cases for the wrap-around block and for gamma != 1 (all schemes)."""
    rng = np.random.default_rng(5000 + case)
    scheme = [sc.SC_RANDBLOCK_WRAP, sc.SC_TOPK, sc.SC_RANDK, sc.SC_RANDBLOCK][case % 4] if case >= 4 else sc.SC_RANDBLOCK_WRAP
    gamma = 1.0 if case < 4 else float(np.float32(10.0 ** rng.uniform(-3, 1) * (-1 if rng.random() < 0.3 else 1)))
    segs, n = _table(rng, big=(case % 3 == 0))
    W = int(rng.integers(1, 6))
    g = torch.stack([_values(rng, n, int(rng.integers(0, 5))) for _ in range(W)])
    e = torch.stack([_values(rng, n, int(rng.integers(0, 5))) * 0.1 for _ in range(W)])
    shared = rng.random() < 0.5
    seeds = [int(rng.integers(0, 2 ** 62))] * W if shared else [int(x) for x in rng.integers(0, 2 ** 62, W)]
    use = ["step", "split", "host"][int(rng.integers(0, 3))]
    e = run_step_both(ctx, scheme, g, e, segs, seeds, use=use, gamma=gamma)
    run_step_both(ctx, scheme, g, e, segs, [s + 1 for s in seeds], use="step", gamma=gamma)
