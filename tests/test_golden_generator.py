"""The coordinate generators against the stored known answers (tests/golden/generator_kat.txt,
written by tests/golden/make_generator_kat.py from the oracle alone)."""
import os

import numpy as np
import pytest
import torch

from oracle import sparsify_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))


def _cases():
    out = []
    for line in open(os.path.join(HERE, "golden", "generator_kat.txt")):
        if line.startswith("#") or "|" not in line:
            continue
        head, ss, start, coords = [p.strip() for p in line.split("|")]
        seed, n, k = (int(v) for v in head.split())
        out.append((seed, n, k, int(ss), int(start), [int(v) for v in coords.split()]))
    return out


def test_oracle_matches_stored_answers():
    cases = _cases()
    assert len(cases) >= 8
    for seed, n, k, ss, start, coords in cases:
        assert O.segment_seed(seed, 0) == ss
        assert O.block_start(ss, n, k) == start
        assert O.randk_indices(ss, n, k).tolist() == coords
    for line in open(os.path.join(HERE, "golden", "generator_kat.txt")):
        if line.startswith("mix64"):
            _, a, b, _, v = line.split()
            assert O.mix64(int(a), int(b)) == int(v)
        if line.startswith("mix32"):
            _, x, _, v = line.split()
            assert O.mix32(int(x)) == int(v)


@pytest.mark.gpu
def test_cuda_library_matches_stored_answers():
    import paper_2009_09271_b200 as sc
    for seed, n, k, ss, start, coords in _cases():
        if n > 2_000_000:
            continue
        ctx = sc.Context(max_n=n, max_W=1, max_segments=1)
        g = torch.zeros(n, device="cuda"); e = torch.zeros(n, device="cuda")
        vals = torch.empty(k, device="cuda"); idx = torch.empty(k, device="cuda", dtype=torch.int32)
        ctx.sc_compress(sc.SC_RANDK, g, e, k, seed, vals, idx)
        assert ctx.sc_sync_status() == 0
        assert idx.cpu().numpy().view(np.uint32).tolist() == coords
        ctx.sc_compress(sc.SC_RANDBLOCK, g, e, k, seed, vals, idx)
        assert ctx.sc_sync_status() == 0
        assert idx.cpu().numpy().view(np.uint32).tolist() == list(range(start, start + k))
        ctx.close()
