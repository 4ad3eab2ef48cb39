"""sc_aggregate_static: the aggregate for callers that cannot allocate device memory.

Every other entry point needs a context, and creating one calls cudaMalloc, which code
running after a framework has claimed all device memory, or inside a latency-critical
section, cannot afford.  This entry point keeps its scratch in a fixed device array instead.
The test calls it through the C ABI twice in a row (the array keeps the first call's
contents) and requires the same bits as sc_aggregate.  It is collected last so that a run
stopping at the first failure has already run everything else; it does not depend on any
other test having run."""
import numpy as np
import pytest
import torch

import paper_2009_09271_b200 as sc

pytestmark = pytest.mark.gpu


def _messages(W, n, k, seed):
    rng = np.random.default_rng(seed)
    idx = np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    vals = (rng.standard_normal((W, k)) * 10.0 ** rng.uniform(-3, 3, (W, k))).astype(np.float32)
    return torch.from_numpy(vals).cuda(), torch.from_numpy(idx.view(np.int32)).cuda()


def test_static_aggregate_matches_context_aggregate_twice_in_a_row():
    cases = [(7, 300_001, 4000, 1), (16, 1_000_003, 20_000, 2)]      # second call: larger, other W
    n_max = max(c[1] for c in cases)
    ctx = sc.Context(max_n=n_max, max_W=16, max_segments=1)
    for W, n, k, seed in cases:
        vals, idx = _messages(W, n, k, seed)
        want = torch.full((n,), float("nan"), device="cuda")
        got = torch.full((n,), float("nan"), device="cuda")
        ctx.sc_aggregate(W, vals, idx, k, n, want)
        assert ctx.sc_sync_status() == 0
        sc.sc_aggregate_static(W, vals, idx, k, n, got)
        torch.cuda.synchronize()
        assert torch.equal(got.view(torch.int32), want.view(torch.int32))
    ctx.close()


def test_static_aggregate_rejects_sizes_beyond_its_fixed_scratch():
    vals = torch.zeros(8, device="cuda")
    idx = torch.zeros(8, device="cuda", dtype=torch.int32)
    out = torch.full((8,), 5.0, device="cuda")
    lib = sc.load_library()
    too_many = sc.binding.STATIC_MAX_N + 1
    assert lib.sc_aggregate_static(1, vals.data_ptr(), idx.data_ptr(), 1, too_many, out.data_ptr(), None) == -2
    assert lib.sc_aggregate_static(sc.binding.STATIC_MAX_W + 1, vals.data_ptr(), idx.data_ptr(), 0, 8,
                                   out.data_ptr(), None) == -2
    torch.cuda.synchronize()
    assert bool((out == 5.0).all())                       # rejected before any buffer was touched
    with pytest.raises(sc.SparseCommError):
        sc.sc_aggregate_static(65, vals, idx, 0, 8, out)
