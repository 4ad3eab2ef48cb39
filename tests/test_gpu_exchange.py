"""The exchange step of Algorithm 1 on a GPU: worker w = rank w, NCCL collectives, the aggregate enqueued on
the same stream right behind them.  This machine gives one GPU, so the process group has one rank; what is
checked is the whole chain compress -> exchange -> aggregate on device tensors (buffer layouts, stream order
without a host synchronisation in between, both ways to exchange shared coordinates) against the oracle."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import paper_2009_09271_b200 as sc
from oracle import sparsify_oracle as O
from paper_2009_09271_b200.exchange import exchange_and_aggregate, exchange_and_apply
from parity_util import assert_bits_equal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def one_rank_nccl():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    yield
    dist.destroy_process_group()


@pytest.mark.parametrize("scheme", [sc.SC_TOPK, sc.SC_RANDK, sc.SC_RANDBLOCK])
def test_compress_exchange_aggregate_one_rank(one_rank_nccl, scheme):
    n, k = 300_007, 3001
    ctx = sc.Context(max_n=n, max_W=1, max_segments=1)
    gen = torch.Generator().manual_seed(5 + scheme)
    g = torch.randn(n, generator=gen) * 1e-3
    e0 = torch.randn(n, generator=gen) * 1e-4
    ov, oi, oe, oout = O.step(scheme, [g.numpy()], [e0.numpy()], [(0, n, k)], [17])
    for shared, mode in ((False, "allgather"), (True, "allgather"), (True, "allreduce")):
        if scheme == sc.SC_TOPK and shared:
            continue                                                     # top-k coordinates are never shared
        e = e0.cuda().clone()
        vals = torch.empty(k, device="cuda")
        idx = torch.empty(k, device="cuda", dtype=torch.int32)
        out = torch.full((n,), float("nan"), device="cuda")
        ctx.sc_compress(scheme, g.cuda(), e, k, 17, vals, idx)           # no synchronisation from here ...
        exchange_and_aggregate(ctx, vals, idx, n, out, shared_coordinates=shared, mode=mode)
        assert ctx.sc_sync_status() == 0                                 # ... to here
        assert_bits_equal(e, oe[0], "residual")
        if mode == "allgather":
            assert_bits_equal(out, oout, "average (ordered sum)")
        else:                                                            # the collective owns the order of the sum
            assert np.allclose(out.cpu().numpy(), oout, rtol=1e-6, atol=1e-9)
        x0 = torch.randn(n, generator=gen)
        x = x0.cuda().clone()
        exchange_and_apply(ctx, vals, idx, n, x, shared_coordinates=shared, mode=mode)
        assert ctx.sc_sync_status() == 0
        want = O.aggregate_apply(x0.numpy(), ov, oi)
        if mode == "allgather":
            assert_bits_equal(x, want, "model update")
        else:
            assert np.allclose(x.cpu().numpy(), want, rtol=1e-6, atol=1e-9)
    ctx.close()
