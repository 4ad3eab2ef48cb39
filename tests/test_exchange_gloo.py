"""The exchange step on CPU tensors with the gloo backend (world size 2): which collective runs,
what every rank ends up holding, and in which order."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, errors):
    try:
        sys.path.insert(0, ROOT)
        from paper_2009_09271_b200.exchange import exchange_messages
        os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
        dist.init_process_group("gloo", rank=rank, world_size=world)
        k = 5
        vals = torch.arange(k, dtype=torch.float32) + 10.0 * rank
        idx = (torch.arange(k, dtype=torch.int32) * 3 + rank)
        v, i, rows = exchange_messages(vals, idx, shared_coordinates=False)
        assert rows == world and v.shape == (world, k) and i.shape == (world, k)
        for r in range(world):                                   # rank order = worker order
            assert torch.equal(v[r], torch.arange(k, dtype=torch.float32) + 10.0 * r)
            assert torch.equal(i[r], torch.arange(k, dtype=torch.int32) * 3 + r)
        shared_idx = torch.arange(k, dtype=torch.int32) * 7
        v, i, rows = exchange_messages(vals, shared_idx, shared_coordinates=True, mode="allgather")
        assert rows == world and v.shape == (world, k) and i.shape == (1, k)
        v, i, rows = exchange_messages(vals, shared_idx, shared_coordinates=True, mode="allreduce")
        assert rows == 1 and i.shape == (1, k)
        want = sum(torch.arange(k, dtype=torch.float32) + 10.0 * r for r in range(world)) / world
        assert torch.allclose(v[0], want, rtol=1e-6, atol=1e-9)
        # exchange_and_aggregate up to the aggregate call: a stand-in context records what it is handed, and the
        # result is formed with the oracle (this test has no GPU): every rank must end with the same average
        import numpy as np
        from oracle import sparsify_oracle as O
        from paper_2009_09271_b200.exchange import exchange_and_aggregate
        n = 40

        class Recorder:
            calls = []

            def sc_aggregate(self, W, v, i, k_, n_, out):
                self.calls.append(("private", W, tuple(v.shape), tuple(i.shape), k_, n_))
                out.copy_(torch.from_numpy(O.aggregate([r.numpy() for r in v], [r.numpy().view(np.uint32) for r in i], n_)))

            def sc_aggregate_shared(self, W, v, i, k_, n_, out):
                self.calls.append(("shared", W, tuple(v.shape), tuple(i.shape), k_, n_))
                out.copy_(torch.from_numpy(O.aggregate([r.numpy() for r in v], [i.numpy().view(np.uint32)] * W, n_)))

        rec = Recorder()
        all_vals = [torch.arange(k, dtype=torch.float32) + 10.0 * r for r in range(world)]
        all_idx = [(torch.arange(k, dtype=torch.int32) * 3 + r) for r in range(world)]
        out = torch.full((n,), float("nan"))
        exchange_and_aggregate(rec, vals, idx, n, out, shared_coordinates=False)
        want = O.aggregate([v.numpy() for v in all_vals], [i.numpy().view(np.uint32) for i in all_idx], n)
        assert np.array_equal(out.numpy().view(np.uint32), want.view(np.uint32))
        assert rec.calls[-1] == ("private", world, (world, k), (world, k), k, n)
        for mode, rows in (("allgather", world), ("allreduce", 1)):
            out = torch.full((n,), float("nan"))
            exchange_and_aggregate(rec, vals, shared_idx, n, out, shared_coordinates=True, mode=mode)
            want = O.aggregate([v.numpy() for v in all_vals], [shared_idx.numpy().view(np.uint32)] * world, n)
            assert rec.calls[-1] == ("shared", rows, (rows, k), (k,), k, n)          # after an allreduce: ONE row, already the average
            if mode == "allgather":
                assert np.array_equal(out.numpy().view(np.uint32), want.view(np.uint32))
            else:
                assert np.allclose(out.numpy(), want, rtol=1e-6, atol=1e-9)
        dist.barrier()
        dist.destroy_process_group()
    except Exception as exc:                                      # pragma: no cover
        errors.put(f"rank {rank}: {exc!r}")
        raise


def test_exchange_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    errors = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29741, errors)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
    assert errors.empty(), errors.get()
    assert all(p.exitcode == 0 for p in procs)
