"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU oracle
on the same bits and compare element by element (bit patterns, not values)."""
from __future__ import annotations

import numpy as np
import torch

import paper_2009_09271_b200 as sc
from oracle import sparsify_oracle as O


def bits(a) -> np.ndarray:
    """Bit patterns.  NaN payloads are canonicalised: IEEE-754 leaves the payload of
    NaN + x to the hardware (x86 keeps the input's, NVIDIA returns 0x7FFFFFFF), so a
    NaN is compared by position only."""
    a = a.detach().cpu().numpy() if isinstance(a, torch.Tensor) else np.asarray(a)
    if a.dtype == np.float32:
        b = a.view(np.uint32).copy()
        b[np.isnan(a)] = 0x7FC00000
        return b
    return a.astype(np.uint32)


def assert_bits_equal(got, want, what: str):
    g, w = bits(got), bits(want)
    assert g.shape == w.shape, f"{what}: shape {g.shape} vs {w.shape}"
    if not np.array_equal(g, w):
        bad = np.nonzero(g != w)[0]
        raise AssertionError(f"{what}: {bad.size} of {g.size} differ, first at {bad[:5]}: "
                             f"got {g[bad[:5]]} want {w[bad[:5]]}")


def segs_tuple(segs):
    return [(s.offset, s.n, s.k) if hasattr(s, "offset") else tuple(s) for s in segs]


def run_step_both(ctx, scheme, grads_cpu, res_cpu, segs, seeds, check_status=True, use="step", gamma=1.0):
    """grads_cpu/res_cpu: [W, n] fp32 CPU tensors.  Runs one step on both sides,
    asserts bit equality of messages, residuals and the dense average, and
    returns the new residuals (CPU tensor) so that steps can be chained."""
    W, n = grads_cpu.shape
    segs = segs_tuple(segs)
    K = sum(s[2] for s in segs)
    dev = "cuda"
    g = grads_cpu.to(dev)
    e = res_cpu.to(dev).clone()
    vals = torch.full((W, max(K, 1)), float("nan"), device=dev)
    idx = torch.full((W, max(K, 1)), -1, device=dev, dtype=torch.int32)
    out = torch.full((n,), float("nan"), device=dev)
    ctx.sc_set_gamma(gamma)
    if use == "step":
        ctx.sc_step(scheme, g, e, segs, seeds, vals, idx, out)
    elif use == "split":
        ctx.sc_compress_batch(scheme, g, e, segs, seeds, vals, idx)
        ctx.sc_aggregate(W, vals[:, :K].contiguous(), idx[:, :K].contiguous(), K, n, out)
    elif use == "host":
        h_out = torch.empty(n, dtype=torch.float32).pin_memory()
        ctx.sc_step_host(scheme, grads_cpu.contiguous().pin_memory(), e, segs, seeds, h_out)
        out = h_out
    ctx.sc_set_gamma(1.0)
    if check_status:
        assert ctx.sc_sync_status() == 0
    torch.cuda.synchronize()
    gn = [grads_cpu[w].numpy() for w in range(W)]
    en = [res_cpu[w].numpy() for w in range(W)]
    ov, oi, oe, oout = O.step(scheme, gn, en, segs, list(seeds), gamma)
    for w in range(W):
        if use != "host":
            assert_bits_equal(idx[w, :K], oi[w], f"idx[w={w}]")
            assert_bits_equal(vals[w, :K], ov[w], f"vals[w={w}]")
        assert_bits_equal(e[w], oe[w], f"residual[w={w}]")
    assert_bits_equal(out, oout, "aggregate")
    return e.cpu()
