"""Synthetic gradient generators and segment tables for the five workloads.

Every value here is an *input* to the compressor: gradient vectors, the
per-tensor segment table (offset, n_s, k_s) and seeds.  The paper trains
ResNet-18 on CIFAR-10 (Section "Experimental setup"); these generators stand in
for real gradients with the same structure: many small and a few huge
per-tensor segments, per-layer scale disparity, heavy tails, exactly-zero rows.

All generators take a torch device so that large cases can be produced on the
GPU and the very same bits copied to the host for the CPU oracle.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import torch

__all__ = [
    "Segment", "Workload", "kept_count", "segment_table", "flat_table",
    "resnet18_sizes", "resnet50_sizes", "lstm_lm_sizes",
    "gen_gaussian", "gen_segment_gaussian", "gen_segment_laplace", "gen_lstm_lm",
    "gen_student_t", "gen_small_integers", "make_generator", "step_seed",
    "WORKLOADS", "workload", "generate",
]


@dataclass(frozen=True)
class Segment:
    offset: int
    n: int
    k: int


def kept_count(n: int, num: int, den: int) -> int:
    """k = ceil(n * num / den) in integers (density num/den of one segment)."""
    return (n * num + den - 1) // den


def segment_table(sizes: Sequence[int], num: int, den: int) -> List[Segment]:
    """Layer-wise scope: one k per tensor, segments concatenated in order."""
    out, off = [], 0
    for s in sizes:
        out.append(Segment(off, s, kept_count(s, num, den)))
        off += s
    return out


def flat_table(n: int, num: int, den: int) -> List[Segment]:
    """Global scope: the whole vector is one segment."""
    return [Segment(0, n, kept_count(n, num, den))]


# --------------------------------------------------------------------------
# Parameter-tensor sizes, in registration order, derived from the layer shapes.
# --------------------------------------------------------------------------
def _bn(c: int) -> List[int]:
    return [c, c]  # scale, shift


def resnet18_sizes(num_classes: int = 1000) -> List[int]:
    sizes = [64 * 3 * 7 * 7] + _bn(64)
    inplanes = 64
    for planes, stride in ((64, 1), (128, 2), (256, 2), (512, 2)):
        for blk in range(2):
            s = stride if blk == 0 else 1
            sizes += [planes * inplanes * 9] + _bn(planes)
            sizes += [planes * planes * 9] + _bn(planes)
            if blk == 0 and (s != 1 or inplanes != planes):
                sizes += [planes * inplanes] + _bn(planes)
            inplanes = planes
    sizes += [512 * num_classes, num_classes]
    return sizes


def resnet50_sizes(num_classes: int = 1000) -> List[int]:
    sizes = [64 * 3 * 7 * 7] + _bn(64)
    inplanes = 64
    for planes, blocks, stride in ((64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)):
        for blk in range(blocks):
            s = stride if blk == 0 else 1
            sizes += [planes * inplanes] + _bn(planes)
            sizes += [planes * planes * 9] + _bn(planes)
            sizes += [4 * planes * planes] + _bn(4 * planes)
            if blk == 0 and (s != 1 or inplanes != 4 * planes):
                sizes += [4 * planes * inplanes] + _bn(4 * planes)
            inplanes = 4 * planes
    sizes += [2048 * num_classes, num_classes]
    return sizes


LSTM_VOCAB, LSTM_HIDDEN, LSTM_TOTAL = 33278, 650, 66_034_000


def lstm_lm_sizes() -> List[int]:
    """Input embedding, two LSTM layers, output embedding, output bias, and a
    dense remainder that brings the total to the stated 66,034,000 elements
    (the stated shapes alone sum to less)."""
    emb = LSTM_VOCAB * LSTM_HIDDEN
    lstm = 4 * LSTM_HIDDEN * (2 * LSTM_HIDDEN) + 2 * 4 * LSTM_HIDDEN
    sizes = [emb, lstm, lstm, emb, LSTM_VOCAB]
    sizes.append(LSTM_TOTAL - sum(sizes))
    return sizes


# --------------------------------------------------------------------------
# Seeds
# --------------------------------------------------------------------------
def make_generator(base: int, worker: int, step: int, device) -> torch.Generator:
    """One independent stream per (base seed, worker, step)."""
    g = torch.Generator(device=device)
    g.manual_seed((base * 1_000_003 + worker) * 1_000_003 + step + 12345)
    return g


def step_seed(base: int, step: int, worker: int | None = None) -> int:
    """Seed handed to the compressor at one step.  With worker=None all workers
    share the coordinates; otherwise each worker draws its own."""
    s = (base * 0x9E3779B1 + step * 0x85EBCA77 + 0x1234567) & 0xFFFFFFFFFFFFFFFF
    if worker is not None:
        s = (s * 0xC2B2AE3D + worker + 1) & 0xFFFFFFFFFFFFFFFF
    return s


# --------------------------------------------------------------------------
# Value generators (fp32 tensors of length n on `device`)
# --------------------------------------------------------------------------
def gen_gaussian(n: int, gen: torch.Generator, device, std: float = 1e-3) -> torch.Tensor:
    return torch.randn(n, generator=gen, device=device, dtype=torch.float32) * std


def _segment_scales(nseg: int, base: int, kind: str) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(base * 7919 + 17)
    if kind == "lognormal":  # sigma_s = exp(z), z ~ N(0, 1)
        return torch.exp(torch.randn(nseg, generator=g, dtype=torch.float64))
    if kind == "loguniform":  # b_s = 10 ** U[-5, -2]
        return 10.0 ** (torch.rand(nseg, generator=g, dtype=torch.float64) * 3.0 - 5.0)
    raise ValueError(kind)


def gen_segment_gaussian(sizes: Sequence[int], base: int, gen, device) -> torch.Tensor:
    scales = _segment_scales(len(sizes), base, "lognormal")
    out = torch.randn(sum(sizes), generator=gen, device=device, dtype=torch.float32)
    off = 0
    for s, sc in zip(sizes, scales.tolist()):
        out[off:off + s] *= sc
        off += s
    return out


def gen_segment_laplace(sizes: Sequence[int], base: int, gen, device) -> torch.Tensor:
    scales = _segment_scales(len(sizes), base, "loguniform")
    n = sum(sizes)
    u = torch.rand(n, generator=gen, device=device, dtype=torch.float32) - 0.5
    out = -torch.sign(u) * torch.log1p(-2.0 * u.abs())
    off = 0
    for s, sc in zip(sizes, scales.tolist()):
        out[off:off + s] *= sc
        off += s
    return out


def gen_lstm_lm(gen, device, sizes: Sequence[int] | None = None, width: int = LSTM_HIDDEN,
                zero_prob: float = 0.95, std: float = 1e-3) -> torch.Tensor:
    """Embedding segments (index 0 and 3) have whole rows of `width` elements
    exactly zero with probability zero_prob; everything else is N(0, std)."""
    sizes = list(sizes) if sizes is not None else lstm_lm_sizes()
    out = torch.randn(sum(sizes), generator=gen, device=device, dtype=torch.float32) * std
    off = 0
    for i, s in enumerate(sizes):
        if i in (0, 3):
            rows = s // width
            keep = torch.rand(rows, generator=gen, device=device) >= zero_prob
            out[off:off + rows * width].view(rows, width).mul_(keep.unsqueeze(1).to(out.dtype))
        off += s
    # multiplying by 0.0 may give -0.0; make the zero rows +0.0 exactly
    out += 0.0
    return out


def gen_student_t(n: int, gen, device, nu: int = 3, scale: float = 1e-3,
                  chunk: int = 1 << 26) -> torch.Tensor:
    """scale * t_nu, built as z / sqrt(chi2_nu / nu) from nu + 1 normals, in
    chunks so that the temporaries stay small."""
    out = torch.empty(n, device=device, dtype=torch.float32)
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        z = torch.randn(b - a, generator=gen, device=device, dtype=torch.float32)
        c = torch.zeros(b - a, device=device, dtype=torch.float32)
        for _ in range(nu):
            c += torch.randn(b - a, generator=gen, device=device, dtype=torch.float32) ** 2
        out[a:b] = z * torch.rsqrt(c / nu) * scale
    return out


def gen_small_integers(n: int, gen, device, bound: int = 1024) -> torch.Tensor:
    """Integer-valued fp32 gradients in [-bound, bound]: sums of a few thousand
    of them are exact in fp32, which makes multi-step identities bit-exact."""
    return torch.randint(-bound, bound + 1, (n,), generator=gen, device=device).to(torch.float32)


# --------------------------------------------------------------------------
# The five workloads
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    W: int
    sizes: Tuple[int, ...]          # per-tensor sizes (one entry = flat vector)
    schemes: Tuple[str, ...]
    densities: Tuple[Tuple[int, int], ...]   # (num, den)
    steps: int
    base_seed: int
    values: str                      # which generator


WORKLOADS = {
    "c1": Workload("c1", 1_048_576, 4, (1_048_576,), ("topk",), ((1, 100),), 3, 0, "gaussian"),
    "c2": Workload("c2", 11_689_512, 8, tuple(resnet18_sizes()), ("randblock",), ((1, 100),), 10, 1,
                   "segment_gaussian"),
    "c3": Workload("c3", 25_557_032, 16, tuple(resnet50_sizes()), ("topk", "randk", "randblock"),
                   ((1, 1000),), 10, 2, "segment_laplace"),
    "c4": Workload("c4", LSTM_TOTAL, 8, tuple(lstm_lm_sizes()), ("topk", "randblock"),
                   ((1, 1000), (1, 100), (1, 10)), 10, 3, "lstm_lm"),
    "c5": Workload("c5", 350_000_000, 16, (350_000_000,), ("topk", "randk", "randblock"),
                   ((1, 10000), (1, 1000), (1, 100), (1, 10)), 20, 4, "student_t"),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


def generate(wl: Workload, worker: int, step: int, device, sizes: Sequence[int] | None = None) -> torch.Tensor:
    """Gradient of one (worker, step).  `sizes` overrides the tensor sizes (a
    reduced copy of the same structure for quick tests)."""
    sizes = list(sizes) if sizes is not None else list(wl.sizes)
    gen = make_generator(wl.base_seed, worker, step, device)
    n = sum(sizes)
    if wl.values == "gaussian":
        return gen_gaussian(n, gen, device)
    if wl.values == "segment_gaussian":
        return gen_segment_gaussian(sizes, wl.base_seed, gen, device)
    if wl.values == "segment_laplace":
        return gen_segment_laplace(sizes, wl.base_seed, gen, device)
    if wl.values == "lstm_lm":
        return gen_lstm_lm(gen, device, sizes)
    if wl.values == "student_t":
        return gen_student_t(n, gen, device)
    raise ValueError(wl.values)
