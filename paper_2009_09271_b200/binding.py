"""ctypes binding of libsparsecomm.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the
library's CUDA kernels.  There is no CPU fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

SC_TOPK, SC_RANDK, SC_RANDBLOCK, SC_RANDBLOCK_WRAP = 0, 1, 2, 3
SCHEMES = {"topk": SC_TOPK, "randk": SC_RANDK, "randblock": SC_RANDBLOCK, "randblock_wrap": SC_RANDBLOCK_WRAP}

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparsecomm.so")

EXPORTS = ["sc_create", "sc_destroy", "sc_strerror", "sc_sync_status", "sc_set_gamma", "sc_scratch_bytes", "sc_launch_count",
           "sc_topk_path_counts", "sc_topk_path_detail", "sc_debug_set_poll_limits", "sc_debug_wait_probe", "sc_profile", "sc_profile_kinds", "sc_profile_name", "sc_profile_read",
           "sc_compress", "sc_compress_batch", "sc_aggregate", "sc_aggregate_shared", "sc_aggregate_static", "sc_aggregate_apply",
           "sc_aggregate_apply_shared", "sc_step", "sc_step_apply", "sc_step_host"]


class ScSegment(ctypes.Structure):
    _fields_ = [("offset", ctypes.c_uint64), ("n", ctypes.c_uint64), ("k", ctypes.c_uint64)]


class SparseCommError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2009_09271_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, u64, sz, ci = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_size_t, ctypes.c_int
    lib.sc_create.argtypes = [ctypes.POINTER(vp), sz, ci, ci]
    lib.sc_create.restype = ci
    lib.sc_destroy.argtypes = [vp]
    lib.sc_destroy.restype = None
    lib.sc_strerror.argtypes = [ci]
    lib.sc_strerror.restype = ctypes.c_char_p
    lib.sc_set_gamma.argtypes = [vp, ctypes.c_float]
    lib.sc_set_gamma.restype = ci
    lib.sc_sync_status.argtypes = [vp, vp]
    lib.sc_sync_status.restype = ci
    lib.sc_scratch_bytes.argtypes = [vp]
    lib.sc_scratch_bytes.restype = sz
    lib.sc_launch_count.argtypes = [vp]
    lib.sc_launch_count.restype = u64
    lib.sc_topk_path_counts.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.sc_topk_path_counts.restype = ci
    lib.sc_topk_path_detail.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.sc_topk_path_detail.restype = ci
    lib.sc_debug_set_poll_limits.argtypes = [vp, ctypes.c_uint32, ctypes.c_uint32]
    lib.sc_debug_set_poll_limits.restype = ci
    lib.sc_debug_wait_probe.argtypes = [vp, ci, vp]
    lib.sc_debug_wait_probe.restype = ci
    lib.sc_profile.argtypes = [vp, ci]
    lib.sc_profile.restype = ci
    lib.sc_profile_kinds.argtypes = []
    lib.sc_profile_kinds.restype = ci
    lib.sc_profile_name.argtypes = [ci]
    lib.sc_profile_name.restype = ctypes.c_char_p
    lib.sc_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(u64)]
    lib.sc_profile_read.restype = ci
    lib.sc_compress.argtypes = [vp, ci, vp, vp, sz, sz, u64, vp, vp, vp]
    lib.sc_compress.restype = ci
    lib.sc_compress_batch.argtypes = [vp, ci, ci, vp, vp, sz, ctypes.POINTER(ScSegment), ci,
                                      ctypes.POINTER(u64), vp, vp, vp]
    lib.sc_compress_batch.restype = ci
    lib.sc_aggregate.argtypes = [vp, ci, vp, vp, sz, sz, vp, vp]
    lib.sc_aggregate.restype = ci
    lib.sc_aggregate_shared.argtypes = [vp, ci, vp, vp, sz, sz, vp, vp]
    lib.sc_aggregate_shared.restype = ci
    for name in ("sc_aggregate_apply", "sc_aggregate_apply_shared"):
        getattr(lib, name).argtypes = [vp, ci, vp, vp, sz, sz, vp, vp]
        getattr(lib, name).restype = ci
    lib.sc_aggregate_static.argtypes = [ci, vp, vp, sz, sz, vp, vp]
    lib.sc_aggregate_static.restype = ci
    lib.sc_step.argtypes = [vp, ci, ci, vp, vp, sz, ctypes.POINTER(ScSegment), ci, ctypes.POINTER(u64),
                            vp, vp, vp, vp]
    lib.sc_step.restype = ci
    lib.sc_step_apply.argtypes = lib.sc_step.argtypes
    lib.sc_step_apply.restype = ci
    lib.sc_step_host.argtypes = [vp, ci, ci, vp, vp, sz, ctypes.POINTER(ScSegment), ci, ctypes.POINTER(u64),
                                 vp, vp]
    lib.sc_step_host.restype = ci
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().sc_strerror(code).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def _segments(segs: Sequence) -> "ctypes.Array[ScSegment]":
    arr = (ScSegment * max(len(segs), 1))()
    for i, s in enumerate(segs):
        off, n, k = (s.offset, s.n, s.k) if hasattr(s, "offset") else s
        arr[i] = ScSegment(int(off), int(n), int(k))
    return arr


def _seeds(seeds: Sequence[int]):
    return (ctypes.c_uint64 * max(len(seeds), 1))(*[int(s) & 0xFFFFFFFFFFFFFFFF for s in seeds])


def _check(code: int, what: str) -> None:
    if code != 0:
        raise SparseCommError(code, what)


def _want(t: torch.Tensor, dtype, name: str, cuda: bool = True) -> None:
    if t.dtype != dtype or not t.is_contiguous() or (cuda and not t.is_cuda):
        raise TypeError(f"{name}: expected a contiguous {'CUDA ' if cuda else ''}{dtype} tensor")


STATIC_MAX_N, STATIC_MAX_W = 1 << 24, 64


def sc_aggregate_static(W: int, vals, idx, k: int, n: int, out, stream=None) -> None:
    """sc_aggregate without a Context, for callers that may not allocate device memory (the
    library's own scratch for it is a fixed device array).  Limits: W <= 64, n <= 2**24.
    All calls on one GPU share that scratch, so calls that may overlap on the GPU race."""
    lib = load_library()
    _want(vals, torch.float32, "vals"), _want(idx, torch.int32, "idx"), _want(out, torch.float32, "out")
    if vals.numel() < W * k or idx.numel() < W * k or out.numel() < n:
        raise ValueError("buffer sizes do not match W, k and n")
    code = lib.sc_aggregate_static(W, _ptr(vals), _ptr(idx), k, n, _ptr(out), _stream(stream))
    if code != 0:
        raise SparseCommError(code, f"sc_aggregate_static (limits: W <= {STATIC_MAX_W}, n <= {STATIC_MAX_N})")


class Context:
    """Owns an sc_ctx (scratch memory on the current CUDA device)."""

    def __init__(self, max_n: int, max_W: int = 1, max_segments: int = 1):
        lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("sparsecomm needs a CUDA device (there is no CPU fallback)")
        torch.cuda.init()
        torch.zeros(1, device="cuda")          # make sure the primary context exists
        self._lib = lib
        self._h = ctypes.c_void_p()
        _check(lib.sc_create(ctypes.byref(self._h), max_n, max_W, max_segments), "sc_create")

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.sc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def scratch_bytes(self) -> int:
        return self._lib.sc_scratch_bytes(self._h)

    @property
    def launch_count(self) -> int:
        return self._lib.sc_launch_count(self._h)

    def sc_topk_path_counts(self, stream=None) -> tuple:
        """(small-segment radix select, one-pass path, radix select after a missed bracket)."""
        out = (ctypes.c_uint32 * 3)()
        _check(self._lib.sc_topk_path_counts(self._h, _stream(stream), out), "sc_topk_path_counts")
        return tuple(out)

    PATH_DETAIL = ("short", "one_pass", "radix_after_failure", "tie_key_seen", "ties_admitted",
                   "failed_list_overflow", "failed_bracket", "failed_short_list")

    def sc_topk_path_detail(self, stream=None) -> dict:
        out = (ctypes.c_uint32 * 8)()
        _check(self._lib.sc_topk_path_detail(self._h, _stream(stream), out), "sc_topk_path_detail")
        return dict(zip(self.PATH_DETAIL, out))

    def sc_debug_set_poll_limits(self, lookback_polls: int = 0, barrier_polls: int = 0) -> None:
        _check(self._lib.sc_debug_set_poll_limits(self._h, lookback_polls, barrier_polls), "sc_debug_set_poll_limits")

    def sc_debug_wait_probe(self, which: int, stream=None) -> None:
        _check(self._lib.sc_debug_wait_probe(self._h, which, _stream(stream)), "sc_debug_wait_probe")

    def sc_profile(self, enable: bool) -> None:
        _check(self._lib.sc_profile(self._h, 1 if enable else 0), "sc_profile")

    def sc_profile_read(self) -> dict:
        """{kernel kind: (milliseconds, launches)} since sc_profile(True)."""
        kinds = self._lib.sc_profile_kinds()
        ms = (ctypes.c_double * kinds)()
        cnt = (ctypes.c_uint64 * kinds)()
        _check(self._lib.sc_profile_read(self._h, ms, cnt), "sc_profile_read")
        return {self._lib.sc_profile_name(i).decode(): (ms[i], cnt[i]) for i in range(kinds)}

    # -- the C ABI, one method per entry point ---------------------------------
    def sc_set_gamma(self, gamma: float) -> None:
        _check(self._lib.sc_set_gamma(self._h, float(gamma)), "sc_set_gamma")

    def sc_sync_status(self, stream=None) -> int:
        return self._lib.sc_sync_status(self._h, _stream(stream))

    def sc_compress(self, scheme: int, grad, residual, k: int, seed: int, out_vals, out_idx, stream=None) -> None:
        _want(grad, torch.float32, "grad"), _want(residual, torch.float32, "residual")
        _want(out_vals, torch.float32, "out_vals"), _want(out_idx, torch.int32, "out_idx")
        if residual.numel() != grad.numel() or out_vals.numel() < k or out_idx.numel() < k:
            raise ValueError("buffer sizes do not match n and k")
        _check(self._lib.sc_compress(self._h, scheme, _ptr(grad), _ptr(residual), grad.numel(), k,
                                     int(seed) & 0xFFFFFFFFFFFFFFFF, _ptr(out_vals), _ptr(out_idx),
                                     _stream(stream)), "sc_compress")

    def sc_compress_batch(self, scheme: int, grads, residuals, segs, seeds, out_vals, out_idx, stream=None) -> None:
        W, n = grads.shape
        _want(grads, torch.float32, "grads"), _want(residuals, torch.float32, "residuals")
        _want(out_vals, torch.float32, "out_vals"), _want(out_idx, torch.int32, "out_idx")
        K = sum((s.k if hasattr(s, "k") else s[2]) for s in segs)
        if residuals.shape != grads.shape or len(seeds) != W or out_vals.numel() < W * K or out_idx.numel() < W * K:
            raise ValueError("buffer sizes do not match W, n and the segment table")
        _check(self._lib.sc_compress_batch(self._h, scheme, W, _ptr(grads), _ptr(residuals), n, _segments(segs),
                                           len(segs), _seeds(seeds), _ptr(out_vals), _ptr(out_idx),
                                           _stream(stream)), "sc_compress_batch")

    def sc_aggregate(self, W: int, vals, idx, k: int, n: int, out, stream=None) -> None:
        _want(vals, torch.float32, "vals"), _want(idx, torch.int32, "idx"), _want(out, torch.float32, "out")
        if vals.numel() < W * k or idx.numel() < W * k or out.numel() < n:
            raise ValueError("buffer sizes do not match W, k and n")
        _check(self._lib.sc_aggregate(self._h, W, _ptr(vals), _ptr(idx), k, n, _ptr(out), _stream(stream)),
               "sc_aggregate")

    def sc_aggregate_shared(self, W: int, vals, idx, k: int, n: int, out, stream=None) -> None:
        _want(vals, torch.float32, "vals"), _want(idx, torch.int32, "idx"), _want(out, torch.float32, "out")
        if vals.numel() < W * k or idx.numel() < k or out.numel() < n:
            raise ValueError("buffer sizes do not match W, k and n")
        _check(self._lib.sc_aggregate_shared(self._h, W, _ptr(vals), _ptr(idx), k, n, _ptr(out), _stream(stream)),
               "sc_aggregate_shared")

    def sc_aggregate_apply(self, W: int, vals, idx, k: int, n: int, x, stream=None, shared: bool = False) -> None:
        """x <- x - average of the W messages, touching only the coordinates that were sent."""
        _want(vals, torch.float32, "vals"), _want(idx, torch.int32, "idx"), _want(x, torch.float32, "x")
        if vals.numel() < W * k or idx.numel() < (k if shared else W * k) or x.numel() < n:
            raise ValueError("buffer sizes do not match W, k and n")
        fn = self._lib.sc_aggregate_apply_shared if shared else self._lib.sc_aggregate_apply
        _check(fn(self._h, W, _ptr(vals), _ptr(idx), k, n, _ptr(x), _stream(stream)), "sc_aggregate_apply")

    def sc_step(self, scheme: int, grads, residuals, segs, seeds, out_vals, out_idx, out, stream=None) -> None:
        W, n = grads.shape
        _want(grads, torch.float32, "grads"), _want(residuals, torch.float32, "residuals")
        _want(out_vals, torch.float32, "out_vals"), _want(out_idx, torch.int32, "out_idx")
        _want(out, torch.float32, "out")
        K = sum((s.k if hasattr(s, "k") else s[2]) for s in segs)
        if (residuals.shape != grads.shape or len(seeds) != W or out_vals.numel() < W * K
                or out_idx.numel() < W * K or out.numel() < n):
            raise ValueError("buffer sizes do not match W, n and the segment table")
        _check(self._lib.sc_step(self._h, scheme, W, _ptr(grads), _ptr(residuals), n, _segments(segs), len(segs),
                                 _seeds(seeds), _ptr(out_vals), _ptr(out_idx), _ptr(out), _stream(stream)),
               "sc_step")

    def sc_step_apply(self, scheme: int, grads, residuals, segs, seeds, out_vals, out_idx, x, stream=None) -> None:
        """Compress W workers, then x <- x - average of their messages at the sent coordinates only."""
        W, n = grads.shape
        _want(grads, torch.float32, "grads"), _want(residuals, torch.float32, "residuals")
        _want(out_vals, torch.float32, "out_vals"), _want(out_idx, torch.int32, "out_idx")
        _want(x, torch.float32, "x")
        K = sum((s.k if hasattr(s, "k") else s[2]) for s in segs)
        if (residuals.shape != grads.shape or len(seeds) != W or out_vals.numel() < W * K
                or out_idx.numel() < W * K or x.numel() < n):
            raise ValueError("buffer sizes do not match W, n and the segment table")
        _check(self._lib.sc_step_apply(self._h, scheme, W, _ptr(grads), _ptr(residuals), n, _segments(segs), len(segs),
                                       _seeds(seeds), _ptr(out_vals), _ptr(out_idx), _ptr(x), _stream(stream)),
               "sc_step_apply")

    def sc_step_host(self, scheme: int, h_grads, residuals, segs, seeds, h_out, stream=None) -> None:
        W, n = h_grads.shape
        _want(h_grads, torch.float32, "h_grads", cuda=False), _want(h_out, torch.float32, "h_out", cuda=False)
        _want(residuals, torch.float32, "residuals")
        if h_grads.is_cuda or h_out.is_cuda:
            raise TypeError("h_grads and h_out must be host tensors")
        if residuals.shape != h_grads.shape or len(seeds) != W or h_out.numel() < n:
            raise ValueError("buffer sizes do not match W and n")
        _check(self._lib.sc_step_host(self._h, scheme, W, _ptr(h_grads), _ptr(residuals), n, _segments(segs),
                                      len(segs), _seeds(seeds), _ptr(h_out), _stream(stream)), "sc_step_host")
