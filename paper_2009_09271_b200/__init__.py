"""B200-native (sm_100a) gradient compressor for sparsified synchronous SGD with
error feedback: top-k / random-k / block-random-k selection, message packing,
residual writeback and dense aggregation, behind a small C ABI
(include/sparsecomm.h) with a ctypes binding of the same names."""
from .binding import (SC_RANDBLOCK, SC_RANDBLOCK_WRAP, SC_RANDK, SC_TOPK, SCHEMES, Context, EXPORTS, LIB_PATH, ScSegment,
                      SparseCommError, load_library, sc_aggregate_static, strerror)

__all__ = ["SC_TOPK", "SC_RANDK", "SC_RANDBLOCK", "SC_RANDBLOCK_WRAP", "SCHEMES", "Context", "EXPORTS", "LIB_PATH", "ScSegment",
           "SparseCommError", "load_library", "sc_aggregate_static", "strerror"]
