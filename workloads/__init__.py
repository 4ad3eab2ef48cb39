"""Seeded synthetic gradient workloads (inputs only).

This package holds the input recipes shared by the tests, the benchmark and the
CPU oracle's callers.  It contains none of the compressor's arithmetic: it only
produces gradient values, segment tables and (n, k, seed) parameters.
"""
from .gen import *  # noqa: F401,F403
