"""Writes tests/golden/generator_kat.txt: known answers of the coordinate generators.

The paper says only that coordinates are "randomly selected" (Methodology, Random-k and
Block-random-k items); the generator is this project's own specification.  The file pins
that specification against accidental change: it is produced by the CPU oracle alone
(`python tests/golden/make_generator_kat.py`), and both the oracle and the CUDA library
are tested against it."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import sparsify_oracle as O  # noqa: E402

CASES = [(0, 1, 1), (1, 2, 1), (7, 10, 3), (123456789, 1000, 10), (2 ** 63 + 5, 4097, 12),
         (0xDEADBEEF, 65536, 8), (42, 1_000_003, 6), (99, 350_000_000, 5)]


def lines():
    yield "# seed n k | segment seed (s=0) | block start | random-k coordinates (ascending)"
    for seed, n, k in CASES:
        ss = O.segment_seed(seed, 0)
        yield f"{seed} {n} {k} | {ss} | {O.block_start(ss, n, k)} | " + " ".join(str(int(v)) for v in O.randk_indices(ss, n, k))
    yield "# mix64(a, b)"
    for a, b in ((0, 0), (1, 2), (2 ** 64 - 1, 7)):
        yield f"mix64 {a} {b} = {O.mix64(a, b)}"
    yield "# mix32(x)"
    for x in (0, 1, 0x12345678, 0xFFFFFFFF):
        yield f"mix32 {x} = {O.mix32(x)}"


if __name__ == "__main__":
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "generator_kat.txt"), "w") as f:
        f.write("\n".join(lines()) + "\n")
