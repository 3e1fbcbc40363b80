#!/usr/bin/env python
"""Writes tests/golden/derived_kats.txt from the written definitions, with Python integers only.

    python tests/golden/derive_kats.py [--check]

This script imports nothing of the repository (no oracle, no CUDA library, no numpy): it retypes
the definitions -- SplitMix64 with the increment added first, the keyed counter stream per warp,
the exact remainder, the per-word XOR / wrapping-sum fold -- in arbitrary-precision integers and
prints the known answers the oracle is pinned to.  --check compares with the committed file
instead of writing it (tests/test_oracle_kat.py runs that).
"""
from __future__ import annotations

import sys
from pathlib import Path

M64 = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15
OUT = Path(__file__).resolve().parent / "derived_kats.txt"


def sm64(x: int) -> int:
    z = (x + GAMMA) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def word(i: int) -> int:
    return sm64(i) & 0xFFFFFFFF


def key(seed: int, v: int) -> int:
    return sm64(sm64(seed) ^ v)


def draw(seed: int, v: int, i: int) -> int:
    return sm64((key(seed, v) + i * GAMMA) & M64)


def line(seed: int, v: int, i: int, base: int, n: int) -> int:
    return base + draw(seed, v, i) % n


def checksum(seed: int, v: int, W: int, reads: int, base: int, n: int):
    x = s = 0
    for i in range(reads):
        first = line(seed, v, i, base, n) * 32 * W
        for j in range(32 * W):
            w = word(first + j)
            x ^= w
            s = (s + w) & 0xFFFFFFFF
    return x, s


HEADER = """\
# Known answers for the hash fill, the keyed line-index stream and per-warp checksums, derived
# from the written definitions with Python big integers (tests/golden/derive_kats.py, which
# imports nothing of this repository).  The paper prints no worked example: Section 2.1 describes
# its benchmark in prose only.  tests/test_oracle_kat.py checks the oracle against every line.
# Nothing here was produced by the CUDA path or by the oracle.
#
"""


def text() -> str:
    L = [HEADER.rstrip("\n")]
    L.append("# word i0 : hex words           -> buffer contents word(i0), word(i0+1), ...")
    L.append("word 0 : " + " ".join(f"{word(i):08X}" for i in range(8)))
    L.append("# sm64 x : value")
    for x in (0x100000000, 0xFFFFFFFFFFFFFFFF):
        L.append(f"sm64 0x{x:X} : {sm64(x):016X}")
    L.append("# fold first last : X S         -> xor / sum mod 2^32 of word(first..last)")
    x = s = 0
    for i in range(1024):
        x ^= word(i)
        s = (s + word(i)) & 0xFFFFFFFF
    L.append(f"fold 0 1023 : {x:08X} {s:08X}")
    L.append("# key seed v : k_v")
    for seed, v in ((1, 0), (1, 1), (1, 65535), (7, 0), (23, 9471)):
        L.append(f"key {seed} {v} : {key(seed, v):016X}")
    L.append("# draw seed v i0 : r(seed,v,i0), r(seed,v,i0+1), ...")
    L.append("draw 1 0 0 : " + " ".join(f"{draw(1, 0, i):016X}" for i in range(4)))
    L.append("# lines seed v base n : first line indices (decimal)")
    for seed, v, base, n, count in ((1, 0, 0, 1 << 23, 4), (1, 1, 0, 1 << 23, 4),
                                    (1, 65535, 0, 1 << 23, 4), (7, 5, 0, 402653184, 4),
                                    (11, 3, 0, 1 << 27, 4), (23, 42, 1000, 777, 8)):
        L.append(f"lines {seed} {v} {base} {n} : "
                 + " ".join(str(line(seed, v, i, base, n)) for i in range(count)))
    L.append("# sum seed v W reads base n : X S   -> warp checksum")
    for seed, v, W, reads, base, n in ((1, 0, 1, 16, 0, 1 << 23), (1, 1, 1, 16, 0, 1 << 23),
                                       (1, 2, 1, 16, 0, 1 << 23), (1, 65535, 1, 16, 0, 1 << 23),
                                       (7, 5, 1, 4, 0, 402653184), (11, 3, 1, 4, 0, 1 << 28),
                                       (11, 3, 2, 4, 0, 1 << 27), (11, 3, 4, 4, 0, 1 << 26),
                                       (23, 42, 1, 8, 1000, 777)):
        x, s = checksum(seed, v, W, reads, base, n)
        L.append(f"sum {seed} {v} {W} {reads} {base} {n} : {x:08X} {s:08X}")
    return "\n".join(L) + "\n"


def main(argv) -> int:
    t = text()
    if "--check" in argv:
        if OUT.read_text() != t:
            sys.stderr.write("derived_kats.txt differs from what the definitions give\n")
            return 1
        return 0
    OUT.write_text(t)
    return 0


if __name__ == "__main__":
    raise SystemExit(main(sys.argv[1:]))
