#!/usr/bin/env python3
"""Writes the stored answers for the shape tag and the certificate digest.

Stand-alone on purpose: it imports nothing from the oracle, from the tests'
definition module or from the CUDA package, and derives every constant from
integer square roots, so that a change made to the formula in the oracle and in
the tests' restatement at the same time still disagrees with the stored lines.

    python tests/golden/make_tag_kat.py        # prints the lines kept in sf64_kat.txt

Definitions (this project's reading of "a deterministic hash over dtype, shape
and bytes", Sec. 5.2; the paper fixes the properties, not the function):
  mix(z)   : z ^= z >> 32; z *= A; z ^= z >> 29; z *= B; z ^= z >> 32   (mod 2^64)
             A = frac(sqrt 2) * 2^64 made odd, B = frac(sqrt 3) * 2^64
  shape tag: a = mix(frac(sqrt 11) * 2^64  xor  ndim); for each dim: a = mix(a xor dim)
  certificate over majority hashes e_0..e_{C-1}:
             a = mix(frac(sqrt 13) * 2^64  xor  C); for each e: a = mix(a xor e)
"""
from functools import reduce
from math import isqrt

W = 64
MASK = (1 << W) - 1


def frac_sqrt(prime: int) -> int:
    """The first 64 fractional bits of sqrt(prime), as an integer."""
    return isqrt(prime << (2 * W)) & MASK


A = frac_sqrt(2) | 1
B = frac_sqrt(3)
SEED_SHAPE = frac_sqrt(11)
SEED_CERT = frac_sqrt(13)


def mix(z: int) -> int:
    for shift, mult in ((32, A), (29, B)):
        z = ((z ^ (z >> shift)) * mult) & MASK
    return z ^ (z >> 32)


def chain(seed: int, items) -> int:
    items = list(items)
    return reduce(lambda acc, x: mix(acc ^ (x & MASK)), items, mix(seed ^ len(items)))


CASES_SHAPE = [[], [7], [4096, 4096], [14336, 4096], [1, 2, 3, 4, 5, 6]]
CASES_CERT = [[], [1, 2, 3], [MASK, 0, MASK], list(range(100, 165))]


def fmt(xs):
    return ",".join(str(x) for x in xs) if xs else "-"


if __name__ == "__main__":
    for dims in CASES_SHAPE:
        print(f"shapetag {fmt(dims)} {chain(SEED_SHAPE, dims):#018x}")
    for hs in CASES_CERT:
        print(f"cert {fmt(hs)} {chain(SEED_CERT, hs):#018x}")
