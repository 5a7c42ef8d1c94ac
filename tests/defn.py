"""Definitional forms used to pin the CPU oracle: arbitrary-precision integers
for the hash, exact rational / correctly rounded sums for the statistics, and a
counting rule for the vote.  Each is written from the mathematics, in a
different form from the oracle's own code (a direct sum with modular powers
instead of a recurrence; ``Fraction`` and ``math.fsum`` instead of compensated
accumulation; ``collections.Counter`` instead of pairwise comparison)."""
from __future__ import annotations

import math
from collections import Counter
from fractions import Fraction
from math import isqrt

import numpy as np

M64 = 1 << 64
ROW = 128


def golden_ratio_floor(bits: int) -> int:
    """floor(2^bits / phi) with phi = (1 + sqrt 5) / 2, by integer square root:
    2^bits / phi = 2^bits (sqrt 5 - 1) / 2."""
    return (isqrt(5 << (2 * bits)) - (1 << bits)) >> 1


def frac_sqrt64(p: int) -> int:
    """First 64 fractional bits of sqrt(p)."""
    return isqrt(p << 128) % M64


P = golden_ratio_floor(64)
G32 = golden_ratio_floor(32)
C1 = frac_sqrt64(2) | 1
C2 = frac_sqrt64(3)
K0, K1, K2, K3 = (frac_sqrt64(p) for p in (5, 7, 11, 13))


def slot_multiplier(s: int) -> int:
    return (((s + 1) * G32) % (1 << 32)) | 1


def mix64(z: int) -> int:
    z %= M64
    z ^= z >> 32
    z = z * C1 % M64
    z ^= z >> 29
    z = z * C2 % M64
    z ^= z >> 32
    return z


def unmix64(z: int) -> int:
    """Inverse of mix64 (each step is invertible: xor-shift by >= 32 is its own
    inverse, xor-shift by 29 needs two more rounds, odd multipliers invert)."""
    z ^= z >> 32
    z = z * pow(C2, -1, M64) % M64
    z ^= (z >> 29) ^ (z >> 58)
    z = z * pow(C1, -1, M64) % M64
    z ^= z >> 32
    return z


def words(b: bytes):
    n = len(b)
    W = (n + 3) // 4
    padded = b + bytes(4 * W - n)
    return [int.from_bytes(padded[4 * i:4 * i + 4], "little") for i in range(W)]


def hash_raw(b: bytes) -> int:
    """H_raw = sum_i m_{i mod 128} * P^(Q-1-floor(i/128)) * w_i  (mod 2^64)."""
    w = words(b)
    Q = (len(w) + ROW - 1) // ROW
    total = 0
    for i, wi in enumerate(w):
        total += slot_multiplier(i % ROW) * pow(P, Q - 1 - i // ROW, M64) * wi
    return total % M64


def hash_final(h_raw: int, n: int, k: int, d: int, g: int) -> int:
    t = mix64(K0 ^ n)
    t = mix64(t ^ k)
    t = mix64(t ^ d)
    t = mix64(t ^ g)
    return mix64((h_raw + t) % M64)


def sf64(b: bytes, d: int, k: int = 0, g: int = 0) -> int:
    return hash_final(hash_raw(b), len(b), k, d, g)


def shape_tag(dims) -> int:
    a = mix64(K2 ^ len(dims))
    for x in dims:
        a = mix64(a ^ x)
    return a


def rollup(hashes) -> int:
    a = mix64(K1 ^ len(hashes))
    for h in hashes:
        a = mix64(a ^ h)
    return a


def certificate(majority_hashes) -> int:
    a = mix64(K3 ^ len(majority_hashes))
    for h in majority_hashes:
        a = mix64(a ^ h)
    return a


# ---- statistics ------------------------------------------------------------

def values_f64(b: bytes, dtype: str) -> np.ndarray:
    """Element values as float64 (exact for the float types)."""
    a = np.frombuffer(b, dtype=np.uint8)
    if dtype == "f32":
        return a.view("<f4").astype(np.float64)
    if dtype == "bf16":
        return (a.view("<u2").astype(np.uint32) << 16).view("<f4").astype(np.float64)
    if dtype == "f16":
        return a.view("<f2").astype(np.float64)
    if dtype == "f64":
        return a.view("<f8").copy()
    if dtype == "i64":
        return a.view("<i8").astype(np.float64)
    if dtype == "i32":
        return a.view("<i4").astype(np.float64)
    if dtype == "u8":
        return np.zeros(0)
    raise ValueError(dtype)


def stats(b: bytes, dtype: str):
    """(nan, inf, sum, sumsq, sum_abs): sums over finite elements, exactly
    (rational arithmetic), rounded once to double."""
    x = values_f64(b, dtype)
    nan = int(np.isnan(x).sum())
    inf = int(np.isinf(x).sum())
    fin = [float(v) for v in x[np.isfinite(x)]]
    fr = [Fraction(v) for v in fin]

    def rnd(q):
        try:
            return float(q)
        except OverflowError:
            return math.inf if q > 0 else -math.inf
    return nan, inf, rnd(sum(fr, Fraction(0))), rnd(sum((v * v for v in fr), Fraction(0))), \
        rnd(sum((abs(v) for v in fr), Fraction(0)))


# ---- vote ------------------------------------------------------------------

AGREE, ATTRIBUTED, INCONCLUSIVE = 0, 1, 2


def vote_one(hashes):
    """Exact consensus by counting: a value held by MORE than half the group is
    the reference; everyone else is an outlier."""
    N = len(hashes)
    value, count = Counter(hashes).most_common(1)[0]
    if not (count > N / 2):
        return INCONCLUSIVE, 0
    B = sum(1 << j for j, h in enumerate(hashes) if h != value)
    return (ATTRIBUTED if B else AGREE), B
