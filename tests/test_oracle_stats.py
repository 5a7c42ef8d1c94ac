"""Pins for the oracle's sidecar statistics: exact rational sums, closed forms,
and the finite-only rule."""
import math
import random

import numpy as np
import pytest
import torch

import defn
from oracle import scout_oracle as orc

CODE = {"u8": 0, "f32": 1, "bf16": 2, "i64": 3, "f16": 4, "f64": 5, "i32": 6}


def _rand_bytes(dtype, n_el, seed):
    g = torch.Generator().manual_seed(seed)
    if dtype in ("f32", "bf16", "f16", "f64"):
        td = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16,
              "f64": torch.float64}[dtype]
        lo, hi = (-12, 10) if dtype == "f16" else (-20, 20)
        expo = torch.randint(lo, hi, (n_el,), generator=g).to(torch.float64)
        x = (torch.randn(n_el, generator=g, dtype=torch.float64) * torch.pow(2.0, expo)).to(td)
        return x.view(torch.uint8).numpy().tobytes()
    if dtype == "i64":
        return torch.randint(-2**52, 2**52, (n_el,), generator=g).numpy().tobytes()
    if dtype == "i32":
        return torch.randint(-2**31, 2**31 - 1, (n_el,), generator=g, dtype=torch.int64) \
            .to(torch.int32).numpy().tobytes()
    raise ValueError(dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16", "f64", "i64", "i32"])
def test_sums_match_exact_rational_arithmetic(dtype):
    b = _rand_bytes(dtype, 3001, 5)
    nan, inf, s, q, a = orc.stats(b, CODE[dtype])
    dn, di, ds, dq, da = defn.stats(b, dtype)
    assert (nan, inf) == (dn, di) == (0, 0)
    # the oracle's own error is far below the parity tolerance: at most 1 ulp here
    assert abs(s - ds) <= 2**-52 * da
    assert abs(q - dq) <= 2**-52 * dq
    assert abs(a - da) <= 2**-52 * da
    x = defn.values_f64(b, dtype)
    assert abs(s - math.fsum(x)) <= 2**-52 * da


def test_closed_forms():
    n = 4096
    v = np.float32(0.3125)
    const = np.full(n, v, np.float32).tobytes()
    nan, inf, s, q, a = orc.stats(const, CODE["f32"])
    assert (nan, inf, s, q) == (0, 0, n * 0.3125, n * 0.3125**2)
    alt = (np.float32(0.3125) * np.where(np.arange(n) % 2, -1, 1)).astype(np.float32).tobytes()
    _, _, s, q, a = orc.stats(alt, CODE["f32"])
    assert (s, q, a) == (0.0, n * 0.3125**2, n * 0.3125)
    ints = np.arange(1, 1001, dtype=np.int64).tobytes()
    _, _, s, q, _ = orc.stats(ints, CODE["i64"])
    assert (s, q) == (1000 * 1001 / 2, 1000 * 1001 * 2001 / 6)
    # catastrophic cancellation: naive double summation gets this wrong
    x = np.array([1e30, 1.0, -1e30, 1.0] * 100, np.float64).tobytes()
    _, _, s, _, _ = orc.stats(x, CODE["f64"])
    assert s == 200.0


def test_non_finite_elements_are_counted_and_left_out_of_the_sums():
    x = np.array([1.5, np.nan, -2.0, np.inf, -np.inf, 0.25, np.nan], np.float32)
    nan, inf, s, q, a = orc.stats(x.tobytes(), CODE["f32"])
    assert (nan, inf) == (2, 2)
    assert (s, q, a) == (-0.25, 1.5**2 + 4 + 0.0625, 3.75)
    # bf16: 0x7FC0 quiet NaN, 0x7F80 +inf, 0xFF80 -inf, 0x7F81 signalling NaN pattern
    h = np.array([0x3F80, 0x7FC0, 0x7F80, 0xFF80, 0x7F81, 0xBF80, 0x4000], np.uint16)
    nan, inf, s, q, _ = orc.stats(h.tobytes(), CODE["bf16"])
    assert (nan, inf, s, q) == (2, 2, 2.0, 6.0)
    f = np.array([1.0, np.nan, np.inf, 65504.0], np.float16)
    assert orc.stats(f.tobytes(), CODE["f16"])[:4] == (1, 1, 65505.0, 1.0 + 65504.0**2)
    # integers and bytes have no non-finite values; bytes carry no statistics at all
    assert orc.stats(bytes(range(64)), CODE["u8"]) == (0, 0, 0.0, 0.0, 0.0)


def test_denormals_and_signed_zero():
    tiny = np.array([1e-45, -1e-45, 1e-40, 0.0, -0.0], np.float32)
    nan, inf, s, q, a = orc.stats(tiny.tobytes(), CODE["f32"])
    want = defn.stats(tiny.tobytes(), "f32")
    assert (nan, inf, s, q, a) == want
    sub = np.array([0x0001, 0x8001, 0x007F], np.uint16)        # bf16 subnormals
    assert orc.stats(sub.tobytes(), CODE["bf16"]) == defn.stats(sub.tobytes(), "bf16")


def test_fp16_decode_matches_numpy_for_every_pattern():
    allp = np.arange(65536, dtype=np.uint16)
    vals = allp.view(np.float16).astype(np.float64)
    fin = np.isfinite(vals)
    nan, inf, s, q, a = orc.stats(allp.tobytes(), CODE["f16"])
    assert nan == int(np.isnan(vals).sum()) and inf == int(np.isinf(vals).sum())
    assert a == math.fsum(np.abs(vals[fin])) and q == math.fsum(vals[fin] ** 2)


def test_int64_beyond_2_53_rounds_to_nearest_double_first():
    x = np.array([2**53 + 1, 2**62 + 3, -(2**60) - 1], np.int64)
    _, _, s, q, _ = orc.stats(x.tobytes(), CODE["i64"])
    d = [float(v) for v in x]
    assert s == float(sum(map(lambda v: __import__("fractions").Fraction(v), d)))
