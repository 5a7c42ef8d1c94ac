"""Oracle for statistical consensus (TEST INFRASTRUCTURE, not product code).

Algorithm 1's Statistical branch and Sec. 5.4, step by step in plain Python
floats (IEEE fp64, one rounding per operation, no fused multiply-add):
m = median, d = RobustScale (median absolute deviation, else interquartile
range, else scaled range), d = 0 -> Agree, else B[j] = 1{|tau_j - m| > kappa d}.

Parity status.  The structure is the paper's.  The constants of RobustScale are
not given there (MAD scaling, quantile rule, range scaling): the readings in
``robust_scale`` are this project's, so those constants are "parity unpinned"
against the paper.  Pinned: median and quantiles against numpy's library
routines, the property the paper states (the scale is zero only when all timings
are identical, and then the result is Agree), closed-form cases, and the
fallback order.
"""
import math

AGREE, ATTRIBUTED = 0, 1


def median(xs):
    s = sorted(xs)
    n = len(s)
    if n % 2:
        return s[n // 2]
    return (s[n // 2 - 1] + s[n // 2]) * 0.5


def quantile(xs, p):
    """Linear interpolation between order statistics at h = (n - 1) p."""
    s = sorted(xs)
    n = len(s)
    h = (n - 1) * p
    k = math.floor(h)
    if k + 1 >= n:
        return s[k]
    return s[k] + (h - k) * (s[k + 1] - s[k])


def robust_scale(xs, m):
    d = median([abs(x - m) for x in xs])              # median absolute deviation, unscaled
    if d == 0.0:
        d = quantile(xs, 0.75) - quantile(xs, 0.25)   # interquartile range
    if d == 0.0:
        d = (max(xs) - min(xs)) / len(xs)             # scaled observed range
    return d


def consensus(xs, kappa):
    """-> (status, bitmap, median, scale)"""
    m = median(xs)
    d = robust_scale(xs, m)
    if d == 0.0:
        return AGREE, 0, m, d
    B = 0
    for j, x in enumerate(xs):
        if abs(x - m) > kappa * d:
            B |= 1 << j
    return (ATTRIBUTED if B else AGREE), B, m, d
