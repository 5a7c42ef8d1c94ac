"""Statistical consensus (Algorithm 1, Statistical branch): oracle pins on CPU,
then the device kernel against the oracle, bit for bit."""
import random

import numpy as np
import pytest

from oracle import timing_oracle as T


# ---------------------------------------------------------------- oracle pins (CPU)

def test_median_and_quantiles_reduce_to_the_library_routines():
    rng = random.Random(2)
    for _ in range(400):
        n = rng.randrange(2, 65)
        xs = [rng.choice([1.0, 1.5, rng.uniform(0.5, 3.0)]) for _ in range(n)]
        assert T.median(xs) == float(np.median(xs))
        for p in (0.25, 0.75):
            assert T.quantile(xs, p) == float(np.quantile(xs, p, method="linear"))


def test_scale_is_zero_only_when_all_timings_are_identical():
    assert T.consensus([2.5] * 7, 3.5) == (T.AGREE, 0, 2.5, 0.0)
    rng = random.Random(3)
    for _ in range(2000):
        n = rng.randrange(2, 12)
        xs = [rng.choice([1.0, 1.0, 1.0, 2.0, 5.0]) for _ in range(n)]
        _, _, m, d = T.consensus(xs, 3.5)
        assert (d == 0.0) == (len(set(xs)) == 1)
        assert d >= 0.0


def test_fallback_order_and_closed_forms():
    # MAD: values 1..5 -> median 3, deviations {2,1,0,1,2} -> MAD 1
    assert T.robust_scale([1.0, 2.0, 3.0, 4.0, 5.0], 3.0) == 1.0
    # more than half identical: MAD = 0, the interquartile range takes over
    xs = [1.0, 1.0, 1.0, 1.0, 1.0, 2.0, 3.0, 9.0]
    assert T.median([abs(x - 1.0) for x in xs]) == 0.0
    assert T.robust_scale(xs, 1.0) == T.quantile(xs, 0.75) - T.quantile(xs, 0.25) == 1.25
    # one straggler among identical peers: MAD = IQR = 0, scaled range (max-min)/N
    xs = [1.0] * 7 + [9.0]
    assert T.robust_scale(xs, 1.0) == 1.0
    st, B, m, d = T.consensus(xs, 3.5)
    assert (st, B, m, d) == (T.ATTRIBUTED, 1 << 7, 1.0, 1.0)
    # deviations within kappa d stay unreported; a larger kappa needs a larger deviation
    xs = [10.0, 10.1, 9.9, 10.05, 9.95, 10.0, 13.0]
    assert T.consensus(xs, 3.5)[:2] == (T.ATTRIBUTED, 1 << 6)
    assert T.consensus(xs, 100.0)[:2] == (T.AGREE, 0)
    # a fleet-wide slowdown is invisible: shifting every timing changes nothing
    a = T.consensus(xs, 3.5)
    b = T.consensus([x + 100.0 for x in xs], 3.5)
    assert a[1] == b[1]


# ---------------------------------------------------------------- device vs oracle

def _groups(seed, G, N):
    rng = random.Random(seed)
    rows = []
    for g in range(G):
        kind = rng.randrange(6)
        base = rng.uniform(0.5, 50.0)
        if kind == 0:
            row = [base] * N
        elif kind == 1:
            row = [base] * N
            row[rng.randrange(N)] = base * rng.uniform(1.5, 20.0)
        elif kind == 2:
            row = [base * (1 + 0.01 * rng.gauss(0, 1)) for _ in range(N)]
            row[rng.randrange(N)] *= rng.uniform(1.2, 5.0)
        elif kind == 3:
            row = [rng.choice([base, base * 1.01, base * 2]) for _ in range(N)]
        elif kind == 4:
            row = [base * (1 + 0.05 * rng.gauss(0, 1)) for _ in range(N)]
        else:
            row = [float(rng.randrange(1, 4)) for _ in range(N)]
        rows.append(row)
    return rows


@pytest.mark.gpu
@pytest.mark.parametrize("N", [2, 3, 4, 5, 8, 16, 31, 32, 33, 63, 64])
def test_device_kernel_is_bit_identical_to_the_oracle(N):
    import torch
    from paper_2608_11034_b200 import binding as B
    G = 700
    rows = _groups(N, G, N)
    t = torch.tensor(rows, dtype=torch.float64, device="cuda")
    status = torch.empty(G, dtype=torch.uint8, device="cuda")
    bitmap = torch.empty(G, dtype=torch.int64, device="cuda")
    med = torch.empty(G, dtype=torch.float64, device="cuda")
    scale = torch.empty(G, dtype=torch.float64, device="cuda")
    for kappa in (3.5, 1.0):
        B.scout_consensus_timing(N, G, t.data_ptr(), kappa, status.data_ptr(), bitmap.data_ptr(),
                                 med.data_ptr(), scale.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        s, b = status.cpu().numpy(), bitmap.cpu().numpy().view(np.uint64)
        m, d = med.cpu().numpy(), scale.cpu().numpy()
        for g, row in enumerate(rows):
            want = T.consensus(row, kappa)
            assert (int(s[g]), int(b[g]), float(m[g]), float(d[g])) == want, (g, row)
    assert (s == T.ATTRIBUTED).any() and (s == T.AGREE).any()


@pytest.mark.gpu
def test_device_kernel_rejects_bad_arguments():
    import torch
    from paper_2608_11034_b200 import binding as B
    x = torch.zeros(64, dtype=torch.float64, device="cuda")
    for N, kappa, code in ((1, 3.5, B.ERR_INVALID), (65, 3.5, B.ERR_UNSUPPORTED), (4, 0.0, B.ERR_INVALID),
                           (4, float("nan"), B.ERR_INVALID)):
        with pytest.raises(B.ScoutError) as e:
            B.scout_consensus_timing(N, 1, x.data_ptr(), kappa, x.data_ptr(), x.data_ptr(), 0, 0, 0)
        assert e.value.code == code
