"""Pins for the oracle's exact consensus (Algorithm 1, Exact branch): brute
force against an independently written counting rule, and every case the
paper's prose fixes."""
import itertools

import numpy as np
import pytest

import defn
from oracle import scout_oracle as orc


def _sigs(rows):
    """rows: list of per-chunk lists of hash values -> sigs[C, R]."""
    a = np.zeros((len(rows), len(rows[0])), dtype=orc.SIG_DTYPE)
    for c, row in enumerate(rows):
        a["hash"][c] = row
    # sidecar fields must never influence the vote: fill them with junk
    a["sum"] = np.arange(a.size).reshape(a.shape)
    a["nan_count"] = 3
    return a


@pytest.mark.parametrize("R", [2, 3, 4, 5, 6])
def test_brute_force_all_assignments(R):
    rows = [list(t) for t in itertools.product(range(4), repeat=R)]
    out = orc.vote(_sigs(rows))
    n_out, und = 0, []
    for c, row in enumerate(rows):
        s, B = defn.vote_one(row)
        assert out["status"][c] == s and int(out["bitmap"][c]) == B, row
        n_out += bin(B).count("1")
        if s == defn.INCONCLUSIVE:
            und.append(c)
    assert out["undecided"] == und
    assert out["counts"][0] == len(rows) and out["counts"][4] == n_out == len(out["outliers"])
    assert out["outliers"] == sorted(out["outliers"])
    assert sum(out["counts"][1:4]) == len(rows)


def test_cases_fixed_by_the_paper():
    a, b, c, d = 11, 22, 33, 44
    cases = [
        ([a, a], orc.AGREE, 0),                      # two ranks, equal
        ([a, b], orc.INCONCLUSIVE, 0),               # two ranks differ: refuse to pick a side
        ([a, a, a], orc.AGREE, 0),
        ([a, b, a], orc.ATTRIBUTED, 0b010),
        ([a, b, c], orc.INCONCLUSIVE, 0),            # no strict majority
        ([a, a, b, b], orc.INCONCLUSIVE, 0),         # 2-vs-2: c* = N/2 is not a majority
        ([a, b, c, a], orc.INCONCLUSIVE, 0),         # 2-1-1 of four
        ([a, a, a, b, c], orc.ATTRIBUTED, 0b11000),  # several distinct minority values
        ([b, b, b, a, a], orc.ATTRIBUTED, 0b11000),  # a fault held by the majority wins
        ([a, a, a, b, b, b], orc.INCONCLUSIVE, 0),
        ([a, a, a, a, b, c, d], orc.ATTRIBUTED, 0b1110000),
    ]
    for row, status, B in cases:
        out = orc.vote(_sigs([row]))
        assert (out["status"][0], int(out["bitmap"][0])) == (status, B), row


def test_wide_groups_and_bit_positions():
    R = 64
    row = [7] * R
    row[63] = 9
    row[0] = 8
    out = orc.vote(_sigs([row]))
    assert out["status"][0] == orc.ATTRIBUTED and int(out["bitmap"][0]) == (1 << 63) | 1
    assert out["outliers"] == [(0, 0), (0, 63)]
    half = [1] * 32 + [2] * 32
    assert orc.vote(_sigs([half]))["status"][0] == orc.INCONCLUSIVE
    with pytest.raises(ValueError):
        orc.vote(np.zeros((1, 1), dtype=orc.SIG_DTYPE))       # a singleton has no comparison
    with pytest.raises(ValueError):
        orc.vote(np.zeros((1, 65), dtype=orc.SIG_DTYPE))


def test_list_truncation_keeps_true_counts():
    rows = [[1, 1, 2], [1, 2, 3], [5, 5, 5], [4, 9, 4], [1, 2, 3]]
    full = orc.vote(_sigs(rows))
    assert full["rc"] == 0 and full["outliers"] == [(0, 2), (3, 1)] and full["undecided"] == [1, 4]
    cut = orc.vote(_sigs(rows), outlier_cap=1, undecided_cap=1)
    assert cut["rc"] == -6 and cut["counts"] == full["counts"]
    assert cut["outliers"] == [(0, 2)] and cut["undecided"] == [1]


def test_permuting_replicas_permutes_bitmap_bits_only():
    import random
    rng = random.Random(3)
    for _ in range(200):
        R = rng.randrange(2, 9)
        row = [rng.randrange(3) for _ in range(R)]
        perm = list(range(R))
        rng.shuffle(perm)
        s0, B0 = (lambda o: (o["status"][0], int(o["bitmap"][0])))(orc.vote(_sigs([row])))
        s1, B1 = (lambda o: (o["status"][0], int(o["bitmap"][0])))(
            orc.vote(_sigs([[row[p] for p in perm]])))
        assert s0 == s1
        assert B1 == sum(((B0 >> perm[j]) & 1) << j for j in range(R))


def test_certify_rollup():
    a = 5
    clean = _sigs([[a, a, a], [7, 7, 7]])
    r = orc.certify(clean)
    assert r["report"]["verdict"] == 0 and r["report"]["replica_union_bitmap"] == 0
    assert r["report"]["certificate"] == defn.certificate([a, 7])
    one_bad = _sigs([[a, a, 9], [7, 7, 7], [3, 2, 2]])
    r = orc.certify(one_bad)
    rep = r["report"]
    assert rep["verdict"] == 1 and rep["replica_union_bitmap"] == 0b101
    assert rep["certificate"] == defn.certificate([a, 7, 2])
    assert r["replica_bad"] == [1, 0, 1] and r["outliers"] == [(0, 2), (2, 0)]
    assert (rep["n_chunks"], rep["n_agree"], rep["n_attributed"], rep["n_inconclusive"]) == (3, 1, 2, 0)
    split = _sigs([[a, a, a], [1, 2, 3]])
    rep = orc.certify(split)["report"]
    assert rep["verdict"] == 2 and rep["certificate"] == 0 and rep["n_undecided"] == 1


def test_wide_vote_equals_the_narrow_one_and_the_counting_rule():
    import random
    rng = random.Random(17)
    # R <= 64: the wide form must reproduce orc_vote, in both table layouts
    for R in (2, 3, 5, 17, 64):
        rows = [[rng.randrange(3) for _ in range(R)] for _ in range(60)]
        sig = _sigs(rows)
        narrow = orc.vote(sig)
        for table, cs, rs in ((sig, R, 1), (np.ascontiguousarray(sig.T), 1, len(rows))):
            wide = orc.vote_wide(table, R, len(rows), cs, rs)
            assert (wide["status"] == narrow["status"]).all()
            assert (wide["bitmap"][:, 0] == narrow["bitmap"]).all()
            assert wide["outliers"] == narrow["outliers"] and wide["undecided"] == narrow["undecided"]
            assert wide["counts"] == narrow["counts"]
    # R > 64: against the counting rule, bit positions across words
    for R in (65, 100, 192, 300):
        rows = []
        for _ in range(25):
            row = [7] * R
            for j in rng.sample(range(R), rng.choice([0, 1, 3, R // 2, R // 2 + 1, R - 1])):
                row[j] = rng.choice([8, 9])
            rows.append(row)
        wide = orc.vote_wide(_sigs(rows), R, len(rows), R, 1)
        for c, row in enumerate(rows):
            s, B = defn.vote_one(row)
            got = sum(int(w) << (64 * k) for k, w in enumerate(wide["bitmap"][c]))
            assert (int(wide["status"][c]), got) == (s, B)
        assert wide["outliers"] == sorted(wide["outliers"])
