"""Property-based pins of the oracle (hypothesis): the algebra that any correct
implementation of the signature and the vote must satisfy, on random inputs."""
import numpy as np
from hypothesis import given, settings, strategies as st

import defn
from oracle import scout_oracle as orc

M64 = 1 << 64
blobs = st.binary(min_size=1, max_size=3000)


@settings(max_examples=150, deadline=None)
@given(blobs)
def test_hash_equals_the_big_integer_definition(b):
    assert orc.hash_raw(b) == defn.hash_raw(b)


@settings(max_examples=150, deadline=None)
@given(blobs, st.integers(min_value=0, max_value=5))
def test_segment_combine_at_any_row_boundary(b, r):
    rows = (len(b) + 511) // 512
    r = min(r, rows)
    left, right = b[:512 * r], b[512 * r:]
    hl = orc.hash_raw(left) if left else 0
    hr = orc.hash_raw(right) if right else 0
    assert orc.hash_raw(b) == (hl * pow(defn.P, rows - r, M64) + hr) % M64


@settings(max_examples=150, deadline=None)
@given(blobs, st.data())
def test_changing_one_word_always_changes_the_hash(b, data):
    pos = data.draw(st.integers(min_value=0, max_value=len(b) - 1))
    new = data.draw(st.integers(min_value=1, max_value=255))
    c = bytearray(b)
    c[pos] ^= new
    assert orc.hash_raw(bytes(c)) != orc.hash_raw(b)
    # linearity: the difference depends only on the changed word and its position
    w = pos // 4
    rows = (len(b) + 3) // 4
    rows = (rows + 127) // 128
    delta = (int.from_bytes(bytes(c[4 * w:4 * w + 4]).ljust(4, b"\0"), "little")
             - int.from_bytes(bytes(b[4 * w:4 * w + 4]).ljust(4, b"\0"), "little"))
    want = defn.slot_multiplier(w % 128) * pow(defn.P, rows - 1 - w // 128, M64) * delta
    assert (orc.hash_raw(bytes(c)) - orc.hash_raw(b)) % M64 == want % M64


@settings(max_examples=100, deadline=None)
@given(st.lists(st.floats(allow_nan=True, allow_infinity=True, width=32), min_size=1, max_size=400))
def test_fp32_statistics_against_exact_rationals(xs):
    b = np.array(xs, dtype=np.float32).tobytes()
    nan, inf, s, q, a = orc.stats(b, orc.DT_F32)
    dn, di, ds, dq, da = defn.stats(b, "f32")
    assert (nan, inf) == (dn, di)
    assert abs(s - ds) <= 2**-52 * da and abs(q - dq) <= 2**-52 * dq and abs(a - da) <= 2**-52 * da


@settings(max_examples=200, deadline=None)
@given(st.lists(st.integers(min_value=0, max_value=4), min_size=2, max_size=64))
def test_vote_against_the_counting_rule(row):
    sig = np.zeros((1, len(row)), dtype=orc.SIG_DTYPE)
    sig["hash"][0] = [1000 + v for v in row]
    out = orc.vote(sig)
    s, B = defn.vote_one(row)
    assert (int(out["status"][0]), int(out["bitmap"][0])) == (s, B)
    # the three statuses keep an all-zero bitmap from being ambiguous
    if B == 0:
        assert s in (defn.AGREE, defn.INCONCLUSIVE)
        assert (s == defn.AGREE) == (len(set(row)) == 1)
    wide = orc.vote_wide(sig, len(row), 1, len(row), 1)
    assert int(wide["status"][0]) == s and int(wide["bitmap"][0, 0]) == B
