"""Pins for the oracle's SF64 hash: constants from their derivations, stored
known answers, big-integer brute force of the plain definition, and the
algebraic properties that make single-word faults certain to be caught."""
import os
import random

import numpy as np
import pytest

import defn
from oracle import scout_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sf64_kat.txt")
M64 = 1 << 64


def _gen(name, n):
    if name == "one":
        return bytes([1, 0, 0, 0])
    if name == "mod251":
        return bytes(i % 251 for i in range(n))
    if name == "quad":
        return bytes((i * i + 7 * i) % 256 for i in range(n))
    if name == "zero":
        return bytes(n)
    if name == "lin":
        return bytes((31 * i + 7) % 256 for i in range(n))
    raise ValueError(name)


def _int_list(field):
    return [] if field == "-" else [int(x) for x in field.split(",")]


def _golden_tags():
    """-> (shape-tag cases, certificate cases) from the stored file."""
    shape, cert = [], []
    for line in open(GOLDEN):
        f = line.split()
        if f and f[0] == "shapetag":
            shape.append((_int_list(f[1]), int(f[2], 16)))
        elif f and f[0] == "cert":
            cert.append((_int_list(f[1]), int(f[2], 16)))
    return shape, cert


def _golden():
    kat, roll, mult, mix = [], [], [], []
    for line in open(GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#") or f[0] in ("shapetag", "cert"):
            continue
        if f[0] == "rollup":
            roll.append(([] if f[1] == "-" else [int(x) for x in f[1].split(",")], int(f[2], 16)))
        elif f[0] == "mult":
            mult.append((int(f[1]), int(f[2], 16)))
        elif f[0] == "mix":
            mix.append((int(f[1]), int(f[2], 16)))
        else:
            kat.append((f[0], int(f[1]), int(f[2]), int(f[3]), int(f[4], 0), int(f[5], 16), int(f[6], 16)))
    return kat, roll, mult, mix


def test_constants_follow_their_derivations():
    # floor(2^64/phi), floor(2^32/phi), fractional bits of square roots of primes
    assert defn.P == 0x9E3779B97F4A7C15 and defn.P % 4 == 1
    assert defn.G32 == 0x9E3779B9
    assert (defn.C1, defn.C2) == (0x6A09E667F3BCC909, 0xBB67AE8584CAA73B)
    assert (defn.K0, defn.K1, defn.K2, defn.K3) == (0x3C6EF372FE94F82B, 0xA54FF53A5F1D36F1,
                                                    0x510E527FADE682D1, 0x9B05688C2B3E6C1F)
    ms = [orc.slot_multiplier(s) for s in range(128)]
    assert ms == [defn.slot_multiplier(s) for s in range(128)]
    assert len(set(ms)) == 128 and all(m & 1 and m < 2**32 for m in ms)


def test_known_answers():
    kat, roll, mult, mix = _golden()
    assert len(kat) == 8
    for name, n, d, k, g, h_raw, h in kat:
        b = _gen(name, n)
        assert orc.hash_raw(b) == h_raw, (name, n)
        assert orc.hash_final(h_raw, n, k, d, g) == h, (name, n)
        assert int(orc.sign_chunk(b, d, k, g)["hash"]) == h
        # the definitional form agrees with the stored values too
        assert defn.hash_raw(b) == h_raw and defn.sf64(b, d, k, g) == h
    for hs, want in roll:
        assert orc.rollup(hs) == want == defn.rollup(hs)
    for s, want in mult:
        assert orc.slot_multiplier(s) == want
    for z, want in mix:
        assert orc.mix64(z) == want


def test_shape_tag_and_certificate_known_answers():
    """Stored values from a stand-alone big-integer script (tests/golden/make_tag_kat.py):
    the oracle and the tests' restatement must both reproduce them."""
    shape, cert = _golden_tags()
    assert len(shape) >= 3 and len(cert) >= 2
    for dims, want in shape:
        assert orc.shape_tag(dims) == want, dims
        assert defn.shape_tag(dims) == want, dims
    for hashes, want in cert:
        # every replica holds the same hash per chunk: each chunk's majority hash is that hash
        R = 3
        sigs = np.zeros((len(hashes), R), dtype=orc.SIG_DTYPE)
        for c, h in enumerate(hashes):
            sigs["hash"][c, :] = h
        rep = orc.certify(sigs)["report"]
        assert rep["verdict"] == 0 and rep["certificate"] == want, hashes
        assert defn.certificate(hashes) == want
    # one outvoted replica does not change the certificate: it is over the majority hashes
    hashes, want = cert[1]
    sigs = np.zeros((len(hashes), 3), dtype=orc.SIG_DTYPE)
    for c, h in enumerate(hashes):
        sigs["hash"][c, :] = h
    sigs["hash"][1, 2] ^= 0x10
    rep = orc.certify(sigs)["report"]
    assert rep["verdict"] == 1 and rep["certificate"] == want


def test_stored_tag_lines_match_their_generator():
    """The committed generator still prints exactly the stored lines."""
    import subprocess
    import sys
    script = os.path.join(os.path.dirname(GOLDEN), "make_tag_kat.py")
    out = subprocess.run([sys.executable, script], capture_output=True, text=True, check=True).stdout
    stored = [ln.strip() for ln in open(GOLDEN) if ln.startswith(("shapetag", "cert"))]
    assert out.split("\n")[:-1] == stored


def test_mix64_is_a_bijection():
    rng = random.Random(1)
    for _ in range(2000):
        z = rng.getrandbits(64)
        assert orc.mix64(z) == defn.mix64(z)
        assert defn.unmix64(orc.mix64(z)) == z
    assert orc.mix64(0) == 0


@pytest.mark.parametrize("n", list(range(1, 40)) + [127, 128, 129, 255, 256, 257, 508, 509, 510,
                                                    511, 512, 513, 515, 516, 1023, 1024, 1025,
                                                    1536, 2047, 2049, 4096, 5000])
def test_brute_force_big_integer_definition(n):
    rng = random.Random(n)
    b = bytes(rng.getrandbits(8) for _ in range(n))
    assert orc.hash_raw(b) == defn.hash_raw(b)
    for d, k, g in ((0, 0, 0), (2, 7, 0x1234), (5, 2**40 + 3, M64 - 1)):
        assert orc.hash_final(orc.hash_raw(b), n, k, d, g) == defn.sf64(b, d, k, g)


def test_closed_forms():
    # all-zero bytes hash to 0 before the metadata mix, whatever the length
    for n in (1, 4, 512, 513, 70000):
        assert orc.hash_raw(bytes(n)) == 0
    # a single non-zero word w at slot s of the last row contributes m_s * w
    for s in (0, 1, 5, 127):
        b = bytearray(512)
        b[4 * s:4 * s + 4] = (0xDEADBEEF).to_bytes(4, "little")
        assert orc.hash_raw(bytes(b)) == defn.slot_multiplier(s) * 0xDEADBEEF % M64
    # the same word one row earlier is multiplied by P once more
    b = bytearray(1024)
    b[4:8] = (12345).to_bytes(4, "little")
    assert orc.hash_raw(bytes(b)) == defn.slot_multiplier(1) * 12345 * defn.P % M64
    # trailing bytes beyond a word boundary read as zero: 01 == 01 00 00 00 before the mix
    assert orc.hash_raw(b"\x01") == orc.hash_raw(b"\x01\x00\x00\x00") == 0x9E3779B9
    # ... but the byte length enters the final hash
    assert orc.sign_chunk(b"\x01", 0)["hash"] != orc.sign_chunk(b"\x01\x00\x00\x00", 0)["hash"]


def test_segment_combine_identity():
    """H_raw(whole) = H_raw(left) * P^(rows right) + H_raw(right) for a split
    on a row boundary: the identity that lets a scan be cut into pieces."""
    rng = random.Random(7)
    b = bytes(rng.getrandbits(8) for _ in range(512 * 9 + 130))
    Q = (len(b) + 511) // 512
    for r in (1, 2, 5, 9):
        left, right = b[:512 * r], b[512 * r:]
        want = (orc.hash_raw(left) * pow(defn.P, Q - r, M64) + orc.hash_raw(right)) % M64
        assert orc.hash_raw(b) == want


def test_every_single_bit_flip_changes_the_hash():
    rng = random.Random(11)
    n = 4096
    base = bytearray(rng.getrandbits(8) for _ in range(n))
    h0 = orc.hash_raw(bytes(base))
    seen = {h0}
    for byte in range(n):
        for bit in range(8):
            base[byte] ^= 1 << bit
            h = orc.hash_raw(bytes(base))
            base[byte] ^= 1 << bit
            assert h != h0
            seen.add(h)
    assert len(seen) == 8 * n + 1          # all distinct, too


def test_word_swaps_are_detected():
    rng = random.Random(13)
    n = 2048                                 # 512 words: 4 rows
    b = bytearray(rng.getrandbits(8) for _ in range(n))
    w = [bytes(b[4 * i:4 * i + 4]) for i in range(n // 4)]
    h0 = orc.hash_raw(bytes(b))
    pairs = [(i, j) for i in range(len(w)) for j in range(i + 1, len(w))]
    for i, j in rng.sample(pairs, 6000):
        if w[i] == w[j]:
            continue
        same_row, same_slot = i // 128 == j // 128, i % 128 == j % 128
        c = bytearray(b)
        c[4 * i:4 * i + 4], c[4 * j:4 * j + 4] = w[j], w[i]
        if same_row or same_slot:            # proven; other pairs only with high probability
            assert orc.hash_raw(bytes(c)) != h0
    assert orc.hash_raw(bytes(b)) == h0


def test_metadata_enters_the_signature():
    b = bytes(range(256)) * 4
    base = orc.sign_chunk(b, orc.DT_F32, 0, 0)["hash"]
    assert orc.sign_chunk(b, orc.DT_I32, 0, 0)["hash"] != base          # dtype
    assert orc.sign_chunk(b, orc.DT_F32, 1, 0)["hash"] != base          # position in tensor
    assert orc.sign_chunk(b, orc.DT_F32, 0, orc.shape_tag([16, 16]))["hash"] != \
        orc.sign_chunk(b, orc.DT_F32, 0, orc.shape_tag([256]))["hash"]  # shape
    assert orc.shape_tag([16, 16]) == defn.shape_tag([16, 16])
    assert orc.shape_tag([]) == defn.shape_tag([])


def test_position_sensitivity_and_determinism():
    b = np.arange(4096, dtype=np.uint32).tobytes()
    assert orc.hash_raw(b) == orc.hash_raw(bytes(b))
    rolled = b[4:] + b[:4]
    assert orc.hash_raw(rolled) != orc.hash_raw(b)
    # +0.0 and -0.0 are different bytes, so different evidence
    pz = np.zeros(128, np.float32).tobytes()
    nz = (-np.zeros(128, np.float32)).tobytes()
    assert orc.hash_raw(pz) != orc.hash_raw(nz)
