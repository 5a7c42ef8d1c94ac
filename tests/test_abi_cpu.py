"""The C-ABI library loads without a GPU and exports what include/scout.h
declares; argument validation that needs no device works."""
import os
import re

import numpy as np
import pytest

import defn
from paper_2608_11034_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    inc = os.path.join(ROOT, "include")
    header = "".join(open(os.path.join(inc, h)).read() for h in sorted(os.listdir(inc)))
    names = set(re.findall(r"SCOUT_API[^;(]*?\b(scout_\w+)\s*\(", header))
    assert {"scout_sign_chunks", "scout_consensus_vote", "scout_certify", "scout_plan_create",
            "scout_plan_bind", "scout_plan_destroy"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), n
    assert binding.scout_version() >= 100
    # the binding offers one function per C entry point, under the same name
    for n in names:
        assert n in ("scout_strerror", "scout_last_cuda_error") or hasattr(binding, n), n


def test_error_strings(lib):
    for code in range(0, -7, -1):
        assert lib.scout_strerror(code)
    assert b"unknown" in lib.scout_strerror(-99)


def test_shape_tag_matches_its_definition():
    for dims in ([], [7], [4096, 4096], [14336, 4096], [2**40, 3, 1]):
        assert binding.scout_shape_tag(dims) == defn.shape_tag(dims)
    # and the stored answers (written by a stand-alone script, tests/golden/make_tag_kat.py)
    stored = [ln.split() for ln in open(os.path.join(ROOT, "tests", "golden", "sf64_kat.txt"))
              if ln.startswith("shapetag")]
    assert len(stored) >= 3
    for _, dims, want in stored:
        dims = [] if dims == "-" else [int(x) for x in dims.split(",")]
        assert binding.scout_shape_tag(dims) == int(want, 16)


def test_plan_arguments_are_validated_before_any_device_work():
    t = np.zeros(1, dtype=binding.TENSOR_DTYPE)
    t[0] = (1024, binding.DT_F32, 0, 0)
    bad = [
        (0, t, 512, binding.ERR_INVALID),
        (1025, t, 512, binding.ERR_UNSUPPORTED),  # beyond the widest supported peer group
        (3, t, 0, binding.ERR_INVALID),
        (3, t, 1000, binding.ERR_INVALID),       # chunk size must be a multiple of 512
        (3, t, (1 << 30) + 512, binding.ERR_INVALID),
    ]
    for R, tt, cb, code in bad:
        with pytest.raises(binding.ScoutError) as e:
            binding.scout_plan_create(R, tt, cb)
        assert e.value.code == code
    for nbytes, dt in ((0, binding.DT_F32), (6, binding.DT_F32), (12, binding.DT_I64), (4, 99)):
        t2 = t.copy()
        t2[0] = (nbytes, dt, 0, 0)
        with pytest.raises(binding.ScoutError) as e:
            binding.scout_plan_create(3, t2, 512)
        assert e.value.code == binding.ERR_INVALID


def test_vote_arguments_are_validated(lib):
    assert lib.scout_consensus_vote(1, 1, 8, 0, 0, 0, 0, 0, 0, 8, 0) == binding.ERR_INVALID
    assert lib.scout_consensus_vote(65, 1, 8, 0, 0, 0, 0, 0, 0, 8, 0) == binding.ERR_UNSUPPORTED
    assert lib.scout_consensus_vote(3, 1, 8, 0, 0, 0, 0, 0, 0, 0, 0) == binding.ERR_INVALID
    assert lib.scout_consensus_vote(3, 1, 8, 0, 0, 0, 5, 0, 0, 8, 0) == binding.ERR_INVALID
    # a singleton has no comparison, whatever the bitmap width
    assert lib.scout_consensus_vote_wide(1, 1, 8, 1, 1, 0, 0, 0, 0, 0, 0, 8, 0) == binding.ERR_INVALID
    assert lib.scout_consensus_vote_wide(1025, 1, 8, 1025, 1, 0, 0, 0, 0, 0, 0, 8, 0) == binding.ERR_UNSUPPORTED
    assert lib.scout_consensus_vote_wide(3, 1, 8, 0, 1, 0, 0, 0, 0, 0, 0, 8, 0) == binding.ERR_INVALID
