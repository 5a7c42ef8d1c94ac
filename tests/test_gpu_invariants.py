"""Invariants of the CUDA path that follow from the paper's statements about exact
consensus (Sec. 5.3) and from its evaluation protocol (Sec. 10): they must hold
whatever the data, so no oracle run is needed here."""
import random

import numpy as np
import pytest
import torch

import helpers
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def test_thirty_clean_runs_stay_clean_and_identical():
    # the paper reports 30/30 fault-free runs with no report; here: 30 scans of clean replicas
    w = inputs.workload(3, "clean", 1 / 4096)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    first = None
    for _ in range(30):
        plan.sign_and_vote()
        got = plan.fetch()
        assert got["outliers"] == [] and got["undecided"] == []
        assert got["counts"][1] == plan.C
        blob = got["sigs"].tobytes()
        first = first or blob
        assert blob == first
    helpers.assert_guards(plan)
    plan.close()


def test_permuting_the_replicas_permutes_columns_and_bitmap_bits_only():
    w = inputs.workload(5, "default", 1 / 200)
    _, views = inputs.generate(w, "cuda")
    base = helpers.gpu_sign_vote(w, views)
    rng = random.Random(4)
    perm = list(range(w.R))
    rng.shuffle(perm)
    got = helpers.gpu_sign_vote(w, [views[p] for p in perm])
    assert np.ascontiguousarray(got["sigs"]).tobytes() == np.ascontiguousarray(base["sigs"][:, perm]).tobytes()
    assert (got["status"] == base["status"]).all()
    for c in range(len(base["bitmap"])):
        b0 = int(base["bitmap"][c])
        assert int(got["bitmap"][c]) == sum(((b0 >> perm[j]) & 1) << j for j in range(w.R))
    inv = {p: j for j, p in enumerate(perm)}
    assert got["outliers"] == sorted((c, inv[r]) for c, r in base["outliers"])


def test_a_fault_held_by_the_majority_blames_the_clean_minority_and_half_is_undecided():
    w = inputs.workload(2, "clean", 1 / 64)
    _, views = inputs.generate(w, "cuda")          # R = 4
    el = 4321
    chunk = (2 * el) // w.chunk_bytes
    flip = lambda reps: [inputs.Patch(r, 0, el, "xor", 1 << 3) for r in reps]
    old = inputs.apply_patches(views, w.specs, flip([0, 1, 3]))
    got = helpers.gpu_sign_vote(w, views)
    assert got["outliers"] == [(chunk, 2)] and got["undecided"] == []       # indistinguishable from "2 is faulty"
    inputs.revert_patches(views, w.specs, flip([0, 1, 3]), old)
    old = inputs.apply_patches(views, w.specs, flip([1, 2]))
    got = helpers.gpu_sign_vote(w, views)
    assert got["outliers"] == [] and got["undecided"] == [chunk] and int(got["bitmap"][chunk]) == 0
    inputs.revert_patches(views, w.specs, flip([1, 2]), old)
    old = inputs.apply_patches(views, w.specs, flip([0, 1, 2, 3]))            # common-mode corruption is invisible
    got = helpers.gpu_sign_vote(w, views)
    assert got["outliers"] == [] and got["undecided"] == []
    inputs.revert_patches(views, w.specs, flip([0, 1, 2, 3]), old)
    assert helpers.gpu_sign_vote(w, views)["outliers"] == []


@pytest.mark.parametrize("dtype", ["f32", "bf16", "i64", "u8"])
def test_every_bit_of_an_element_is_seen(dtype):
    """Flip each bit of one element in turn: every flip is reported at exactly its
    (chunk, replica), and all flipped hashes differ from each other."""
    es = inputs.DTYPE_BYTES[dtype]
    dist = {"u8": "bytes", "i64": "randint40"}.get(dtype, "normal")
    spec = inputs.TensorSpec("x", (50_000 // es,), dtype, dist, 0.02)
    w = inputs.Workload("bits", 0, "x", 3, 8192, [spec], 12)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    el = 20_000 // es
    chunk = (el * es) // 8192
    seen = set()
    for bit in range(8 * es):
        p = [inputs.Patch(1, 0, el, "xor", 1 << bit)]
        old = inputs.apply_patches(views, w.specs, p)
        plan.sign_and_vote()
        got = plan.fetch()
        assert got["outliers"] == [(chunk, 1)], bit
        seen.add(int(got["sigs"]["hash"][chunk, 1]))
        inputs.revert_patches(views, w.specs, p, old)
    assert len(seen) == 8 * es
    plan.sign_and_vote()
    assert plan.fetch()["outliers"] == []
    helpers.assert_guards(plan)
    plan.close()
