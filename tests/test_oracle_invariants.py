"""End-to-end invariants of the oracle pipeline (chunk, sign, vote) on
scaled-down copies of the five benchmark workloads."""
import numpy as np
import pytest

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

SMALL = {1: 1 / 8, 2: 1 / 64, 3: 1 / 4096, 4: 1 / 2048, 5: 1 / 200}


def test_chunk_counts_of_the_full_size_workloads():
    # chunk geometry only: no data is generated
    want = {1: (1, 64), 2: (1, 48), 3: (224, 3712), 4: (3, 717)}
    for cfg, (T, C) in want.items():
        w = inputs.workload(cfg)
        ch = orc.chunk_table(helpers.oracle_tensor_table(w, [0] * len(w.specs)), w.chunk_bytes)
        assert (len(w.specs), len(ch)) == (T, C)
    w4 = inputs.workload(4)
    ch = orc.chunk_table(helpers.oracle_tensor_table(w4, [0] * 3), w4.chunk_bytes)
    last = ch[ch["tensor"] == 2][-1]
    assert int(last["nbytes"]) == 7_022_592 and int(last["index_in_tensor"]) == 238
    w3 = inputs.workload(3)
    assert w3.bytes_per_replica == 15_569_256_448
    w5 = inputs.workload(5)
    assert len(w5.specs) == 10_000
    assert all(256 <= s.nbytes + 8 and s.nbytes <= 4 << 20 and s.nbytes % 8 == 0 for s in w5.specs)
    with pytest.raises(ValueError):
        orc.chunk_table(helpers.oracle_tensor_table(w4, [0] * 3), 1000)   # not a multiple of 512


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_identical_replicas_have_no_outliers(cfg):
    w = inputs.workload(cfg, "clean", SMALL[cfg])
    _, views = inputs.generate(w)
    sigs, chunks = helpers.oracle_sign_all(w, views)
    out = orc.vote(sigs)
    assert out["outliers"] == [] and out["undecided"] == []
    assert out["counts"][1] == len(chunks) and (out["status"] == orc.AGREE).all()
    rep = orc.certify(sigs)["report"]
    assert rep["verdict"] == 0 and rep["certificate"] != 0


@pytest.mark.parametrize("cfg,case", [(1, "default"), (2, "mantissa"), (2, "split22"),
                                      (2, "split211"), (3, "default"), (4, "default"),
                                      (5, "default")])
def test_injected_faults_are_localised_exactly(cfg, case):
    w = inputs.workload(cfg, case, SMALL[cfg])
    _, views = inputs.generate(w)
    sigs, chunks = helpers.oracle_sign_all(w, views)
    want_out, want_und = helpers.expected_from_patches(w, chunks)
    out = orc.vote(sigs)
    assert out["outliers"] == want_out and out["undecided"] == want_und
    assert len(want_out) + len(want_und) >= 1
    if cfg == 2 and case.startswith("split"):
        assert want_out == [] and len(want_und) == 1
        assert int(out["bitmap"][want_und[0]]) == 0
    if cfg == 3:
        assert {r for _, r in want_out} == {5} and len(want_out) == 3
        nan_patch = [p for p in w.patches if p.op == "set"][0]
        c = helpers.chunk_of(chunks, nan_patch.tensor, nan_patch.element * 2)
        assert sigs[c, 5]["nan_count"] == 1 and sigs[c, 0]["nan_count"] == 0
        assert np.isfinite(sigs[c, 5]["sum"]) and np.isfinite(sigs[c, 5]["sumsq"])
    if cfg == 4:
        rep = orc.certify(sigs)
        bad = w.patches[0].replica
        assert rep["report"]["verdict"] == 1
        assert rep["report"]["replica_union_bitmap"] == 1 << bad


def test_fault_then_repair_is_clean_again():
    w = inputs.workload(1, "default", SMALL[1])
    _, views = inputs.generate(inputs.workload(1, "clean", SMALL[1]))
    clean, _ = helpers.oracle_sign_all(w, views)
    old = inputs.apply_patches(views, w.specs, w.patches)
    faulty, chunks = helpers.oracle_sign_all(w, views)
    inputs.revert_patches(views, w.specs, w.patches, old)
    again, _ = helpers.oracle_sign_all(w, views)
    assert orc.vote(clean)["outliers"] == [] and orc.vote(again)["outliers"] == []
    assert orc.vote(faulty)["outliers"] == helpers.expected_from_patches(w, chunks)[0]
    assert (clean["hash"] == again["hash"]).all()


def test_fault_held_by_a_majority_blames_the_clean_minority():
    w = inputs.workload(2, "clean", SMALL[2])
    _, views = inputs.generate(w)
    p = [inputs.Patch(r, 0, 1234, "xor", 4) for r in (0, 1, 3)]
    inputs.apply_patches(views, w.specs, p)
    sigs, chunks = helpers.oracle_sign_all(w, views)
    assert orc.vote(sigs)["outliers"] == [(helpers.chunk_of(chunks, 0, 2468), 2)]


def test_chunk_size_changes_granularity_not_the_faulty_location():
    w = inputs.workload(4, "default", SMALL[4])
    _, views = inputs.generate(w)
    for cb in (512, 4096, 64 << 10, 16 << 20):
        sigs, chunks = helpers.oracle_sign_all(w, views, chunk_bytes=cb)
        out = orc.vote(sigs)
        want = sorted({(helpers.chunk_of(chunks, p.tensor, 4 * p.element), p.replica)
                       for p in w.patches})
        assert out["outliers"] == want and out["undecided"] == []


def test_tensor_rollup_flags_the_tensor_of_a_faulty_chunk():
    w = inputs.workload(5, "default", SMALL[5])
    _, views = inputs.generate(w)
    sigs, chunks = helpers.oracle_sign_all(w, views)
    bad_tensors = {(p.tensor, p.replica) for p in w.patches}
    for t in range(len(w.specs)):
        sel = np.nonzero(chunks["tensor"] == t)[0]
        roll = [orc.rollup(sigs["hash"][sel, r]) for r in range(w.R)]
        differing = {(t, r) for r in range(w.R) if roll[r] != max(set(roll), key=roll.count)}
        assert differing == {(tt, r) for tt, r in bad_tensors if tt == t}


def test_threaded_driver_matches_single_thread():
    w = inputs.workload(5, "default", SMALL[5])
    _, views = inputs.generate(w)
    a, _ = helpers.oracle_sign_all(w, views, nthreads=1)
    b, _ = helpers.oracle_sign_all(w, views, nthreads=5)
    assert a.tobytes() == b.tobytes()
