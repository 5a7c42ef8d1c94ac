"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  Configs 1 and 2 are compared chunk by chunk; for configs 3, 4 and 5 the
oracle signs a sample of (chunk, replica) pairs (every faulty chunk, the first
and last chunks, ragged tails, random ones) and the vote is checked against
what the injected patches imply for EVERY chunk."""
import gc
import random

import numpy as np
import pytest
import torch

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def _free():
    gc.collect()
    torch.cuda.empty_cache()


def _need(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip(f"needs {gb} GB of free device memory, {free / 1e9:.0f} GB available")


def _oracle_chunk(w, views, chunks, c, r, tags):
    ch = chunks[c]
    t = int(ch["tensor"])
    lo, n = int(ch["byte_offset"]), int(ch["nbytes"])
    b = views[r][t].view(-1).view(torch.uint8)[lo:lo + n].cpu().numpy()
    sig = orc.sign_chunk(b, helpers.ORC_CODE[w.specs[t].dtype], int(ch["index_in_tensor"]), tags[t])
    import defn
    x = np.abs(defn.values_f64(b.tobytes(), w.specs[t].dtype)) if w.specs[t].dtype != "u8" else np.zeros(1)
    return sig, float(x[np.isfinite(x)].sum())


def _check_sampled(w, views, sigs, chunks, pairs):
    tags = helpers.shape_tags(w)
    for c, r in pairs:
        o, abs_sum = _oracle_chunk(w, views, chunks, c, r, tags)
        g = sigs[c, r]
        assert int(g["hash"]) == int(o["hash"]), (c, r)
        assert (g["nan_count"], g["inf_count"]) == (o["nan_count"], o["inf_count"]), (c, r)
        assert abs(g["sum"] - o["sum"]) <= helpers.REL_TOL * abs_sum, (c, r)
        assert abs(g["sumsq"] - o["sumsq"]) <= helpers.REL_TOL * abs(o["sumsq"]), (c, r)


def _sample_pairs(w, chunks, want_out, n_random, seed):
    rng = random.Random(seed)
    C = len(chunks)
    pairs = set()
    for c, r in want_out:
        pairs.add((c, r))
        pairs.add((c, (r + 1) % w.R))
    pairs |= {(0, 0), (C - 1, w.R - 1)}
    ragged = [c for c in range(C) if int(chunks[c]["nbytes"]) != w.chunk_bytes]
    for c in rng.sample(ragged, min(4, len(ragged))):
        pairs.add((c, rng.randrange(w.R)))
    for _ in range(n_random):
        pairs.add((rng.randrange(C), rng.randrange(w.R)))
    return sorted(pairs)


@pytest.mark.parametrize("cfg,case", [(1, "default"), (1, "clean"), (2, "clean"), (2, "mantissa"),
                                      (2, "split22"), (2, "split211")])
def test_configs_1_and_2_every_chunk(cfg, case):
    w = inputs.workload(cfg, case)
    _, views = inputs.generate(w, "cuda")
    gpu = helpers.gpu_sign_vote(w, views)
    host = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host, nthreads=8)
    helpers.assert_sigs_match(gpu["sigs"], osigs, helpers.chunk_abs_sums(w, host, chunks))
    ov = orc.vote(osigs)
    want_out, want_und = helpers.expected_from_patches(w, chunks)
    assert gpu["outliers"] == ov["outliers"] == want_out
    assert gpu["undecided"] == ov["undecided"] == want_und
    assert gpu["counts"] == ov["counts"]
    assert (gpu["status"] == ov["status"]).all() and (gpu["bitmap"] == ov["bitmap"]).all()
    del views
    _free()


def test_config_4_certify_full_size():
    from paper_2608_11034_b200 import binding
    _free()
    _need(40)
    w = inputs.workload(4)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    rep = plan.certify()
    chunks = plan.chunk_table()
    assert len(chunks) == 717 and int(chunks[-1]["nbytes"]) == 7_022_592
    want_out, want_und = helpers.expected_from_patches(w, chunks)
    bad = w.patches[0].replica
    assert rep["outliers"] == want_out and rep["undecided"] == want_und == []
    r = rep["report"]
    assert r["verdict"] == binding.VERDICT_ATTRIBUTED and r["replica_union_bitmap"] == 1 << bad
    assert (r["n_chunks"], r["n_attributed"], r["n_agree"]) == (717, len(want_out), 717 - len(want_out))
    assert binding.scout_plan_replica_bad_counts(plan.handle, w.R)[bad] == len(want_out)
    plan.sign()
    torch.cuda.synchronize()
    sigs = plan.d_sigs.cpu().numpy().view(binding.SIG_DTYPE).reshape(plan.C, w.R)
    # every chunk that carries no patch must have identical hashes in all replicas
    clean = np.ones(plan.C, bool)
    clean[[c for c, _ in want_out]] = False
    assert (sigs["hash"][clean] == sigs["hash"][clean][:, :1]).all()
    _check_sampled(w, views, sigs, chunks, _sample_pairs(w, chunks, want_out, 6, 4))
    # the certificate is the chain over the majority hashes: recompute it from the records
    maj = [int(sigs["hash"][c, (bad + 1) % w.R]) for c in range(plan.C)]
    import defn
    assert r["certificate"] == defn.certificate(maj)
    plan.close()
    del views
    _free()


def test_config_5_full_size():
    from paper_2608_11034_b200 import binding
    _free()
    _need(75)
    w = inputs.workload(5)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    plan.sign_and_vote()
    got = plan.fetch()
    chunks = plan.chunk_table()
    want_out, want_und = helpers.expected_from_patches(w, chunks)
    assert len(want_out) == 2 and got["outliers"] == want_out and got["undecided"] == want_und == []
    assert got["counts"][0] == plan.C and got["counts"][2] == 2
    sigs = got["sigs"]
    clean = np.ones(plan.C, bool)
    clean[[c for c, _ in want_out]] = False
    assert (sigs["hash"][clean] == sigs["hash"][clean][:, :1]).all()
    _check_sampled(w, views, sigs, chunks, _sample_pairs(w, chunks, want_out, 40, 5))
    plan.close()
    del views
    _free()


def test_config_3_full_size():
    from paper_2608_11034_b200 import binding
    _free()
    _need(130)
    w = inputs.workload(3)
    assert w.bytes_per_replica * w.R == 124_554_051_584
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    plan.sign_and_vote()
    got = plan.fetch()
    chunks = plan.chunk_table()
    assert plan.C == 3712
    want_out, want_und = helpers.expected_from_patches(w, chunks)
    assert got["outliers"] == want_out and got["undecided"] == want_und == []
    assert len(want_out) == 3 and {r for _, r in want_out} == {5}
    sigs = got["sigs"]
    nan_patch = [p for p in w.patches if p.op == "set"][0]
    c_nan = helpers.chunk_of(chunks, nan_patch.tensor, 2 * nan_patch.element)
    assert sigs[c_nan, 5]["nan_count"] == 1 and int(sigs["nan_count"].sum()) == 1
    assert np.isfinite(sigs[c_nan, 5]["sum"]) and np.isfinite(sigs[c_nan, 5]["sumsq"])
    clean = np.ones(plan.C, bool)
    clean[[c for c, _ in want_out]] = False
    assert (sigs["hash"][clean] == sigs["hash"][clean][:, :1]).all()
    _check_sampled(w, views, sigs, chunks, _sample_pairs(w, chunks, want_out, 8, 3))
    plan.close()
    del views
    _free()


def test_largest_chunk_size_one_gib():
    """chunk_bytes at its maximum (1 GiB): 32,768 tiles per chunk go through the
    finaliser's strided combine; the second chunk of each tensor is one ragged row."""
    from paper_2608_11034_b200 import binding
    _free()
    _need(6)
    n = (1 << 30) + 516
    w = inputs.Workload("one_gib_chunk", 0, "x", 2, 1 << 30,
                        [inputs.TensorSpec("blob", (n,), "u8", "bytes"),
                         inputs.TensorSpec("grad", ((1 << 28) + 129,), "f32", "normal", 0.02)], 99)
    w.patches = [inputs.Patch(1, 0, (1 << 30) - 1, "xor", 0x80), inputs.Patch(0, 1, 1 << 28, "xor", 1)]
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    plan.sign_and_vote()
    got = plan.fetch()
    chunks = plan.chunk_table()
    assert plan.C == 4 and [int(c["nbytes"]) for c in chunks] == [1 << 30, 516, 1 << 30, 516]
    # two replicas: a difference is detected but cannot be attributed (two-rank group)
    assert got["outliers"] == [] and got["undecided"] == [0, 3]
    assert list(got["status"]) == [binding.INCONCLUSIVE, binding.AGREE, binding.AGREE, binding.INCONCLUSIVE]
    _check_sampled(w, views, got["sigs"], chunks, [(0, 1), (1, 0), (2, 0), (3, 0), (3, 1)])
    plan.close()
    del views
    _free()
