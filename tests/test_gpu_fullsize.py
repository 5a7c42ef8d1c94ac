"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  Configs 1 and 2 are compared chunk by chunk.  For configs 3, 4 and 5 the
oracle signs EVERY chunk of one whole replica (so a fold that is wrong in the
same way in all replicas cannot pass) plus a sample of (chunk, replica) pairs of
the other replicas (every faulty chunk, the first and last chunks, ragged tails,
random ones); the vote is checked against what the injected patches imply for
every chunk."""
import gc
import os
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


def _abs_sums_on_device(x, dtype, chunk_bytes):
    """sum |x| over the finite elements of each chunk of one tensor (plain torch on the
    tensor's own device): only the scale of the tolerance on the sums."""
    es = inputs.DTYPE_BYTES[dtype]
    per = chunk_bytes // es
    n_ch = (x.numel() + per - 1) // per
    out = torch.zeros(n_ch, dtype=torch.float64, device=x.device)
    if dtype == "u8":
        return out.cpu().numpy()
    flat = x.reshape(-1)
    step = max(1, (256 << 20) // chunk_bytes)          # chunks per slice: bounds the fp64 temporaries
    for c0 in range(0, n_ch, step):
        part = flat[c0 * per:(c0 + step) * per].to(torch.float64).abs()
        part = torch.where(torch.isfinite(part), part, torch.zeros_like(part))
        full = part.numel() // per
        if full:
            out[c0:c0 + full] = part[:full * per].view(full, per).sum(1)
        if part.numel() > full * per:
            out[c0 + full] = part[full * per:].sum()
    return out.cpu().numpy()


def _check_whole_replica(w, views, sigs, chunks, r):
    """Every chunk of replica r against the oracle (all host cores), tensors taken in
    groups of about 1 GiB so that host memory stays bounded."""
    tags = helpers.shape_tags(w)
    nthreads = os.cpu_count() or 4
    cb = w.chunk_bytes
    group, group_bytes, c0, checked = [], 0, 0, 0

    def flush():
        nonlocal group, group_bytes, c0, checked
        if not group:
            return
        tt = orc.make_tensor_table([(w.specs[t].nbytes, helpers.ORC_CODE[w.specs[t].dtype], tags[t])
                                    for t in group])
        arrays = [inputs.to_numpy_bytes(views[r][t]) for t in group]
        n_ch = sum((w.specs[t].nbytes + cb - 1) // cb for t in group)
        o = np.zeros((n_ch, 1), dtype=orc.SIG_DTYPE)
        orc.sign_replica(tt, arrays, cb, o, 0, nthreads)
        scale = np.concatenate([_abs_sums_on_device(views[r][t], w.specs[t].dtype, cb) for t in group])
        g = sigs[c0:c0 + n_ch, r]
        assert int(chunks["tensor"][c0]) == group[0] and int(chunks["tensor"][c0 + n_ch - 1]) == group[-1]
        helpers.assert_sigs_match(g.reshape(-1, 1), o, scale.reshape(-1, 1))
        c0 += n_ch
        checked += n_ch
        group, group_bytes = [], 0

    for t, s in enumerate(w.specs):
        group.append(t)
        group_bytes += s.nbytes
        if group_bytes >= (1 << 30):
            flush()
    flush()
    assert checked == len(chunks)


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


@pytest.mark.parametrize("cfg,case", [(1, "default"), (2, "mantissa"), (2, "split22"), (2, "split211")])
def test_configs_1_and_2_certify_in_the_default_form(cfg, case):
    """scout_certify as the library launches it by default on these plans (one kernel, a
    thread-block cluster per chunk): report, lists and every record against the oracle."""
    from paper_2608_11034_b200 import binding
    w = inputs.workload(cfg, case)
    _, views = inputs.generate(w, "cuda")
    host = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host, nthreads=8)
    want = orc.certify(osigs)
    plan = helpers.gpu_plan(w)
    assert binding.scout_plan_get(plan.handle, "certify_form") == 2
    assert binding.scout_plan_get(plan.handle, "certify_kernels") == 1
    plan.bind(views)
    for _ in range(2):
        got = plan.certify()
        assert got["report"] == want["report"]
        assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"]
    # the records that run left in the plan: their hashes enter the tensor roll-ups
    d_sigs, _, _ = binding.scout_plan_results(plan.handle)
    d_roll = torch.empty(len(w.specs) * w.R, dtype=torch.int64, device="cuda")
    binding.scout_rollup_tensors(plan.handle, d_sigs, d_roll.data_ptr(), torch.cuda.current_stream().cuda_stream)
    roll = d_roll.cpu().numpy().view(np.uint64).reshape(len(w.specs), w.R)
    for r in range(w.R):
        assert int(roll[0, r]) == orc.rollup(osigs["hash"][:, r])
    # and the same kernel as scout_sign_chunks: full records, sums included
    binding.scout_plan_set(plan.handle, "fused", 2)
    plan.sign()
    torch.cuda.synchronize()
    got_sigs = plan.d_sigs.cpu().numpy().view(binding.SIG_DTYPE).reshape(plan.C, w.R)
    helpers.assert_sigs_match(got_sigs, osigs, helpers.chunk_abs_sums(w, host, chunks))
    helpers.assert_guards(plan)
    plan.close()
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
    _check_whole_replica(w, views, sigs, chunks, bad)
    # the certificate is the chain over the majority hashes: recompute it from the records
    maj = [int(sigs["hash"][c, (bad + 1) % w.R]) for c in range(plan.C)]
    import defn
    assert r["certificate"] == defn.certificate(maj)
    helpers.assert_guards(plan)
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
    _check_whole_replica(w, views, sigs, chunks, want_out[0][1])
    helpers.assert_guards(plan)
    plan.close()
    del views
    _free()


def test_config_3_full_size():
    from paper_2608_11034_b200 import binding
    _free()
    _need(135)
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
    _check_whole_replica(w, views, sigs, chunks, 5)
    helpers.assert_guards(plan)
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
    helpers.assert_guards(plan)
    plan.close()
    del views
    _free()
