"""The one-launch forms of scout_sign_chunks and scout_certify against the oracle and
against the one-kernel-per-stage form.  Form 1 (tickets): the warp that stores a
chunk's last tile record finalises, votes and folds it; nobody waits.  Form 2
(clusters): a thread-block cluster of R CTAs per chunk, records in shared memory, the
vote through distributed shared memory.  Covered here is what only these forms have:
state that must return to zero between launches, a certificate chain folded by many
different warps, lists longer than the report block's head, the launch/collect pair,
chunks taken several at a time, and the choice the library makes by default."""
import numpy as np
import pytest
import torch

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def _oracle_certify(w, views, chunk_bytes=None):
    host = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host, chunk_bytes=chunk_bytes)
    return orc.certify(osigs), osigs, chunks, host


@pytest.mark.parametrize("form", [1, 2])
@pytest.mark.parametrize("cfg,case,scale,chunk_bytes", [
    (1, "default", 1 / 4, None), (2, "split22", 1 / 32, None), (2, "split211", 1 / 32, 65536),
    (3, "default", 1 / 2048, 65536), (4, "default", 1 / 512, 8192),       # 8 KiB chunks: 2,862 chunks
    (4, "default", 1 / 512, 512),                                          # one-row chunks, 16 per cluster pass
    (5, "default", 1 / 100, 4096), (5, "clean", 1 / 100, None)])
def test_certify_in_one_launch_equals_the_oracle_and_the_staged_form(cfg, case, scale, chunk_bytes, form):
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(cfg, case, scale)
    if form == 2 and w.R > 8:
        w.R = 8                                              # the cluster form takes at most 8 replicas
        w.patches = [p for p in w.patches if p.replica < 8]
    _, views = inputs.generate(w, "cuda")
    want, osigs, chunks, host = _oracle_certify(w, views, chunk_bytes)
    plan = helpers.gpu_plan(w, chunk_bytes=chunk_bytes)
    assert B.scout_plan_get(plan.handle, "fused") == -1      # the default: one launch where it is faster
    if form == 2:
        assert B.scout_plan_get(plan.handle, "cluster_ok") == 1
    B.scout_plan_set(plan.handle, "fused", form)
    assert B.scout_plan_get(plan.handle, "certify_kernels") == 1
    assert B.scout_plan_get(plan.handle, "certify_form") == form
    plan.bind(views)
    for round_ in range(3):                      # the device state must be back to zero every time
        got = plan.certify()
        assert got["report"] == want["report"], round_
        assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"]
        assert B.scout_plan_replica_bad_counts(plan.handle, w.R) == want["replica_bad"]
    # the records that certify run left in the plan: every hash enters the tensor roll-ups
    d_sigs, _, _ = B.scout_plan_results(plan.handle)
    d_roll = torch.empty(len(w.specs) * w.R, dtype=torch.int64, device="cuda")
    B.scout_rollup_tensors(plan.handle, d_sigs, d_roll.data_ptr(), torch.cuda.current_stream().cuda_stream)
    roll = d_roll.cpu().numpy().view(np.uint64).reshape(len(w.specs), w.R)
    cb = w.chunk_bytes if chunk_bytes is None else chunk_bytes
    for t in range(len(w.specs)):
        sel = np.nonzero(chunks["tensor"] == t)[0]
        for r in range(w.R):
            assert int(roll[t, r]) == orc.rollup(osigs["hash"][sel, r])
    # and the one-launch sign (scan + finalise) on the same plan: full records
    plan.sign()
    torch.cuda.synchronize()
    gs = plan.d_sigs.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, w.R)
    helpers.assert_sigs_match(gs, osigs, helpers.chunk_abs_sums(w, host, chunks))
    # the staged form on the same plan gives the same report, and the one-launch form still works after it
    B.scout_plan_set(plan.handle, "fused", 0)
    assert B.scout_plan_get(plan.handle, "certify_kernels") == 4
    staged = plan.certify()
    assert staged["report"] == want["report"] and staged["outliers"] == want["outliers"]
    B.scout_plan_set(plan.handle, "fused", form)
    again = plan.certify()
    assert again["report"] == want["report"] and again["outliers"] == want["outliers"]
    helpers.assert_guards(plan)
    plan.close()


@pytest.mark.parametrize("variant", ["fused", "cluster"])
def test_lists_longer_than_the_report_head_and_truncation(variant):
    """More than 64 outlier pairs and more than 64 undecided chunks: the tail of both lists
    comes from the device lists, and capacities below the totals report truncation."""
    from paper_2608_11034_b200 import binding as B
    spec = inputs.TensorSpec("x", (400 * 1024,), "f32", "normal", 1.0)          # 400 chunks of 4 KiB
    w = inputs.Workload("many_faults", 0, "x", 4, 4096, [spec], 21)
    per = 1024
    w.patches = [inputs.Patch(1, 0, c * per + 7, "xor", 1 << 3) for c in range(0, 200, 2)]          # 100 attributed
    w.patches += [inputs.Patch(r, 0, c * per + 9, "xor", 1 << 5) for c in range(201, 400, 2) for r in (0, 2)]  # 2-vs-2
    _, views = inputs.generate(w, "cuda")
    want, _, _, _ = _oracle_certify(w, views)
    assert want["report"]["n_outliers"] == 100 and want["report"]["n_undecided"] == 100
    plan = helpers.gpu_plan(w, variant=variant)
    plan.bind(views)
    got = plan.certify()
    assert got["report"] == want["report"] and got["report"]["verdict"] == B.UNDECIDED
    assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"]
    cut = plan.certify(outlier_cap=70, undecided_cap=3)
    assert cut["rc"] == B.ERR_TRUNCATED and cut["report"] == want["report"]
    assert len(cut["outliers"]) == 70 and set(cut["outliers"]) <= set(want["outliers"])
    assert len(cut["undecided"]) == 3 and set(cut["undecided"]) <= set(want["undecided"])
    full = plan.certify()
    assert full["outliers"] == want["outliers"] and full["undecided"] == want["undecided"]
    helpers.assert_guards(plan)
    plan.close()


def test_launch_and_collect():
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(1, "default", 1 / 2)
    _, views = inputs.generate(w, "cuda")
    want, _, _, _ = _oracle_certify(w, views)
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    with pytest.raises(B.ScoutError):                      # nothing was launched
        plan.certify_collect()
    side = torch.cuda.Stream()
    for fused in (2, 1, 0):
        B.scout_plan_set(plan.handle, "fused", fused)
        plan.certify_launch(stream=side.cuda_stream)
        with pytest.raises(B.ScoutError):                  # one run in flight per plan
            plan.certify_launch(stream=side.cuda_stream)
        with pytest.raises(B.ScoutError):
            plan.certify()
        got = plan.certify_collect()
        assert got["report"] == want["report"] and got["outliers"] == want["outliers"]
        with pytest.raises(B.ScoutError):                  # already collected
            plan.certify_collect()
    helpers.assert_guards(plan)
    plan.close()


def test_sign_in_one_launch_with_one_replica_and_with_sixty_four():
    """R = 1 (the local step of the distributed form) and R = 64 (the widest one-word bitmap)."""
    from paper_2608_11034_b200 import binding as B
    spec = inputs.TensorSpec("x", (100_003,), "bf16", "normal", 0.02)
    for R in (1, 64):
        w = inputs.Workload("r%d" % R, 0, "x", R, 8192, [spec], 5)
        if R == 64:
            w.patches = [inputs.Patch(63, 0, 77, "xor", 1), inputs.Patch(31, 0, 50_000, "xor", 2),
                         inputs.Patch(32, 0, 50_001, "xor", 4)]
        _, views = inputs.generate(w, "cuda")
        host = [[v.cpu() for v in rep] for rep in views]
        osigs, chunks = helpers.oracle_sign_all(w, host)
        plan = helpers.gpu_plan(w, variant="fused")
        assert B.scout_plan_get(plan.handle, "sign_kernels") == 1
        plan.bind(views)
        plan.sign()
        torch.cuda.synchronize()
        gs = plan.d_sigs.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, R)
        helpers.assert_sigs_match(gs, osigs, helpers.chunk_abs_sums(w, host, chunks))
        if R == 64:
            got = plan.certify()
            want = orc.certify(osigs)
            assert got["report"] == want["report"] and got["outliers"] == want["outliers"]
            assert got["report"]["replica_union_bitmap"] == (1 << 63) | (1 << 31) | (1 << 32)
        helpers.assert_guards(plan)
        plan.close()


def test_cluster_form_with_one_to_eight_replicas_and_the_limits():
    """Every cluster size, mixed dtypes (tensor boundaries inside a cluster pass), and the
    shapes the form refuses."""
    from paper_2608_11034_b200 import binding as B
    specs = [inputs.TensorSpec("a", (300_001,), "f32", "normal", 0.02),
             inputs.TensorSpec("b", (123_457,), "bf16", "normal", 0.02),
             inputs.TensorSpec("c", (77_001,), "i64", "randint40", 0.0)]
    for R, chunk_bytes in ((1, 65536), (2, 65536), (3, 2048), (4, 1536), (5, 8192), (6, 512), (7, 16384), (8, 40960)):
        w = inputs.Workload("mix", 0, "x", R, chunk_bytes, specs, 100 + R)
        if R >= 3:
            w.patches = [inputs.Patch(R - 1, 1, 5000, "xor", 4), inputs.Patch(0, 2, 77_000, "xor", 1 << 40)]
        _, views = inputs.generate(w, "cuda")
        host = [[v.cpu() for v in rep] for rep in views]
        osigs, chunks = helpers.oracle_sign_all(w, host)
        plan = helpers.gpu_plan(w, variant="cluster")
        plan.bind(views)
        plan.sign()
        torch.cuda.synchronize()
        gs = plan.d_sigs.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, R)
        helpers.assert_sigs_match(gs, osigs, helpers.chunk_abs_sums(w, host, chunks))
        if R >= 2:
            want = orc.certify(osigs)
            for _ in range(2):
                got = plan.certify()
                assert got["report"] == want["report"]
                assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"]
        helpers.assert_guards(plan)
        plan.close()
    # nine replicas, or more than 512 tiles in a chunk: the form is refused, the others still run
    spec = inputs.TensorSpec("x", (1 << 20,), "f32", "normal", 1.0)
    for R, chunk_bytes, tile in ((9, 65536, None), (3, 2 << 20, 2048)):
        w = inputs.Workload("no", 0, "x", R, chunk_bytes, [spec], 3)
        plan = helpers.gpu_plan(w, tile_bytes=tile)
        assert B.scout_plan_get(plan.handle, "cluster_ok") == 0
        with pytest.raises(B.ScoutError):
            B.scout_plan_set(plan.handle, "fused", 2)
        assert B.scout_plan_get(plan.handle, "certify_form") in (0, 1)
        plan.close()


def test_the_default_picks_the_form_by_shape():
    """Key "fused" = -1: clusters for small plans of few-tile chunks and R <= 8, tickets for other
    plans of few-tile chunks up to 16 MiB, one kernel per stage otherwise; scout_sign_chunks always per stage."""
    from paper_2608_11034_b200 import binding as B
    def form(R, numel, chunk_bytes, dtype="f32"):
        w = inputs.Workload("p", 0, "x", R, chunk_bytes, [inputs.TensorSpec("x", (numel,), dtype, "normal", 1.0)], 3)
        plan = helpers.gpu_plan(w)
        f = (B.scout_plan_get(plan.handle, "certify_form"), B.scout_plan_get(plan.handle, "sign_form"))
        plan.close()
        return f
    assert form(3, 1 << 20, 65536) == (2, 0)            # 12.6 MB, 16 tiles per chunk
    assert form(4, 25_165_824, 1 << 20, "bf16") == (2, 0)   # 201 MB in 1 MiB chunks, 64 tiles per chunk
    assert form(16, 1 << 18, 65536) == (1, 0)           # 16 replicas of 1 MiB (16 MiB in all): no cluster, tickets
    assert form(3, 1 << 20, 4 << 20) == (0, 0)          # one chunk of 1,024 tiles, 12.6 MB: per stage
    assert form(3, 16 << 20, 4 << 20) == (0, 0)         # 201 MB in 4 MiB chunks (256 tiles each): per stage
    assert form(3, 2 << 20, 2048) == (0, 0)             # 4,096 chunks: the chain decides, per stage


def test_several_plans_in_flight_on_different_streams():
    """Six plans of different shapes, each in the form the library picks for it (clusters,
    tickets, one kernel per stage), launched on six streams before any is collected, 300 times
    over: every report equals the plan's own staged result (no state is shared between plans,
    and every launch leaves its plan's device state ready for the next)."""
    from paper_2608_11034_b200 import binding as B
    ws = [inputs.workload(1, "default", 1.0), inputs.workload(2, "mantissa", 0.25), inputs.workload(3, "default", 0.002),
          inputs.workload(1, "default", 0.5), inputs.workload(5, "default", 0.005), inputs.workload(4, "default", 0.002)]
    plans, refs, streams, keep = [], [], [], []
    for w in ws:
        _, views = inputs.generate(w, "cuda")
        keep.append(views)
        p = helpers.gpu_plan(w)
        p.bind(views)
        B.scout_plan_set(p.handle, "fused", 0)
        refs.append(p.certify())
        B.scout_plan_set(p.handle, "fused", -1)
        plans.append(p)
        streams.append(torch.cuda.Stream())
    assert {B.scout_plan_get(p.handle, "certify_form") for p in plans} == {0, 1, 2}
    for _ in range(300):
        for p, s in zip(plans, streams):
            p.certify_launch(stream=s.cuda_stream)
        for p, ref in zip(plans, refs):
            got = p.certify_collect()
            assert got["report"] == ref["report"] and got["outliers"] == ref["outliers"]
    for p in plans:
        helpers.assert_guards(p)
        p.close()
