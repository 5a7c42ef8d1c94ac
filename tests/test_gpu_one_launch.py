"""The one-launch forms of scout_sign_chunks and scout_certify (the warp that stores
a chunk's last tile record finalises, votes and folds it; nobody waits) against the
oracle and against the one-kernel-per-stage form, including what only the one-launch
form has: state that must return to zero between launches, a certificate chain
folded by many different warps, lists longer than the report block's head, and the
launch/collect pair."""
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


@pytest.mark.parametrize("cfg,case,scale,chunk_bytes", [
    (1, "default", 1 / 4, None), (2, "split22", 1 / 32, None), (2, "split211", 1 / 32, 65536),
    (3, "default", 1 / 2048, 65536), (4, "default", 1 / 512, 8192),       # 8 KiB chunks: 2,862 chunks
    (5, "default", 1 / 100, 4096), (5, "clean", 1 / 100, None)])
def test_certify_in_one_launch_equals_the_oracle_and_the_staged_form(cfg, case, scale, chunk_bytes):
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(cfg, case, scale)
    _, views = inputs.generate(w, "cuda")
    want, osigs, chunks, host = _oracle_certify(w, views, chunk_bytes)
    plan = helpers.gpu_plan(w, chunk_bytes=chunk_bytes)
    assert B.scout_plan_get(plan.handle, "fused") == -1      # the default: one launch where it is faster
    B.scout_plan_set(plan.handle, "fused", 1)
    assert B.scout_plan_get(plan.handle, "certify_kernels") == 1
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
    B.scout_plan_set(plan.handle, "fused", 1)
    again = plan.certify()
    assert again["report"] == want["report"] and again["outliers"] == want["outliers"]
    helpers.assert_guards(plan)
    plan.close()


def test_lists_longer_than_the_report_head_and_truncation():
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
    plan = helpers.gpu_plan(w, variant="fused")
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
    for fused in (1, 0):
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
