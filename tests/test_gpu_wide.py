"""Groups wider than 64 peers and the one-replica-per-GPU form: the strided,
multi-word vote against its oracle, and per-replica signing + a gathered
(rank-major) record table against the fused single-GPU path."""
import numpy as np
import pytest
import torch

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def _vote_wide(sig_table, R, C, cs, rs, caps=None):
    from paper_2608_11034_b200 import binding as B
    W = (R + 63) // 64
    ocap, ucap = caps or (C * R, C)
    d_sigs = torch.from_numpy(np.ascontiguousarray(sig_table).view(np.uint8).reshape(-1)).cuda()
    d_status = torch.empty(C, dtype=torch.uint8, device="cuda")
    d_bitmap = torch.empty(C * W, dtype=torch.int64, device="cuda")
    d_out = torch.full((max(ocap, 1) * 16,), 0xEE, dtype=torch.uint8, device="cuda")
    d_und = torch.empty(max(ucap, 1), dtype=torch.int64, device="cuda")
    d_counts = torch.empty(6, dtype=torch.int64, device="cuda")
    B.scout_consensus_vote_wide(R, C, d_sigs.data_ptr(), cs, rs, d_status.data_ptr(), d_bitmap.data_ptr(),
                                d_out.data_ptr(), ocap, d_und.data_ptr(), ucap, d_counts.data_ptr(),
                                torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    counts = [int(x) for x in d_counts.cpu().numpy()]
    outl = d_out.cpu().numpy().view(B.OUTLIER_DTYPE)[:min(counts[4], ocap)]
    return dict(status=d_status.cpu().numpy(),
                bitmap=d_bitmap.cpu().numpy().view(np.uint64).reshape(C, W), counts=counts,
                outliers=sorted((int(o["chunk"]), int(o["replica"])) for o in outl),
                undecided=sorted(int(x) for x in d_und.cpu().numpy()[:min(counts[5], ucap)]),
                raw_outliers=d_out.cpu().numpy())


@pytest.mark.parametrize("R", [2, 3, 31, 64, 65, 100, 128, 192, 333, 1024])
def test_wide_vote_matches_the_oracle_in_both_layouts(R):
    rng = np.random.default_rng(R)
    C = 200 if R <= 192 else 40
    sigs = np.zeros((C, R), dtype=orc.SIG_DTYPE)
    alphabet = rng.integers(1, 2**63, size=4, dtype=np.uint64)
    for c in range(C):
        kind = c % 5
        sigs["hash"][c] = alphabet[0]
        if kind == 1:
            sigs["hash"][c, rng.integers(0, R)] = alphabet[1]
        elif kind == 2:
            sigs["hash"][c, rng.choice(R, size=R // 2, replace=False)] = alphabet[2]      # exactly half
        elif kind == 3:
            k = min(R - 1, R // 2 + 1)
            sigs["hash"][c, rng.choice(R, size=k, replace=False)] = alphabet[3]           # a majority of faults
        elif kind == 4:
            sigs["hash"][c] = alphabet[rng.integers(0, 3, size=R)]
    for table, cs, rs in ((sigs, R, 1), (np.ascontiguousarray(sigs.T), 1, C)):
        want = orc.vote_wide(table, R, C, cs, rs)
        got = _vote_wide(table, R, C, cs, rs)
        assert got["counts"] == want["counts"]
        assert (got["status"] == want["status"]).all()
        assert (got["bitmap"] == want["bitmap"]).all()
        assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"]
    cut = _vote_wide(sigs, R, C, R, 1, caps=(2, 1))
    assert cut["counts"] == want["counts"]
    assert (cut["raw_outliers"][2 * 16:] == 0xEE).all()


def test_one_replica_per_plan_then_gathered_vote_equals_the_fused_path():
    """The multi-GPU form on one GPU: every replica is signed by its own
    single-replica plan into row r of a rank-major [R][C] table (what an AllGather
    of per-rank records yields), then voted with strides (1, C)."""
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(5, "default", 1 / 200)
    _, views = inputs.generate(w, "cuda")
    fused = helpers.gpu_sign_vote(w, views)
    C = len(fused["status"])
    table = torch.empty(w.R * C * 32, dtype=torch.uint8, device="cuda")
    tt = B.make_tensor_table(w.specs, helpers.shape_tags(w))
    s = torch.cuda.current_stream().cuda_stream
    for r in range(w.R):
        plan = B.scout_plan_create(1, tt, w.chunk_bytes)
        assert B.scout_plan_num_chunks(plan) == C
        B.scout_plan_bind(plan, [v.data_ptr() for v in views[r]])
        B.scout_sign_chunks(plan, s, table.data_ptr() + r * C * 32)
        torch.cuda.synchronize()
        with pytest.raises(B.ScoutError):             # a singleton has nothing to vote on
            B.scout_certify(plan, s)
        B.scout_plan_destroy(plan)
    gathered = table.cpu().numpy().view(B.SIG_DTYPE).reshape(w.R, C)
    assert gathered.T.tobytes() == np.ascontiguousarray(fused["sigs"]).tobytes()    # same records, bit for bit
    got = _vote_wide(gathered, w.R, C, 1, C)
    assert got["outliers"] == fused["outliers"] and got["undecided"] == fused["undecided"]
    assert (got["status"] == fused["status"]).all()
    assert (got["bitmap"][:, 0] == fused["bitmap"]).all()
    assert got["counts"] == fused["counts"]


def test_signing_more_than_64_replicas():
    from paper_2608_11034_b200 import binding as B
    R = 100
    spec = inputs.TensorSpec("x", (30_000,), "f32", "normal", 1.0)
    w = inputs.Workload("wide", 0, "x", R, 8192, [spec], 5)
    w.patches = [inputs.Patch(77, 0, 12_345, "xor", 1 << 20), inputs.Patch(3, 0, 5, "xor", 1)]
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    plan.sign()
    torch.cuda.synchronize()
    sigs = plan.d_sigs.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, R)
    host = [[v.cpu() for v in rep] for rep in views[:4]] + [None] * (R - 4)
    osig = orc.sign_chunk(inputs.to_numpy_bytes(views[77][0])[8192 * 6:8192 * 7], orc.DT_F32, 6,
                          helpers.shape_tags(w)[0])
    assert int(sigs["hash"][6, 77]) == int(osig["hash"])
    got = _vote_wide(sigs, R, plan.C, R, 1)
    want = orc.vote_wide(sigs, R, plan.C, R, 1)
    assert got["outliers"] == want["outliers"] == [(0, 3), (6, 77)]
    with pytest.raises(B.ScoutError) as e:
        plan.certify()
    assert e.value.code == B.ERR_UNSUPPORTED
    helpers.assert_guards(plan)
    plan.close()
