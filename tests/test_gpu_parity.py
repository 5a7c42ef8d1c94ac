"""Parity of the CUDA path (through the C ABI) with the CPU oracle: hashes,
counts, statuses, bitmaps and lists bit-exact; fp64 sums within 1e-12."""
import random

import numpy as np
import pytest
import torch

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu

SMALL = {1: 1 / 8, 2: 1 / 64, 3: 1 / 4096, 4: 1 / 2048, 5: 1 / 200}


def _binding():
    from paper_2608_11034_b200 import binding
    return binding


# direct loads with one kernel per stage, the same scan with the whole call as one launch, register
# prefetch, per-warp bulk-async ring, block-wide ring
VARIANTS = ["unfused", "fused", "cluster", 0, 1, 2, 4]   # "unfused": the default front end (1), one kernel per stage


def _compare_everything(w, views, chunk_bytes=None, tile_bytes=None, variant=None):
    gpu = helpers.gpu_sign_vote(w, views, chunk_bytes=chunk_bytes, tile_bytes=tile_bytes,
                                variant=variant)
    host_views = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host_views, chunk_bytes=chunk_bytes)
    helpers.assert_sigs_match(gpu["sigs"], osigs, helpers.chunk_abs_sums(w, host_views, chunks))
    ov = orc.vote(osigs)
    assert (gpu["status"] == ov["status"]).all()
    assert (gpu["bitmap"] == ov["bitmap"]).all()
    assert gpu["counts"] == ov["counts"]
    assert gpu["outliers"] == ov["outliers"] and gpu["undecided"] == ov["undecided"]
    return gpu, osigs, chunks


@pytest.mark.parametrize("cfg,case", [(1, "clean"), (1, "default"), (2, "clean"), (2, "mantissa"),
                                      (2, "split22"), (2, "split211"), (3, "default"),
                                      (4, "default"), (5, "default")])
@pytest.mark.parametrize("variant", VARIANTS)
def test_scaled_workloads(cfg, case, variant):
    w = inputs.workload(cfg, case, SMALL[cfg])
    _, views = inputs.generate(w, "cuda")
    gpu, _, chunks = _compare_everything(w, views, variant=variant)
    want_out, want_und = helpers.expected_from_patches(w, chunks)
    assert gpu["outliers"] == want_out and gpu["undecided"] == want_und


def _odd_workload(dtype, seed):
    """Sizes around every boundary: one element, a row +-1 element, a tile +-1,
    a chunk +-1 element, several chunks with a ragged tail."""
    es = inputs.DTYPE_BYTES[dtype]
    chunk = 8192
    sizes = [es, 16, 512 - es, 512, 512 + es, 2048 - es, 2048, 2048 + es, chunk - es, chunk,
             chunk + es, 3 * chunk + 512 + es, 5 * chunk - es, 40000 // es * es + es]
    if dtype == "u8":
        sizes += [1, 3, 5, 17, 515, 8191, 8193]
    dist = {"u8": "bytes", "i64": "randint40", "i32": "bytes"}.get(dtype, "normal")
    specs = [inputs.TensorSpec(f"t{i}", (n // es,), dtype, dist, 0.5) for i, n in enumerate(sizes)]
    if dtype == "i32":
        specs = [inputs.TensorSpec(s.name, s.shape, "i32", "randfull") for s in specs]
    return inputs.Workload(f"odd_{dtype}", 0, "odd", 3, chunk, specs, seed)


@pytest.mark.parametrize("dtype", ["u8", "f32", "bf16", "i64", "f16", "f64", "i32"])
@pytest.mark.parametrize("tile_bytes,variant", [(2048, "fused"), (4096, "fused"), (2048, "cluster"), (4096, "cluster"), (2048, "unfused"), (4096, "unfused"),
                                                (4096, 0), (8192, 0), (4096, 1), (8192, 1),
                                                (4096, 2), (8192, 2), (32768, 2), (4096, 4), (8192, 4), (32768, 4)])
def test_every_dtype_and_ragged_sizes(dtype, tile_bytes, variant):
    w = _odd_workload(dtype, 77)
    _, views = inputs.generate(w, "cuda")
    rng = random.Random(5)
    w.patches = [inputs.Patch(rng.randrange(3), t, rng.randrange(s.numel), "xor",
                              1 << rng.randrange(8 * inputs.DTYPE_BYTES[dtype]))
                 for t, s in enumerate(w.specs) if t % 2 == 0]
    inputs.apply_patches(views, w.specs, w.patches)
    _compare_everything(w, views, tile_bytes=tile_bytes, variant=variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_non_finite_elements(variant):
    w = inputs.workload(3, "clean", SMALL[3])
    _, views = inputs.generate(w, "cuda")
    n0 = w.specs[0].numel
    w.patches = [inputs.Patch(2, 0, 5, "set", 0x7FC0),            # NaN
                 inputs.Patch(2, 0, n0 - 1, "set", 0x7F80),       # +Inf in the last element
                 inputs.Patch(4, 1, 100, "set", 0xFF80),          # -Inf
                 inputs.Patch(4, 1, 101, "set", 0x7F81),          # NaN with the smallest payload
                 inputs.Patch(6, 2, 7, "set", 0x7F7F)]            # largest finite bf16: no count
    inputs.apply_patches(views, w.specs, w.patches)
    gpu, osigs, _ = _compare_everything(w, views, variant=variant)
    assert int(gpu["sigs"]["nan_count"].sum()) == 2 and int(gpu["sigs"]["inf_count"].sum()) == 2

    for dtype, pats in (("f32", [0x7FC00000, 0x7F800000, 0xFF800001, 0x7F7FFFFF]),
                        ("f16", [0x7E00, 0x7C00, 0xFC01, 0x7BFF]),
                        ("f64", [0x7FF8000000000000, 0x7FF0000000000000, 0xFFF0000000000001,
                                 0x7FEFFFFFFFFFFFFF])):
        w = _odd_workload(dtype, 78)
        _, views = inputs.generate(w, "cuda")
        w.patches = [inputs.Patch(i % 3, len(w.specs) - 1 - i, i, "set", p) for i, p in enumerate(pats)]
        inputs.apply_patches(views, w.specs, w.patches)
        gpu, _, _ = _compare_everything(w, views, variant=variant)
        assert int(gpu["sigs"]["nan_count"].sum()) == 2 and int(gpu["sigs"]["inf_count"].sum()) == 1


@pytest.mark.parametrize("variant", VARIANTS)
def test_bf16_subnormals_zeros_and_tiny_values(variant):
    """The bf16 fast path widens part of the elements by bit placement, which is
    exact for zeros and normal values; tiles whose squares are all tiny must fall
    back to the exact loop, all-zero tiles must not."""
    n = 40_000
    specs = [inputs.TensorSpec(name, (n,), "bf16", "normal", 1.0)
             for name in ("subnormal", "zeros", "tiny", "mixed", "negzero")]
    w = inputs.Workload("bf16_small_magnitudes", 0, "x", 3, 16384, specs, 123)
    flats, views = inputs.generate(w, "cuda")
    g = torch.Generator(device="cuda").manual_seed(7)
    for r in range(w.R):
        iv = [v.view(torch.int16) for v in views[r]]
        if r == 0:
            pat = torch.randint(0, 0x80, (n,), generator=g, device="cuda", dtype=torch.int32)
            sign = torch.randint(0, 2, (n,), generator=g, device="cuda", dtype=torch.int32) << 15
            sub = ((pat | sign) & 0xFFFF).to(torch.int32)
            sub = torch.where(sub >= 0x8000, sub - 0x10000, sub).to(torch.int16)
            tiny = torch.randint(0x0080, 0x0400, (n,), generator=g, device="cuda", dtype=torch.int32).to(torch.int16)
            mixed = views[r][3].view(torch.int16).clone()
            mixed[::3] = sub[::3]
            mixed[1::7] = 0
            first = (sub, torch.zeros(n, dtype=torch.int16, device="cuda"), tiny, mixed,
                     torch.full((n,), -0x8000, dtype=torch.int16, device="cuda"))
        for dst, src in zip(iv, first):
            dst.copy_(src)
    gpu, osigs, chunks = _compare_everything(w, views, variant=variant)
    assert (osigs["sumsq"][osigs["sumsq"] > 0] < 1e-60).any()      # the tiny-square case is present
    for t in (1, 4):                                               # +0 and -0 tensors: exactly zero
        assert (gpu["sigs"]["sumsq"][chunks["tensor"] == t] == 0).all()


def test_huge_finite_values_take_the_classifying_path_and_stay_exact():
    # squares beyond 2^256 trip the non-finite suspicion although every element is finite
    specs = [inputs.TensorSpec("big", (6000,), "f32", "normal", 3e38 / 4),
             inputs.TensorSpec("big64", (3000,), "f64", "normal", 1e200)]
    w = inputs.Workload("huge", 0, "huge", 2, 4096, specs, 9)
    _, views = inputs.generate(w, "cuda")
    gpu, _, _ = _compare_everything(w, views)
    assert int(gpu["sigs"]["nan_count"].sum()) == 0 and int(gpu["sigs"]["inf_count"].sum()) == 0


@pytest.mark.parametrize("R", [2, 3, 4, 5, 8, 16, 31, 32, 33, 63, 64])
def test_vote_kernel_alone(R):
    b = _binding()
    rng = np.random.default_rng(R)
    C = 1500
    sigs = np.zeros((C, R), dtype=b.SIG_DTYPE)
    alphabet = rng.integers(1, 2**63, size=5, dtype=np.uint64)
    # mix of clean rows, single outliers, splits and noise
    kind = rng.integers(0, 4, size=C)
    for c in range(C):
        if kind[c] == 0:
            sigs["hash"][c] = alphabet[0]
        elif kind[c] == 1:
            sigs["hash"][c] = alphabet[0]
            sigs["hash"][c, rng.integers(0, R)] = alphabet[1]
        elif kind[c] == 2:
            sigs["hash"][c] = alphabet[0]
            sigs["hash"][c, : R // 2] = alphabet[2]
        else:
            sigs["hash"][c] = alphabet[rng.integers(0, 3, size=R)]
    sigs["sum"] = rng.standard_normal((C, R))
    want = orc.vote(sigs)
    d_sigs = torch.from_numpy(sigs.view(np.uint8).reshape(-1)).cuda()
    d_status = torch.empty(C, dtype=torch.uint8, device="cuda")
    d_bitmap = torch.empty(C, dtype=torch.int64, device="cuda")
    ocap, ucap = C * R, C
    d_out = torch.empty(ocap * 16, dtype=torch.uint8, device="cuda")
    d_und = torch.empty(ucap, dtype=torch.int64, device="cuda")
    d_counts = torch.empty(6, dtype=torch.int64, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    b.scout_consensus_vote(R, C, d_sigs.data_ptr(), d_status.data_ptr(), d_bitmap.data_ptr(),
                           d_out.data_ptr(), ocap, d_und.data_ptr(), ucap, d_counts.data_ptr(), s)
    torch.cuda.synchronize()
    counts = [int(x) for x in d_counts.cpu().numpy()]
    assert counts == want["counts"]
    assert (d_status.cpu().numpy() == want["status"]).all()
    assert (d_bitmap.cpu().numpy().view(np.uint64) == want["bitmap"]).all()
    outl = d_out.cpu().numpy().view(b.OUTLIER_DTYPE)[:counts[4]]
    assert sorted((int(o["chunk"]), int(o["replica"])) for o in outl) == want["outliers"]
    assert sorted(int(x) for x in d_und.cpu().numpy()[:counts[5]]) == want["undecided"]

    # short lists: entries beyond capacity are dropped, counters keep the true totals
    d_counts.zero_()
    d_out.fill_(0xEE)
    b.scout_consensus_vote(R, C, d_sigs.data_ptr(), 0, 0, d_out.data_ptr(), 3, d_und.data_ptr(), 2,
                           d_counts.data_ptr(), s)
    torch.cuda.synchronize()
    assert [int(x) for x in d_counts.cpu().numpy()] == want["counts"]
    raw = d_out.cpu().numpy()
    assert (raw[3 * 16:] == 0xEE).all()                      # nothing written past the capacity
    kept = raw[:min(3, want["counts"][4]) * 16].view(b.OUTLIER_DTYPE)
    assert len(kept) == min(3, want["counts"][4])
    assert {(int(o["chunk"]), int(o["replica"])) for o in kept} <= set(want["outliers"])


def test_results_are_bitwise_reproducible_and_independent_of_tiling():
    w = inputs.workload(4, "default", SMALL[4])
    _, views = inputs.generate(w, "cuda")
    a = helpers.gpu_sign_vote(w, views)
    b = helpers.gpu_sign_vote(w, views)
    assert a["sigs"].tobytes() == b["sigs"].tobytes()
    for tile, variant in ((2048, "fused"), (32768, "fused"), (2048, "unfused"), (32768, "unfused"), (8192, 0), (32768, 0), (8192, 1), (32768, 2), (65536, 2), (65536, 1), (32768, 4), (2048, 4)):
        c = helpers.gpu_sign_vote(w, views, tile_bytes=tile, variant=variant)
        assert (c["sigs"]["hash"] == a["sigs"]["hash"]).all()
        assert c["outliers"] == a["outliers"]
        assert np.allclose(c["sigs"]["sumsq"], a["sigs"]["sumsq"], rtol=1e-13, atol=0)


def test_certify_and_rollups():
    b = _binding()
    w = inputs.workload(4, "default", SMALL[4])
    _, views = inputs.generate(w, "cuda")
    host_views = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host_views, chunk_bytes=65536)
    want = orc.certify(osigs)
    assert len(want["outliers"]) >= 2        # the seeded flips land in different chunks
    plan = helpers.gpu_plan(w, chunk_bytes=65536)
    plan.bind(views)
    got = plan.certify()
    assert got["rc"] == 0
    assert got["report"] == want["report"]
    assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"]
    assert b.scout_plan_replica_bad_counts(plan.handle, w.R) == want["replica_bad"]
    assert got["report"]["verdict"] == b.VERDICT_ATTRIBUTED
    assert got["report"]["replica_union_bitmap"] == 1 << w.patches[0].replica
    # truncated host lists
    cut = plan.certify(outlier_cap=1, undecided_cap=0)
    assert cut["rc"] == b.ERR_TRUNCATED and cut["report"] == want["report"]
    assert len(cut["outliers"]) == 1 and cut["outliers"][0] in want["outliers"]
    # tensor-level signatures
    d_sigs, _, _ = b.scout_plan_results(plan.handle)
    d_roll = torch.empty(len(w.specs) * w.R, dtype=torch.int64, device="cuda")
    b.scout_rollup_tensors(plan.handle, d_sigs, d_roll.data_ptr(), torch.cuda.current_stream().cuda_stream)
    roll = d_roll.cpu().numpy().view(np.uint64).reshape(len(w.specs), w.R)
    for t in range(len(w.specs)):
        sel = np.nonzero(chunks["tensor"] == t)[0]
        for r in range(w.R):
            assert int(roll[t, r]) == orc.rollup(osigs["hash"][sel, r])
    helpers.assert_guards(plan)
    plan.close()

    # clean and undecided verdicts
    wc = inputs.workload(2, "clean", SMALL[2])
    _, vc = inputs.generate(wc, "cuda")
    plan = helpers.gpu_plan(wc)
    plan.bind(vc)
    rep = plan.certify()
    oc, _ = helpers.oracle_sign_all(wc, [[v.cpu() for v in rep_] for rep_ in vc])
    assert rep["report"] == orc.certify(oc)["report"] and rep["report"]["verdict"] == b.CERTIFIED
    ws = inputs.workload(2, "split22", SMALL[2])
    inputs.apply_patches(vc, ws.specs, ws.patches)
    rep = plan.certify()
    assert rep["report"]["verdict"] == b.UNDECIDED and rep["report"]["certificate"] == 0
    assert len(rep["undecided"]) == 1 and rep["outliers"] == []
    helpers.assert_guards(plan)
    plan.close()


def test_certify_host_streams_pinned_replicas():
    b = _binding()
    w = inputs.workload(5, "default", SMALL[5])
    flats, views = inputs.generate(w, "cpu")
    pinned = [f.pin_memory() for f in flats]
    pviews = [inputs.tensor_views(f, w.specs) for f in pinned]
    osigs, _ = helpers.oracle_sign_all(w, views)
    want = orc.certify(osigs)
    plan = helpers.gpu_plan(w)
    got = b.scout_certify_host(plan.handle, [v.data_ptr() for rep in pviews for v in rep])
    assert got["report"] == want["report"] and got["outliers"] == want["outliers"]
    d_sigs, _, _ = b.scout_plan_results(plan.handle)
    helpers.assert_guards(plan)
    plan.close()


def test_bind_rejects_misaligned_and_null_pointers():
    b = _binding()
    w = inputs.workload(1, "clean", SMALL[1])
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    ptrs = [v.data_ptr() for rep in views for v in rep]
    for bad, code in ((ptrs[0] + 4, b.ERR_ALIGN), (0, b.ERR_INVALID)):
        with pytest.raises(b.ScoutError) as e:
            b.scout_plan_bind(plan.handle, [bad] + ptrs[1:])
        assert e.value.code == code
    with pytest.raises(b.ScoutError):           # signing before a successful bind
        plan.sign()
    helpers.assert_guards(plan)
    plan.close()


def test_three_step_protocol_clean_fault_clean():
    w = inputs.workload(1, "default", SMALL[1])
    _, views = inputs.generate(inputs.workload(1, "clean", SMALL[1]), "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    plan.sign_and_vote()
    assert plan.fetch()["outliers"] == []
    old = inputs.apply_patches(views, w.specs, w.patches)
    plan.sign_and_vote()
    faulty = plan.fetch()
    chunks = plan.chunk_table()
    assert faulty["outliers"] == helpers.expected_from_patches(w, chunks)[0]
    inputs.revert_patches(views, w.specs, w.patches, old)
    plan.sign_and_vote()
    assert plan.fetch()["outliers"] == []
    helpers.assert_guards(plan)
    plan.close()
