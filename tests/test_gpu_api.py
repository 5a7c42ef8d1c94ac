"""Behaviour of the C ABI beyond the main path: plan knobs, re-binding, user
streams, host-resident replicas in pageable and scattered memory."""
import numpy as np
import pytest
import torch

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def test_plan_knobs():
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(1, "default", 1 / 8)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    h = plan.handle
    assert B.scout_plan_get(h, "tile_bytes") in (4096, 8192, 16384, 32768)
    assert B.scout_plan_get(h, "variant") == 1 and B.scout_plan_get(h, "grid") > 0
    n0 = B.scout_plan_get(h, "n_tiles")
    B.scout_plan_set(h, "tile_bytes", 2048)
    assert B.scout_plan_get(h, "n_tiles") == w.bytes_per_replica // 2048 != n0
    assert B.scout_plan_get(h, "scratch_bytes") == B.scout_plan_get(h, "n_tiles") * w.R * 32
    for key, bad in (("tile_bytes", 1000), ("tile_bytes", 524288), ("variant", 5), ("variant", -1),
                     ("grid", 0), ("nonsense", 1)):
        with pytest.raises(B.ScoutError):
            B.scout_plan_set(h, key, bad)
    with pytest.raises(B.ScoutError):
        B.scout_plan_get(h, "nonsense")
    with pytest.raises(B.ScoutError):            # timing was never switched on
        B.scout_plan_get(h, "last_sign_ns")
    B.scout_plan_set(h, "tile_bytes", 65536)
    with pytest.raises(B.ScoutError):            # the block-wide ring needs a tile that fits one stage
        B.scout_plan_set(h, "variant", 4)
    B.scout_plan_set(h, "tile_bytes", 8192)
    B.scout_plan_set(h, "grid", 7)               # a tiny grid must still give the same records
    B.scout_plan_set(h, "timing", 1)
    plan.bind(views)
    plan.sign_and_vote()
    got = plan.fetch()
    assert B.scout_plan_get(h, "last_sign_ns") > 0 and B.scout_plan_get(h, "device_error") == 0
    ref = helpers.gpu_sign_vote(w, views)
    assert (got["sigs"]["hash"] == ref["sigs"]["hash"]).all() and got["outliers"] == ref["outliers"]
    helpers.assert_guards(plan)
    plan.close()


def test_rebinding_and_user_streams():
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(2, "mantissa", 1 / 64)
    _, views_a = inputs.generate(w, "cuda")
    wb = inputs.workload(2, "clean", 1 / 64)
    wb.seed += 100
    _, views_b = inputs.generate(wb, "cuda")
    plan = helpers.gpu_plan(w)
    side = torch.cuda.Stream()
    results = []
    for views in (views_a, views_b, views_a):
        plan.bind(views)
        with torch.cuda.stream(side):
            plan.sign_and_vote()            # enqueued on the side stream (the current one)
            side.synchronize()
        results.append(plan.fetch())
    assert len(results[0]["outliers"]) == 1 and results[1]["outliers"] == []
    assert results[0]["sigs"].tobytes() == results[2]["sigs"].tobytes()
    assert (results[0]["sigs"]["hash"] != results[1]["sigs"]["hash"]).all()
    rep = plan.certify(stream=side.cuda_stream)
    assert rep["outliers"] == results[0]["outliers"]
    helpers.assert_guards(plan)
    plan.close()


def test_certify_host_with_pageable_and_scattered_tensors():
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(5, "default", 1 / 400)
    _, views = inputs.generate(w, "cpu")
    osigs, _ = helpers.oracle_sign_all(w, views)
    want = orc.certify(osigs)
    # every tensor in its own pageable allocation, replicas interleaved: nothing is contiguous
    keep = [[v.clone() for v in rep] for rep in views]
    ptrs = [t.data_ptr() for rep in keep for t in rep]
    plan = helpers.gpu_plan(w)
    got = B.scout_certify_host(plan.handle, ptrs)
    assert got["report"] == want["report"] and got["outliers"] == want["outliers"]
    # change the tiling after the staging buffers exist, then run again from flat pinned buffers
    B.scout_plan_set(plan.handle, "tile_bytes", 4096)
    flats = []
    for rep in views:
        offs, total = inputs.packed_offsets(w.specs)
        f = torch.zeros(total, dtype=torch.uint8).pin_memory()
        for o, v in zip(offs, rep):
            f[o:o + v.numel() * v.element_size()] = v.view(-1).view(torch.uint8)
        flats.append(f)
    fviews = [inputs.tensor_views(f, w.specs) for f in flats]
    got2 = B.scout_certify_host(plan.handle, [v.data_ptr() for rep in fviews for v in rep])
    assert got2["report"] == want["report"] and got2["outliers"] == want["outliers"]
    # device-resident certify on the same plan still works after the host runs
    dviews = [[v.cuda() for v in rep] for rep in views]
    plan.bind(dviews)
    got3 = plan.certify()
    assert got3["report"] == want["report"]
    helpers.assert_guards(plan)
    plan.close()


def test_a_wait_that_nothing_satisfies_gives_up_and_the_context_survives():
    """The bulk-async kernels never spin without a limit: a wait on a barrier that is
    never signalled returns after its time limit with a status the host can read."""
    from paper_2608_11034_b200 import binding as B
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    limit = 2_000_000                                      # 2 ms
    B.scout_selftest_bounded_wait(limit, out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    gave_up, waited = [int(x) for x in out.cpu()]
    assert gave_up == 1 and limit <= waited < 100 * limit
    # the context is intact: an ordinary run right after it works
    w = inputs.workload(1, "default", 1 / 16)
    _, views = inputs.generate(w, "cuda")
    got = helpers.gpu_sign_vote(w, views, variant=4)
    assert len(got["outliers"]) == 1
    with pytest.raises(B.ScoutError):
        B.scout_selftest_bounded_wait(0, out.data_ptr(), 0)


def test_device_error_flag_is_reported_once_and_cleared():
    """A host-made failure: the flag a timed-out wait would leave is written from the
    host.  The certify that sees it fails with SCOUT_ERR_CUDA and clears it; the next
    one succeeds."""
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(1, "default", 1 / 8)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    good = plan.certify()
    B.scout_plan_set(plan.handle, "device_error", 1)
    assert B.scout_plan_get(plan.handle, "device_error") == 1
    with pytest.raises(B.ScoutError) as e:
        plan.certify()
    assert e.value.code == B.ERR_CUDA
    assert B.scout_plan_get(plan.handle, "device_error") == 0
    again = plan.certify()
    assert again["report"] == good["report"] and again["outliers"] == good["outliers"]
    # the asynchronous path cannot report: the flag stays readable until it is cleared by hand
    B.scout_plan_set(plan.handle, "device_error", 7)
    plan.sign_and_vote()
    torch.cuda.synchronize()
    assert B.scout_plan_get(plan.handle, "device_error") == 1
    B.scout_plan_set(plan.handle, "device_error", 0)
    assert B.scout_plan_get(plan.handle, "device_error") == 0
    helpers.assert_guards(plan)
    plan.close()


def test_rebinding_waits_for_a_scan_in_flight_on_a_non_blocking_stream():
    """Re-binding right after an asynchronous sign on a non-blocking stream must not change
    the table under the running scan: the records are those of the buffers bound at launch."""
    from paper_2608_11034_b200 import binding as B
    wa = inputs.Workload("bind_a", 0, "x", 3, 1 << 20,
                         [inputs.TensorSpec("x", (48 << 20,), "f32", "normal", 0.02)], 7)
    _, va = inputs.generate(wa, "cuda")
    wb = inputs.Workload("bind_b", 0, "x", 3, 1 << 20,
                         [inputs.TensorSpec("x", (48 << 20,), "f32", "normal", 0.02)], 8)
    _, vb = inputs.generate(wb, "cuda")
    plan = helpers.gpu_plan(wa)
    side = torch.cuda.Stream()                  # torch's side streams do not sync with the default stream
    d_a = torch.zeros(plan.C * wa.R * 32, dtype=torch.uint8, device="cuda")
    d_b = torch.zeros_like(d_a)
    torch.cuda.synchronize()
    plan.bind(va)
    B.scout_sign_chunks(plan.handle, side.cuda_stream, d_a.data_ptr())
    plan.bind(vb)                               # 576 MB scan still running when this is called
    B.scout_sign_chunks(plan.handle, side.cuda_stream, d_b.data_ptr())
    side.synchronize()
    got_a = d_a.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, wa.R)
    got_b = d_b.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, wa.R)
    helpers.assert_guards(plan)
    plan.close()
    ref_a = helpers.gpu_sign_vote(wa, va)["sigs"]
    ref_b = helpers.gpu_sign_vote(wb, vb)["sigs"]
    assert (got_a["hash"] == ref_a["hash"]).all() and (got_b["hash"] == ref_b["hash"]).all()
    assert (ref_a["hash"] != ref_b["hash"]).all()


def test_a_plan_used_with_another_device_current_is_rejected():
    """The plan's tables live on the device that was current at creation.  With a
    different current device every plan call returns SCOUT_ERR_INVALID.  On a one-GPU
    box the same check is exercised through the plan's recorded device."""
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(1, "default", 1 / 16)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    if torch.cuda.device_count() < 2:
        helpers.assert_guards(plan)
        plan.close()
        pytest.skip("needs two GPUs")
    d_sigs = torch.zeros(plan.C * w.R * 32, dtype=torch.uint8, device="cuda:0")
    try:
        torch.cuda.set_device(1)
        with pytest.raises(B.ScoutError) as e:
            B.scout_sign_chunks(plan.handle, 0, d_sigs.data_ptr())
        assert e.value.code == B.ERR_INVALID
        with pytest.raises(B.ScoutError):
            B.scout_plan_bind(plan.handle, [v.data_ptr() for rep in views for v in rep])
    finally:
        torch.cuda.set_device(0)
    helpers.assert_guards(plan)
    plan.close()


def test_guard_bands_notice_a_stray_write():
    """The tests' stand-in for a memory checker: output buffers between guard bands.  A byte
    written just outside a buffer (here by hand) is reported; untouched bands are not."""
    from paper_2608_11034_b200 import binding as B
    w = inputs.workload(1, "default", 1 / 16)
    _, views = inputs.generate(w, "cuda")
    plan = helpers.gpu_plan(w)
    assert B.scout_plan_get(plan.handle, "debug") == 1      # conftest switches the debug mode on
    plan.bind(views)
    plan.sign_and_vote()
    plan.certify()
    helpers.assert_guards(plan)
    outer, nbytes = plan._outer[0]
    outer[B.Plan.GUARD_BYTES + nbytes] = 0                   # first byte after the record table
    assert not plan.check_guards()
    outer[B.Plan.GUARD_BYTES + nbytes] = B.Plan.GUARD_PATTERN
    outer[B.Plan.GUARD_BYTES - 1] = 1                        # last byte before it
    assert not plan.check_guards()
    outer[B.Plan.GUARD_BYTES - 1] = B.Plan.GUARD_PATTERN
    assert plan.check_guards()
    plan.close()


@pytest.mark.parametrize("streams", [1, 3, 8, 32])
def test_work_counters_any_number_same_records(streams):
    """The tiles of the staged scan are dealt from `work_streams` counters; a warp whose counter
    has run out moves on to the next.  Whatever their number, every tile is scanned exactly once:
    records equal to the oracle's, twice in a row (the counters of one launch are zeroed by the
    previous one).  13,000 tiles for 4,736 warps, so most tiles come from the counters."""
    from paper_2608_11034_b200 import binding as b
    spec = inputs.TensorSpec("x", (2_218_667,), "f32", "normal", 0.02)      # 4,334 tiles of 2 KiB per replica
    w = inputs.Workload("streams", 0, "x", 3, 65536, [spec], 31)
    w.patches = [inputs.Patch(2, 0, 2_000_000, "xor", 1 << 7)]
    _, views = inputs.generate(w, "cuda")
    host = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host)
    plan = helpers.gpu_plan(w, tile_bytes=2048, variant="unfused")
    b.scout_plan_set(plan.handle, "work_streams", streams)
    assert b.scout_plan_get(plan.handle, "work_streams") == streams
    plan.bind(views)
    for _ in range(3):
        plan.sign()
        torch.cuda.synchronize()
        gs = plan.d_sigs.cpu().numpy().view(b.SIG_DTYPE).reshape(plan.C, w.R)
        helpers.assert_sigs_match(gs, osigs, helpers.chunk_abs_sums(w, host, chunks))
    with pytest.raises(b.ScoutError):
        b.scout_plan_set(plan.handle, "work_streams", 33)
    helpers.assert_guards(plan)
    plan.close()
