"""Shared test plumbing: run the CPU oracle over a generated workload and work
out, from the fault patches alone, which (chunk, replica) pairs must be named."""
from __future__ import annotations

import numpy as np

import defn
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

ORC_CODE = {"u8": orc.DT_U8, "f32": orc.DT_F32, "bf16": orc.DT_BF16, "i64": orc.DT_I64,
            "f16": orc.DT_F16, "f64": orc.DT_F64, "i32": orc.DT_I32}


def shape_tags(w):
    return [defn.shape_tag(list(s.shape)) for s in w.specs]


def oracle_tensor_table(w, tags=None):
    tags = shape_tags(w) if tags is None else tags
    return orc.make_tensor_table([(s.nbytes, ORC_CODE[s.dtype], g) for s, g in zip(w.specs, tags)])


def oracle_sign_all(w, views, chunk_bytes=None, nthreads=4, tags=None):
    """-> (sigs[C, R], chunk table) computed by the oracle on host copies."""
    cb = w.chunk_bytes if chunk_bytes is None else chunk_bytes
    tt = oracle_tensor_table(w, tags)
    chunks = orc.chunk_table(tt, cb)
    sigs = np.zeros((len(chunks), w.R), dtype=orc.SIG_DTYPE)
    for r in range(w.R):
        arrays = [inputs.to_numpy_bytes(v) for v in views[r]]
        orc.sign_replica(tt, arrays, cb, sigs, r, nthreads)
    return sigs, chunks


def chunk_of(chunks, tensor, byte_in_tensor):
    sel = np.nonzero((chunks["tensor"] == tensor)
                     & (chunks["byte_offset"] <= byte_in_tensor)
                     & (byte_in_tensor < chunks["byte_offset"] + chunks["nbytes"]))[0]
    assert len(sel) == 1
    return int(sel[0])


def expected_from_patches(w, chunks):
    """What the vote must report, derived from the patch list only: replicas
    that received the same edits inside a chunk hold the same bytes there."""
    per_chunk = {}
    for p in w.patches:
        es = inputs.DTYPE_BYTES[w.specs[p.tensor].dtype]
        c = chunk_of(chunks, p.tensor, p.element * es)
        per_chunk.setdefault(c, {}).setdefault(p.replica, set()).add((p.element, p.op, p.value))
    outliers, undecided = [], []
    for c, edits in sorted(per_chunk.items()):
        keys = [frozenset(edits.get(r, ())) for r in range(w.R)]
        status, B = defn.vote_one(keys)
        if status == defn.INCONCLUSIVE:
            undecided.append(c)
        outliers += [(c, r) for r in range(w.R) if (B >> r) & 1]
    return sorted(outliers), undecided


# ---- CUDA path plumbing (imported lazily so CPU-only runs never load it) -----

def gpu_plan(w, chunk_bytes=None, tags=None, tile_bytes=None, variant=None):
    from paper_2608_11034_b200 import binding
    tags = shape_tags(w) if tags is None else tags
    # every output buffer of the tests sits between guard bands (see gpu_sign_vote)
    plan = binding.Plan(w.R, binding.make_tensor_table(w.specs, tags),
                        w.chunk_bytes if chunk_bytes is None else chunk_bytes, guards=True)
    if tile_bytes is not None:
        binding.scout_plan_set(plan.handle, "tile_bytes", tile_bytes)
    if variant == "unfused":      # the default scan (register-prefetch front end), one kernel per stage
        binding.scout_plan_set(plan.handle, "fused", 0)
    elif variant == "fused":      # the default scan, the whole call as one launch (tickets)
        binding.scout_plan_set(plan.handle, "fused", 1)
    elif variant == "cluster":    # one launch, a thread-block cluster per chunk (R <= 8, <= 512 tiles per chunk)
        import pytest
        if not binding.scout_plan_get(plan.handle, "cluster_ok"):
            plan.close()
            pytest.skip("the cluster form does not fit this plan (R > 8 or more than 512 tiles per chunk)")
        binding.scout_plan_set(plan.handle, "fused", 2)
    elif variant is not None:
        binding.scout_plan_set(plan.handle, "variant", variant)
    return plan


def gpu_sign_vote(w, views, chunk_bytes=None, tags=None, tile_bytes=None, caps=(4096, 4096),
                  variant=None):
    """-> fetch() dict of the CUDA path over device-resident views[r][t]."""
    from paper_2608_11034_b200 import binding
    plan = gpu_plan(w, chunk_bytes, tags, tile_bytes, variant)
    plan.bind(views)
    plan.sign_and_vote(*caps)
    out = plan.fetch()
    assert binding.scout_plan_get(plan.handle, "device_error") == 0
    # nothing was written outside the caller's output buffers, nor (debug mode, which the GPU
    # tests switch on through SCOUT_DEBUG=1) outside any buffer the plan owns
    assert plan.check_guards()
    if binding.scout_plan_get(plan.handle, "debug"):
        assert binding.scout_plan_get(plan.handle, "guards_ok") == 1
    plan.close()
    return out


def assert_guards(plan):
    """No kernel wrote outside the caller's output buffers nor outside the plan's own."""
    from paper_2608_11034_b200 import binding
    assert plan.check_guards()
    if binding.scout_plan_get(plan.handle, "debug"):
        assert binding.scout_plan_get(plan.handle, "guards_ok") == 1


def chunk_abs_sums(w, views, chunks):
    """sum |x| over the finite elements of every (chunk, replica): the scale of
    the tolerance on the sums."""
    out = np.zeros((len(chunks), w.R))
    for r in range(w.R):
        host = [inputs.to_numpy_bytes(v) for v in views[r]]
        for c, ch in enumerate(chunks):
            dt = w.specs[int(ch["tensor"])].dtype
            if dt == "u8":
                continue
            b = host[int(ch["tensor"])][int(ch["byte_offset"]):int(ch["byte_offset"] + ch["nbytes"])]
            x = np.abs(defn.values_f64(b.tobytes(), dt))
            out[c, r] = x[np.isfinite(x)].sum()
    return out


REL_TOL = 1e-12


def assert_sigs_match(gpu_sigs, orc_sigs, abs_sums):
    """Bit-exact hashes and counts; sums within 1e-12 of the un-cancelled scale
    (|d sum| <= 1e-12 * sum|x|, |d sumsq| <= 1e-12 * sumsq)."""
    assert gpu_sigs.shape == orc_sigs.shape
    assert (gpu_sigs["hash"] == orc_sigs["hash"]).all()
    assert (gpu_sigs["nan_count"] == orc_sigs["nan_count"]).all()
    assert (gpu_sigs["inf_count"] == orc_sigs["inf_count"]).all()
    for name, scale in (("sum", abs_sums), ("sumsq", np.abs(orc_sigs["sumsq"]))):
        g, o = gpu_sigs[name], orc_sigs[name]
        both_inf = np.isinf(g) & np.isinf(o) & (np.sign(g) == np.sign(o))
        err = np.where(both_inf, 0.0, np.abs(g - o))
        assert np.isfinite(err).all(), name
        assert (err <= REL_TOL * scale).all(), (name, float(err.max()))
