"""Seeded random plans through every launch form against the oracle.

Each case draws a tensor table (1 to 6 tensors of mixed dtypes and ragged sizes), a
chunk size, a replica count, a tile size and a handful of faults (bit flips, NaN and Inf
overwrites, the same edit in several replicas), then runs scout_certify in the
per-stage, ticket and cluster forms and scout_sign_chunks + scout_consensus_vote, and
compares records, vote and report with the oracle.  The cases are fixed by their seeds,
so a failure reproduces."""
import random

import numpy as np
import pytest
import torch

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu

DTYPES = ["f32", "bf16", "i64", "f16", "u8", "f64", "i32"]
DIST = {"u8": "bytes", "i64": "randint40", "i32": "randfull"}
NONFINITE = {"f32": (0x7FC00000, 0x7F800000), "bf16": (0x7FC0, 0xFF80), "f16": (0x7E00, 0x7C00)}


def _random_workload(seed):
    rng = random.Random(seed)
    R = rng.choice([2, 3, 3, 4, 5, 8, 11, 16])
    chunk_bytes = 512 * rng.choice([1, 3, 8, 16, 33, 128, 512])
    specs = []
    for t in range(rng.randint(1, 6)):
        dt = rng.choice(DTYPES)
        es = inputs.DTYPE_BYTES[dt]
        nbytes = rng.choice([es, 16, 512, 4096, chunk_bytes, rng.randrange(1, 6 * chunk_bytes), rng.randrange(1, 300_000)])
        numel = max(1, nbytes // es)
        specs.append(inputs.TensorSpec(f"t{t}", (numel,), dt, DIST.get(dt, "normal"), 10.0 ** rng.randint(-6, 3)))
    w = inputs.Workload(f"random_{seed}", 0, "random", R, chunk_bytes, specs, 9000 + seed)
    patches = []
    for _ in range(rng.randint(0, 5)):
        t = rng.randrange(len(specs))
        s = specs[t]
        el = rng.randrange(s.numel)
        kind = rng.random()
        if kind < 0.2 and s.dtype in NONFINITE:
            patches.append(inputs.Patch(rng.randrange(R), t, el, "set", rng.choice(NONFINITE[s.dtype])))
        elif kind < 0.4:      # the same edit in several replicas: majority-held or split votes
            bit = 1 << rng.randrange(8 * inputs.DTYPE_BYTES[s.dtype])
            for r in rng.sample(range(R), rng.randint(1, R)):
                patches.append(inputs.Patch(r, t, el, "xor", bit))
        else:
            patches.append(inputs.Patch(rng.randrange(R), t, el, "xor", 1 << rng.randrange(8 * inputs.DTYPE_BYTES[s.dtype])))
    w.patches = patches
    tile = rng.choice([None, 2048, 4096, 8192])
    return w, tile


@pytest.mark.parametrize("seed", range(64))
def test_random_plan_every_form(seed):
    from paper_2608_11034_b200 import binding as B
    w, tile = _random_workload(seed)
    _, views = inputs.generate(w, "cuda")
    host = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host)
    want = orc.certify(osigs)
    ov = orc.vote(osigs)
    scale = helpers.chunk_abs_sums(w, host, chunks)

    gpu = helpers.gpu_sign_vote(w, views, tile_bytes=tile)          # two calls, default forms
    helpers.assert_sigs_match(gpu["sigs"], osigs, scale)
    assert (gpu["status"] == ov["status"]).all() and (gpu["bitmap"] == ov["bitmap"]).all()
    assert gpu["counts"] == ov["counts"]
    assert gpu["outliers"] == ov["outliers"] and gpu["undecided"] == ov["undecided"]

    plan = helpers.gpu_plan(w, tile_bytes=tile)
    plan.bind(views)
    forms = [0, 1] + ([2] if B.scout_plan_get(plan.handle, "cluster_ok") else [])
    for form in forms + [-1]:
        B.scout_plan_set(plan.handle, "fused", form)
        for _ in range(2):
            got = plan.certify()
            assert got["report"] == want["report"], (seed, form)
            assert got["outliers"] == want["outliers"] and got["undecided"] == want["undecided"], (seed, form)
            assert B.scout_plan_replica_bad_counts(plan.handle, w.R) == want["replica_bad"]
        if form >= 0:       # the same kernels as scout_sign_chunks: full records
            plan.sign()
            torch.cuda.synchronize()
            gs = plan.d_sigs.cpu().numpy().view(B.SIG_DTYPE).reshape(plan.C, w.R)
            helpers.assert_sigs_match(gs, osigs, scale)
    helpers.assert_guards(plan)
    plan.close()
