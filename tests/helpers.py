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
