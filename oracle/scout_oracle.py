"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not product code).

Only tests, the smoke check and the benchmark's CPU legs may import this
module.  It compiles ``scout_oracle.c`` with gcc on first use and exposes the C
functions on numpy arrays.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "scout_oracle.c")
_HDR = os.path.join(_HERE, "scout_oracle.h")
_LIB = os.path.join(_HERE, "libscout_oracle.so")
_lock = threading.Lock()
_lib = None

DT_U8, DT_F32, DT_BF16, DT_I64, DT_F16, DT_F64, DT_I32 = range(7)
AGREE, ATTRIBUTED, INCONCLUSIVE = 0, 1, 2

SIG_DTYPE = np.dtype([("hash", "<u8"), ("nan_count", "<u4"), ("inf_count", "<u4"),
                      ("sum", "<f8"), ("sumsq", "<f8")])
TENSOR_DTYPE = np.dtype([("nbytes", "<u8"), ("dtype", "<u4"), ("reserved", "<u4"),
                         ("meta_tag", "<u8")])
OUTLIER_DTYPE = np.dtype([("chunk", "<u8"), ("replica", "<u4"), ("reserved", "<u4")])
CHUNK_DTYPE = np.dtype([("tensor", "<u8"), ("index_in_tensor", "<u8"),
                        ("byte_offset", "<u8"), ("nbytes", "<u8")])
REPORT_DTYPE = np.dtype([("n_chunks", "<u8"), ("n_agree", "<u8"), ("n_attributed", "<u8"),
                         ("n_inconclusive", "<u8"), ("n_outliers", "<u8"),
                         ("n_undecided", "<u8"), ("replica_union_bitmap", "<u8"),
                         ("certificate", "<u8"), ("verdict", "<i4"), ("reserved", "<i4")])


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 (no vector intrinsics, no tuning)."""
    with _lock:
        stale = (not os.path.exists(_LIB)
                 or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
        if force or stale:
            tmp = _LIB + ".tmp%d" % os.getpid()
            subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread",
                                   "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u64p, vp = C.POINTER(C.c_uint8), C.POINTER(C.c_uint64), C.c_void_p
        L.orc_dtype_size.restype = C.c_uint32
        L.orc_dtype_size.argtypes = [C.c_uint32]
        L.orc_mix64.restype = C.c_uint64
        L.orc_mix64.argtypes = [C.c_uint64]
        L.orc_slot_multiplier.restype = C.c_uint64
        L.orc_slot_multiplier.argtypes = [C.c_uint32]
        L.orc_hash_raw.restype = C.c_uint64
        L.orc_hash_raw.argtypes = [vp, C.c_uint64]
        L.orc_hash_final.restype = C.c_uint64
        L.orc_hash_final.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64]
        L.orc_shape_tag.restype = C.c_uint64
        L.orc_shape_tag.argtypes = [C.c_uint32, u64p]
        L.orc_stats.restype = None
        L.orc_stats.argtypes = [vp, C.c_uint64, C.c_uint32, C.POINTER(C.c_uint32),
                                C.POINTER(C.c_uint32), C.POINTER(C.c_double),
                                C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.orc_sign_chunk.restype = None
        L.orc_sign_chunk.argtypes = [vp, C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64, vp]
        L.orc_chunk_table.restype = C.c_uint64
        L.orc_chunk_table.argtypes = [C.c_uint64, vp, C.c_uint64, vp, C.c_uint64]
        L.orc_sign_replica.restype = C.c_int
        L.orc_sign_replica.argtypes = [C.c_uint64, vp, vp, C.c_uint64, vp, C.c_uint64,
                                       C.c_uint64, C.c_int]
        L.orc_vote.restype = C.c_int
        L.orc_vote.argtypes = [C.c_uint32, C.c_uint64, vp, vp, vp, vp, C.c_uint64, vp,
                               C.c_uint64, vp]
        L.orc_vote_wide.restype = C.c_int
        L.orc_vote_wide.argtypes = [C.c_uint32, C.c_uint64, vp, C.c_uint64, C.c_uint64, vp, vp, vp,
                                    C.c_uint64, vp, C.c_uint64, vp]
        L.orc_rollup.restype = C.c_uint64
        L.orc_rollup.argtypes = [vp, C.c_uint64]
        L.orc_certificate.restype = C.c_uint64
        L.orc_certificate.argtypes = [C.c_uint32, C.c_uint64, vp, vp, vp]
        L.orc_certify.restype = C.c_int
        L.orc_certify.argtypes = [C.c_uint32, C.c_uint64, vp, vp, vp, C.c_uint64, vp,
                                  C.c_uint64, vp]
        _lib = L
    return _lib


def _bytes_view(buf) -> np.ndarray:
    a = np.ascontiguousarray(np.frombuffer(buf, dtype=np.uint8) if isinstance(buf, (bytes, bytearray, memoryview))
                             else np.asarray(buf))
    return a.reshape(-1).view(np.uint8)


def mix64(z: int) -> int:
    return int(lib().orc_mix64(C.c_uint64(z & (2**64 - 1))))


def slot_multiplier(s: int) -> int:
    return int(lib().orc_slot_multiplier(s))


def hash_raw(buf) -> int:
    a = _bytes_view(buf)
    return int(lib().orc_hash_raw(a.ctypes.data, a.size))


def hash_final(h_raw: int, n: int, k: int, dtype: int, meta_tag: int) -> int:
    return int(lib().orc_hash_final(h_raw, n, k, dtype, meta_tag & (2**64 - 1)))


def shape_tag(dims) -> int:
    d = np.asarray(list(dims), dtype=np.uint64)
    return int(lib().orc_shape_tag(len(d), d.ctypes.data_as(C.POINTER(C.c_uint64))))


def stats(buf, dtype: int):
    """-> (nan_count, inf_count, sum, sumsq, sum_abs) over one chunk."""
    a = _bytes_view(buf)
    nn, ni = C.c_uint32(), C.c_uint32()
    s, q, ab = C.c_double(), C.c_double(), C.c_double()
    lib().orc_stats(a.ctypes.data, a.size, dtype, C.byref(nn), C.byref(ni), C.byref(s),
                    C.byref(q), C.byref(ab))
    return nn.value, ni.value, s.value, q.value, ab.value


def sign_chunk(buf, dtype: int, k: int = 0, meta_tag: int = 0) -> np.ndarray:
    a = _bytes_view(buf)
    out = np.zeros(1, dtype=SIG_DTYPE)
    lib().orc_sign_chunk(a.ctypes.data, a.size, dtype, k, meta_tag & (2**64 - 1), out.ctypes.data)
    return out[0]


def make_tensor_table(tensors) -> np.ndarray:
    """tensors: iterable of (nbytes, dtype code, meta_tag)."""
    t = np.zeros(len(tensors), dtype=TENSOR_DTYPE)
    for i, (nbytes, dt, tag) in enumerate(tensors):
        t[i] = (nbytes, dt, 0, tag & (2**64 - 1))
    return t


def chunk_table(tensor_table: np.ndarray, chunk_bytes: int) -> np.ndarray:
    L = lib()
    n = L.orc_chunk_table(len(tensor_table), tensor_table.ctypes.data, chunk_bytes, None, 0)
    if n == 2**64 - 1:
        raise ValueError("invalid tensor table or chunk size")
    out = np.zeros(n, dtype=CHUNK_DTYPE)
    L.orc_chunk_table(len(tensor_table), tensor_table.ctypes.data, chunk_bytes, out.ctypes.data, n)
    return out


def sign_replica(tensor_table: np.ndarray, arrays, chunk_bytes: int, sigs: np.ndarray,
                 replica: int, nthreads: int = 1) -> None:
    """Sign every chunk of one replica into sigs[C, R] (column ``replica``).

    arrays: one contiguous numpy array per tensor (host memory)."""
    assert sigs.dtype == SIG_DTYPE and sigs.ndim == 2 and sigs.flags.c_contiguous
    keep = [np.ascontiguousarray(a) for a in arrays]
    ptrs = (C.c_void_p * len(keep))(*[a.ctypes.data for a in keep])
    rc = lib().orc_sign_replica(len(tensor_table), tensor_table.ctypes.data,
                                C.cast(ptrs, C.c_void_p), chunk_bytes, sigs.ctypes.data,
                                sigs.shape[1], replica, nthreads)
    if rc != 0:
        raise ValueError("orc_sign_replica failed: %d" % rc)


def vote(sigs: np.ndarray, outlier_cap: int | None = None, undecided_cap: int | None = None):
    """sigs[C, R] -> dict(status, bitmap, outliers [(chunk, replica)], undecided, counts, rc)."""
    assert sigs.dtype == SIG_DTYPE and sigs.ndim == 2
    sigs = np.ascontiguousarray(sigs)
    Cn, R = sigs.shape
    ocap = Cn * R if outlier_cap is None else outlier_cap
    ucap = Cn if undecided_cap is None else undecided_cap
    status = np.zeros(Cn, dtype=np.uint8)
    bitmap = np.zeros(Cn, dtype=np.uint64)
    outl = np.zeros(max(ocap, 1), dtype=OUTLIER_DTYPE)
    und = np.zeros(max(ucap, 1), dtype=np.uint64)
    counts = np.zeros(6, dtype=np.uint64)
    rc = lib().orc_vote(R, Cn, sigs.ctypes.data, status.ctypes.data, bitmap.ctypes.data,
                        outl.ctypes.data, ocap, und.ctypes.data, ucap, counts.ctypes.data)
    if rc == -1:
        raise ValueError("orc_vote: invalid arguments")
    no, nu = min(int(counts[4]), ocap), min(int(counts[5]), ucap)
    return dict(status=status, bitmap=bitmap,
                outliers=[(int(o["chunk"]), int(o["replica"])) for o in outl[:no]],
                undecided=[int(x) for x in und[:nu]], counts=[int(x) for x in counts], rc=rc)


def vote_wide(sigs: np.ndarray, R: int, Cn: int, chunk_stride: int, replica_stride: int):
    """Vote over a flat record table with strides (in records); any R >= 2.
    -> dict(status, bitmap [C, W], outliers, undecided, counts, rc)"""
    assert sigs.dtype == SIG_DTYPE
    flat = np.ascontiguousarray(sigs).reshape(-1)
    W = (R + 63) // 64
    status = np.zeros(Cn, dtype=np.uint8)
    bitmap = np.zeros((Cn, W), dtype=np.uint64)
    outl = np.zeros(max(Cn * R, 1), dtype=OUTLIER_DTYPE)
    und = np.zeros(max(Cn, 1), dtype=np.uint64)
    counts = np.zeros(6, dtype=np.uint64)
    rc = lib().orc_vote_wide(R, Cn, flat.ctypes.data, chunk_stride, replica_stride, status.ctypes.data,
                             bitmap.ctypes.data, outl.ctypes.data, Cn * R, und.ctypes.data, Cn,
                             counts.ctypes.data)
    if rc == -1:
        raise ValueError("orc_vote_wide: invalid arguments")
    return dict(status=status, bitmap=bitmap,
                outliers=[(int(o["chunk"]), int(o["replica"])) for o in outl[:int(counts[4])]],
                undecided=[int(x) for x in und[:int(counts[5])]], counts=[int(x) for x in counts], rc=rc)


def rollup(hashes) -> int:
    h = np.ascontiguousarray(np.asarray(hashes, dtype=np.uint64))
    return int(lib().orc_rollup(h.ctypes.data, h.size))


def certify(sigs: np.ndarray, outlier_cap: int | None = None, undecided_cap: int | None = None):
    assert sigs.dtype == SIG_DTYPE and sigs.ndim == 2
    sigs = np.ascontiguousarray(sigs)
    Cn, R = sigs.shape
    ocap = Cn * R if outlier_cap is None else outlier_cap
    ucap = Cn if undecided_cap is None else undecided_cap
    rep = np.zeros(1, dtype=REPORT_DTYPE)
    outl = np.zeros(max(ocap, 1), dtype=OUTLIER_DTYPE)
    und = np.zeros(max(ucap, 1), dtype=np.uint64)
    bad = np.zeros(R, dtype=np.uint64)
    rc = lib().orc_certify(R, Cn, sigs.ctypes.data, rep.ctypes.data, outl.ctypes.data, ocap,
                           und.ctypes.data, ucap, bad.ctypes.data)
    if rc == -1:
        raise ValueError("orc_certify: invalid arguments")
    r = rep[0]
    no, nu = min(int(r["n_outliers"]), ocap), min(int(r["n_undecided"]), ucap)
    return dict(report={k: int(r[k]) for k in REPORT_DTYPE.names},
                outliers=[(int(o["chunk"]), int(o["replica"])) for o in outl[:no]],
                undecided=[int(x) for x in und[:nu]],
                replica_bad=[int(x) for x in bad], rc=rc)
