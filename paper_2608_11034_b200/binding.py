"""Thin ctypes binding of libscout_b200.so: argument marshalling only.

Every ``scout_*`` function below has the name and argument order of its C
declaration in ``include/scout.h``; addresses are plain integers
(``tensor.data_ptr()``), streams are ``cudaStream_t`` handles as integers
(``torch.cuda.current_stream().cuda_stream``).  ``Plan`` is a small convenience
wrapper that keeps the marshalled arrays alive.  There is no fallback: if the
library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# SCOUT_LIB selects another build of the same library (e.g. other compile-time settings)
LIB_PATH = os.environ.get("SCOUT_LIB") or os.path.join(_HERE, "libscout_b200.so")

OK, ERR_INVALID, ERR_ALIGN, ERR_UNSUPPORTED, ERR_CUDA, ERR_NOMEM, ERR_TRUNCATED = 0, -1, -2, -3, -4, -5, -6
DT_U8, DT_F32, DT_BF16, DT_I64, DT_F16, DT_F64, DT_I32 = range(7)
AGREE, ATTRIBUTED, INCONCLUSIVE = 0, 1, 2
CERTIFIED, VERDICT_ATTRIBUTED, UNDECIDED = 0, 1, 2
MAX_REPLICAS = 1024          # SCOUT_MAX_REPLICAS of scout.h
DTYPE_CODE = {"u8": DT_U8, "f32": DT_F32, "bf16": DT_BF16, "i64": DT_I64, "f16": DT_F16,
              "f64": DT_F64, "i32": DT_I32}

SIG_DTYPE = np.dtype([("hash", "<u8"), ("nan_count", "<u4"), ("inf_count", "<u4"),
                      ("sum", "<f8"), ("sumsq", "<f8")])
TENSOR_DTYPE = np.dtype([("nbytes", "<u8"), ("dtype", "<u4"), ("reserved", "<u4"),
                         ("meta_tag", "<u8")])
OUTLIER_DTYPE = np.dtype([("chunk", "<u8"), ("replica", "<u4"), ("reserved", "<u4")])
REPORT_DTYPE = np.dtype([("n_chunks", "<u8"), ("n_agree", "<u8"), ("n_attributed", "<u8"),
                         ("n_inconclusive", "<u8"), ("n_outliers", "<u8"),
                         ("n_undecided", "<u8"), ("replica_union_bitmap", "<u8"),
                         ("certificate", "<u8"), ("verdict", "<i4"), ("reserved", "<i4")])

_lib = None


class ScoutError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().scout_strerror(code).decode()
        if code == ERR_CUDA:
            msg += " [" + lib().scout_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {msg} ({code})")


def lib():
    """Load the C-ABI library; raise loudly if it is missing (no CPU fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH) and not os.environ.get("SCOUT_LIB"):
            try:                      # a source checkout: compile the library once, in-tree
                from . import build as _build
                _build.build()
            except Exception as e:    # noqa: BLE001
                raise RuntimeError(
                    f"{LIB_PATH} is missing and could not be built ({e!r}): run "
                    "`python -m paper_2608_11034_b200.build` (needs nvcc); this package has no "
                    "CPU fallback") from e
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing; this package has no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, u64, u32, i64 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int64
        sigs = {
            "scout_plan_create": (C.c_int, [u32, u64, vp, u64, C.POINTER(vp)]),
            "scout_plan_bind": (C.c_int, [vp, vp]),
            "scout_plan_num_chunks": (C.c_int, [vp, C.POINTER(u64)]),
            "scout_plan_chunk_info": (C.c_int, [vp, u64, C.POINTER(u64), C.POINTER(u64),
                                                C.POINTER(u64), C.POINTER(u64)]),
            "scout_plan_destroy": (C.c_int, [vp]),
            "scout_sign_chunks": (C.c_int, [vp, vp, vp]),
            "scout_consensus_vote": (C.c_int, [u32, u64, vp, vp, vp, vp, u64, vp, u64, vp, vp]),
            "scout_consensus_vote_wide": (C.c_int, [u32, u64, vp, u64, u64, vp, vp, vp, u64, vp, u64, vp, vp]),
            "scout_certify": (C.c_int, [vp, vp, vp, vp, u64, vp, u64]),
            "scout_noalloc_guards_ok": (C.c_int, [vp]),
            "scout_certify_launch": (C.c_int, [vp, vp, u64, u64]),
            "scout_certify_collect": (C.c_int, [vp, vp, vp, u64, vp, u64]),
            "scout_plan_results": (C.c_int, [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]),
            "scout_plan_replica_bad_counts": (C.c_int, [vp, vp]),
            "scout_rollup_tensors": (C.c_int, [vp, vp, vp, vp]),
            "scout_certify_host": (C.c_int, [vp, vp, vp, vp, u64, vp, u64]),
            "scout_sign_chunks_noalloc": (C.c_int, [u32, vp, u64, u32, u64, u64, vp, vp]),
            "scout_shape_tag": (u64, [u32, vp]),
            "scout_plan_set": (C.c_int, [vp, C.c_char_p, i64]),
            "scout_plan_get": (C.c_int, [vp, C.c_char_p, C.POINTER(i64)]),
            "scout_ledger_create": (C.c_int, [u32, C.POINTER(vp)]),
            "scout_ledger_destroy": (C.c_int, [vp]),
            "scout_ledger_state": (C.c_int, [vp, vp]),
            "scout_ledger_save": (C.c_int, [vp, C.c_int, u64, C.c_int, C.c_int, vp]),
            "scout_ledger_retrieve": (C.c_int, [vp, C.c_int, C.c_int, C.c_int, vp]),
            "scout_outcome_from_report": (C.c_int, [vp, C.POINTER(C.c_int)]),
            "scout_mesh_size": (C.c_int, [vp, C.POINTER(u64)]),
            "scout_mesh_coords": (C.c_int, [vp, u64, vp]),
            "scout_mesh_rank": (C.c_int, [vp, vp, C.POINTER(u64)]),
            "scout_peer_group": (C.c_int, [vp, u64, vp, u64, C.POINTER(u64), C.POINTER(C.c_int)]),
            "scout_consensus_timing": (C.c_int, [u32, u64, vp, C.c_double, vp, vp, vp, vp, vp]),
            "scout_rotating_slice": (C.c_int, [u64, u64, u64, C.POINTER(u64), C.POINTER(u64)]),
            "scout_selftest_bounded_wait": (C.c_int, [u64, vp, vp]),
            "scout_strerror": (C.c_char_p, [C.c_int]),
            "scout_version": (C.c_int, []),
            "scout_last_cuda_error": (C.c_char_p, []),
        }
        for name, (res, args) in sigs.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(rc: int, where: str, allow=()) -> int:
    if rc != OK and rc not in allow:
        raise ScoutError(rc, where)
    return rc


# ---- one function per C entry point (same names) ------------------------------

def scout_shape_tag(dims: Sequence[int]) -> int:
    d = np.asarray(list(dims), dtype=np.uint64)
    return int(lib().scout_shape_tag(len(d), d.ctypes.data))


def scout_plan_create(R: int, tensors: np.ndarray, chunk_bytes: int) -> int:
    """tensors: numpy array of TENSOR_DTYPE.  Returns the plan handle."""
    assert tensors.dtype == TENSOR_DTYPE
    t = np.ascontiguousarray(tensors)
    out = C.c_void_p()
    _check(lib().scout_plan_create(R, len(t), t.ctypes.data, chunk_bytes, C.byref(out)),
           "scout_plan_create")
    return out.value


def scout_plan_bind(plan: int, ptrs: Sequence[int]) -> None:
    a = np.asarray(list(ptrs), dtype=np.uint64)
    _check(lib().scout_plan_bind(plan, a.ctypes.data), "scout_plan_bind")


def scout_plan_num_chunks(plan: int) -> int:
    n = C.c_uint64()
    _check(lib().scout_plan_num_chunks(plan, C.byref(n)), "scout_plan_num_chunks")
    return n.value


def scout_plan_chunk_info(plan: int, c: int):
    """-> (tensor, index_in_tensor, byte_offset, nbytes)"""
    a, b, d, e = C.c_uint64(), C.c_uint64(), C.c_uint64(), C.c_uint64()
    _check(lib().scout_plan_chunk_info(plan, c, C.byref(a), C.byref(b), C.byref(d), C.byref(e)),
           "scout_plan_chunk_info")
    return a.value, b.value, d.value, e.value


def scout_plan_destroy(plan: int) -> None:
    _check(lib().scout_plan_destroy(plan), "scout_plan_destroy")


def scout_plan_set(plan: int, key: str, value: int) -> None:
    _check(lib().scout_plan_set(plan, key.encode(), value), "scout_plan_set(%s)" % key)


def scout_plan_get(plan: int, key: str) -> int:
    v = C.c_int64()
    _check(lib().scout_plan_get(plan, key.encode(), C.byref(v)), "scout_plan_get(%s)" % key)
    return v.value


def scout_sign_chunks(plan: int, stream: int, d_sigs: int) -> None:
    _check(lib().scout_sign_chunks(plan, stream, d_sigs), "scout_sign_chunks")


def scout_consensus_vote(R: int, n_chunks: int, d_sigs: int, d_status: int, d_bitmap: int,
                         d_outliers: int, outlier_cap: int, d_undecided: int, undecided_cap: int,
                         d_counts: int, stream: int) -> None:
    _check(lib().scout_consensus_vote(R, n_chunks, d_sigs, d_status, d_bitmap, d_outliers,
                                      outlier_cap, d_undecided, undecided_cap, d_counts, stream),
           "scout_consensus_vote")


_certify_buffers = {}


def scout_consensus_vote_wide(R: int, n_chunks: int, d_sigs: int, chunk_stride: int,
                              replica_stride: int, d_status: int, d_bitmap: int, d_outliers: int,
                              outlier_cap: int, d_undecided: int, undecided_cap: int, d_counts: int,
                              stream: int) -> None:
    _check(lib().scout_consensus_vote_wide(R, n_chunks, d_sigs, chunk_stride, replica_stride, d_status,
                                           d_bitmap, d_outliers, outlier_cap, d_undecided,
                                           undecided_cap, d_counts, stream),
           "scout_consensus_vote_wide")


def _certify_common(fn, name, plan, second, outlier_cap, undecided_cap):
    key = (outlier_cap, undecided_cap)
    if key not in _certify_buffers:      # host landing buffers, reused between calls
        _certify_buffers[key] = (np.zeros(1, dtype=REPORT_DTYPE),
                                 np.zeros(max(outlier_cap, 1), dtype=OUTLIER_DTYPE),
                                 np.zeros(max(undecided_cap, 1), dtype=np.uint64))
    rep, outl, und = _certify_buffers[key]
    rc = _check(fn(plan, second, rep.ctypes.data, outl.ctypes.data, outlier_cap, und.ctypes.data,
                   undecided_cap), name, allow=(ERR_TRUNCATED,))
    r = {k: int(rep[0][k]) for k in REPORT_DTYPE.names}
    no, nu = min(r["n_outliers"], outlier_cap), min(r["n_undecided"], undecided_cap)
    return dict(report=r, outliers=[(int(o["chunk"]), int(o["replica"])) for o in outl[:no]],
                undecided=[int(x) for x in und[:nu]], rc=rc)


def scout_certify(plan: int, stream: int, outlier_cap: int = 4096, undecided_cap: int = 4096):
    """-> dict(report, outliers [(chunk, replica)] sorted, undecided sorted, rc)"""
    return _certify_common(lib().scout_certify, "scout_certify", plan, stream, outlier_cap,
                           undecided_cap)


def scout_certify_launch(plan: int, stream: int, outlier_cap: int = 4096, undecided_cap: int = 4096) -> None:
    """Enqueue one certify run on `stream` and return; scout_certify_collect finishes it."""
    _check(lib().scout_certify_launch(plan, stream, outlier_cap, undecided_cap), "scout_certify_launch")


def scout_certify_collect(plan: int, outlier_cap: int = 4096, undecided_cap: int = 4096):
    """Wait for the launched run.  -> the same dict as scout_certify."""
    fn = lib().scout_certify_collect
    return _certify_common(lambda pl, _unused, *rest: fn(pl, *rest), "scout_certify_collect", plan, None,
                           outlier_cap, undecided_cap)


def scout_certify_host(plan: int, h_ptrs: Sequence[int], outlier_cap: int = 4096,
                       undecided_cap: int = 4096):
    a = np.asarray(list(h_ptrs), dtype=np.uint64)
    return _certify_common(lib().scout_certify_host, "scout_certify_host", plan, a.ctypes.data,
                           outlier_cap, undecided_cap)


def scout_plan_results(plan: int):
    """-> device addresses (d_sigs, d_status, d_bitmap) of the last certify run"""
    a, b, d = C.c_void_p(), C.c_void_p(), C.c_void_p()
    _check(lib().scout_plan_results(plan, C.byref(a), C.byref(b), C.byref(d)), "scout_plan_results")
    return a.value, b.value, d.value


def scout_plan_replica_bad_counts(plan: int, R: int) -> List[int]:
    out = np.zeros(R, dtype=np.uint64)
    _check(lib().scout_plan_replica_bad_counts(plan, out.ctypes.data), "scout_plan_replica_bad_counts")
    return [int(x) for x in out]


def scout_rollup_tensors(plan: int, d_sigs: int, d_tensor_sigs: int, stream: int) -> None:
    _check(lib().scout_rollup_tensors(plan, d_sigs, d_tensor_sigs, stream), "scout_rollup_tensors")


def scout_sign_chunks_noalloc(R: int, replica_ptrs: Sequence[int], nbytes: int, dtype: int,
                              meta_tag: int, chunk_bytes: int, d_sigs: int, stream: int) -> None:
    """Sign R one-tensor replicas without allocating anything (see scout.h for
    who needs this and for the size limit).  d_sigs: device [C][R] records."""
    a = np.asarray(list(replica_ptrs), dtype=np.uint64)
    _check(lib().scout_sign_chunks_noalloc(R, a.ctypes.data, nbytes, dtype, meta_tag, chunk_bytes,
                                           d_sigs, stream), "scout_sign_chunks_noalloc")


def scout_noalloc_guards_ok() -> bool:
    """True if nothing wrote outside the no-allocation entry point's fixed array (synchronises)."""
    ok = C.c_int(0)
    _check(lib().scout_noalloc_guards_ok(C.byref(ok)), "scout_noalloc_guards_ok")
    return bool(ok.value)


def scout_consensus_timing(N: int, G: int, d_times: int, kappa: float, d_status: int,
                           d_bitmap: int, d_median: int, d_scale: int, stream: int) -> None:
    _check(lib().scout_consensus_timing(N, G, d_times, kappa, d_status, d_bitmap, d_median,
                                        d_scale, stream), "scout_consensus_timing")


# ---- host-only entry points: checkpoint ledger, peer groups -----------------------

OUTCOME_HEALTHY, OUTCOME_STRAGGLER, OUTCOME_SDC, OUTCOME_HANG, OUTCOME_OTHER = range(5)
ROLE_NONE, ROLE_LATEST, ROLE_CANDIDATE, ROLE_VERIFIED = range(4)
LEDGER_CAPTURED, LEDGER_BOUNDARY, LEDGER_RETRIEVAL, LEDGER_NEED_SWEEP = range(4)
NO_CHECKPOINT = 2**64 - 1
GROUP_NONE, GROUP_REPLICA, GROUP_SHARD = range(3)
LEDGER_STATE_DTYPE = np.dtype([("latest", "<u8"), ("candidate", "<u8"), ("verified", "<u8"),
                               ("q", "<u4"), ("K", "<u4"), ("n_persisted", "<u8")])
LEDGER_EVENT_DTYPE = np.dtype([("action", "<i4"), ("role", "<i4"), ("checkpoint", "<u8"),
                               ("promoted", "<u8")])
MESH_DTYPE = np.dtype([(k, "<u4") for k in "dstpce"])


def scout_ledger_create(K: int) -> int:
    out = C.c_void_p()
    _check(lib().scout_ledger_create(K, C.byref(out)), "scout_ledger_create")
    return out.value


def scout_ledger_destroy(ledger: int) -> None:
    _check(lib().scout_ledger_destroy(ledger), "scout_ledger_destroy")


def scout_ledger_state(ledger: int) -> dict:
    st = np.zeros(1, dtype=LEDGER_STATE_DTYPE)
    _check(lib().scout_ledger_state(ledger, st.ctypes.data), "scout_ledger_state")
    return {k: int(st[0][k]) for k in LEDGER_STATE_DTYPE.names}


def _event(ev) -> dict:
    return {k: int(ev[0][k]) for k in LEDGER_EVENT_DTYPE.names}


def scout_ledger_save(ledger: int, outcome: int, captured: int, machines_accessible: bool = True,
                      sweep_has_sdc: int = -1) -> dict:
    ev = np.zeros(1, dtype=LEDGER_EVENT_DTYPE)
    _check(lib().scout_ledger_save(ledger, outcome, captured, int(machines_accessible),
                                   sweep_has_sdc, ev.ctypes.data), "scout_ledger_save")
    return _event(ev)


def scout_ledger_retrieve(ledger: int, failure: int, machines_accessible: bool = True,
                          sweep_has_sdc: int = -1) -> dict:
    ev = np.zeros(1, dtype=LEDGER_EVENT_DTYPE)
    _check(lib().scout_ledger_retrieve(ledger, failure, int(machines_accessible), sweep_has_sdc,
                                       ev.ctypes.data), "scout_ledger_retrieve")
    return _event(ev)


def scout_outcome_from_report(report: dict) -> int:
    rep = np.zeros(1, dtype=REPORT_DTYPE)
    for k in REPORT_DTYPE.names:
        rep[0][k] = report[k]
    out = C.c_int()
    _check(lib().scout_outcome_from_report(rep.ctypes.data, C.byref(out)), "scout_outcome_from_report")
    return out.value


def _mesh(shape) -> np.ndarray:
    m = np.zeros(1, dtype=MESH_DTYPE)
    m[0] = tuple(shape)
    return m


def scout_mesh_size(shape) -> int:
    n, m = C.c_uint64(), _mesh(shape)
    _check(lib().scout_mesh_size(m.ctypes.data, C.byref(n)), "scout_mesh_size")
    return n.value


def scout_mesh_coords(shape, rank: int):
    out, m = np.zeros(1, dtype=MESH_DTYPE), _mesh(shape)
    _check(lib().scout_mesh_coords(m.ctypes.data, rank, out.ctypes.data), "scout_mesh_coords")
    return tuple(int(out[0][k]) for k in "dstpce")


def scout_mesh_rank(shape, coords) -> int:
    r, m, at = C.c_uint64(), _mesh(shape), _mesh(coords)
    _check(lib().scout_mesh_rank(m.ctypes.data, at.ctypes.data, C.byref(r)), "scout_mesh_rank")
    return r.value


def scout_peer_group(shape, rank: int, cap: int = 4096):
    """-> (kind, peers) with peers in bitmap order"""
    peers = np.zeros(max(cap, 1), dtype=np.uint64)
    n, kind, m = C.c_uint64(), C.c_int(), _mesh(shape)
    _check(lib().scout_peer_group(m.ctypes.data, rank, peers.ctypes.data, cap, C.byref(n),
                                  C.byref(kind)), "scout_peer_group", allow=(ERR_TRUNCATED,))
    return kind.value, [int(x) for x in peers[:min(n.value, cap)]]


def scout_rotating_slice(numel: int, slice_elems: int, step: int):
    """-> (begin, count) of the window checked at this step"""
    b, n = C.c_uint64(), C.c_uint64()
    _check(lib().scout_rotating_slice(numel, slice_elems, step, C.byref(b), C.byref(n)),
           "scout_rotating_slice")
    return b.value, n.value


def scout_selftest_bounded_wait(limit_ns: int, d_out: int, stream: int) -> None:
    _check(lib().scout_selftest_bounded_wait(limit_ns, d_out, stream), "scout_selftest_bounded_wait")


def scout_version() -> int:
    return int(lib().scout_version())


# ---- convenience wrapper (device memory and streams come from torch) ------------

def make_tensor_table(specs, tags: Optional[Sequence[int]] = None) -> np.ndarray:
    """specs: objects with .nbytes, .dtype (key of DTYPE_CODE) and .shape."""
    t = np.zeros(len(specs), dtype=TENSOR_DTYPE)
    for i, s in enumerate(specs):
        tag = scout_shape_tag(list(s.shape)) if tags is None else tags[i]
        t[i] = (s.nbytes, DTYPE_CODE[s.dtype], 0, tag)
    return t


class Plan:
    """Owns a scout plan plus torch-allocated output buffers for sign and vote."""

    GUARD_BYTES = 256
    GUARD_PATTERN = 0x5A

    def __init__(self, R: int, tensor_table: np.ndarray, chunk_bytes: int, guards: bool = False):
        """guards: allocate every output buffer between two 256-byte bands of a fixed pattern;
        check_guards() then tells whether a kernel wrote outside any of them."""
        import torch
        self._torch = torch
        self._guards = guards
        self._outer = []
        self.R, self.T = R, len(tensor_table)
        self.handle = scout_plan_create(R, tensor_table, chunk_bytes)
        self.C = scout_plan_num_chunks(self.handle)
        self._keep = None
        self.d_sigs = None

    def close(self):
        if getattr(self, "handle", None):
            scout_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:       # interpreter shutdown: module globals may be gone
            pass

    def bind(self, views) -> None:
        """views[r][t]: torch CUDA tensors (kept alive by the plan)."""
        self._keep = views
        scout_plan_bind(self.handle, [v.data_ptr() for rep in views for v in rep])

    def chunk_table(self) -> np.ndarray:
        out = np.zeros(self.C, dtype=[("tensor", "<u8"), ("index_in_tensor", "<u8"),
                                      ("byte_offset", "<u8"), ("nbytes", "<u8")])
        for c in range(self.C):
            out[c] = scout_plan_chunk_info(self.handle, c)
        return out

    def _buffer(self, numel: int, dtype):
        """A device buffer of `numel` elements; with guards, the middle of a larger one."""
        torch = self._torch
        if not self._guards:
            return torch.empty(numel, dtype=dtype, device="cuda")
        nbytes = numel * torch.empty(0, dtype=dtype).element_size()
        g = self.GUARD_BYTES
        outer = torch.full((nbytes + 2 * g,), self.GUARD_PATTERN, dtype=torch.uint8, device="cuda")
        self._outer.append((outer, nbytes))
        return outer[g:g + nbytes].view(dtype)

    def check_guards(self) -> bool:
        """True if no byte of any guard band has changed (synchronises)."""
        g = self.GUARD_BYTES
        self._torch.cuda.synchronize()
        for outer, nbytes in self._outer:
            if not bool((outer[:g] == self.GUARD_PATTERN).all()) or \
                    not bool((outer[g + nbytes:] == self.GUARD_PATTERN).all()):
                return False
        return True

    def _alloc(self, outlier_cap, undecided_cap):
        torch = self._torch
        if self.d_sigs is None:
            self.d_sigs = self._buffer(self.C * self.R * 32, torch.uint8)
            self.d_status = self._buffer(max(self.C, 1), torch.uint8)
            self.d_bitmap = self._buffer(max(self.C, 1), torch.int64)
            self.d_counts = self._buffer(6, torch.int64)
        if getattr(self, "_ocap", -1) < outlier_cap:
            self.d_outliers = self._buffer(max(outlier_cap, 1) * 16, torch.uint8)
            self._ocap = outlier_cap
        if getattr(self, "_ucap", -1) < undecided_cap:
            self.d_undecided = self._buffer(max(undecided_cap, 1), torch.int64)
            self._ucap = undecided_cap

    def sign(self, stream: Optional[int] = None) -> None:
        self._alloc(0, 0)
        s = self._torch.cuda.current_stream().cuda_stream if stream is None else stream
        scout_sign_chunks(self.handle, s, self.d_sigs.data_ptr())

    def vote(self, outlier_cap: int = 4096, undecided_cap: int = 4096, stream: Optional[int] = None) -> None:
        self._alloc(outlier_cap, undecided_cap)
        s = self._torch.cuda.current_stream().cuda_stream if stream is None else stream
        scout_consensus_vote(self.R, self.C, self.d_sigs.data_ptr(), self.d_status.data_ptr(),
                             self.d_bitmap.data_ptr(), self.d_outliers.data_ptr(), outlier_cap,
                             self.d_undecided.data_ptr(), undecided_cap, self.d_counts.data_ptr(), s)
        self._caps = (outlier_cap, undecided_cap)

    def sign_and_vote(self, outlier_cap: int = 4096, undecided_cap: int = 4096) -> None:
        self._alloc(outlier_cap, undecided_cap)
        self.sign()
        self.vote(outlier_cap, undecided_cap)

    def fetch(self):
        """Synchronise and copy the results of sign()/vote() to host numpy."""
        torch = self._torch
        torch.cuda.synchronize()
        sigs = self.d_sigs.cpu().numpy().view(SIG_DTYPE).reshape(self.C, self.R)
        counts = [int(x) for x in self.d_counts.cpu().numpy()]
        ocap, ucap = self._caps
        no, nu = min(counts[4], ocap), min(counts[5], ucap)
        outl = self.d_outliers.cpu().numpy().view(OUTLIER_DTYPE)[:no]
        und = self.d_undecided.cpu().numpy().view(np.uint64)[:nu]
        return dict(sigs=sigs, status=self.d_status.cpu().numpy()[:self.C],
                    bitmap=self.d_bitmap.cpu().numpy().view(np.uint64)[:self.C], counts=counts,
                    outliers=sorted((int(o["chunk"]), int(o["replica"])) for o in outl),
                    undecided=sorted(int(x) for x in und))

    def certify(self, outlier_cap: int = 4096, undecided_cap: int = 4096, stream: Optional[int] = None):
        s = self._torch.cuda.current_stream().cuda_stream if stream is None else stream
        return scout_certify(self.handle, s, outlier_cap, undecided_cap)

    def certify_launch(self, outlier_cap: int = 4096, undecided_cap: int = 4096,
                       stream: Optional[int] = None) -> None:
        s = self._torch.cuda.current_stream().cuda_stream if stream is None else stream
        scout_certify_launch(self.handle, s, outlier_cap, undecided_cap)

    def certify_collect(self, outlier_cap: int = 4096, undecided_cap: int = 4096):
        return scout_certify_collect(self.handle, outlier_cap, undecided_cap)
