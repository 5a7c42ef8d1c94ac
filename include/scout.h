/*
 * scout.h - C ABI of the B200 (sm_100a) sign+vote library.
 *
 * The data-parallel hot path of Consensus Collective Communication (C3):
 * a compact signature for every chunk of R equivalent replicas' tensors, then
 * strict-majority voting over the signatures to name the outlier replicas and
 * the chunks they corrupt.  R replicas are R sets of buffers in one GPU's
 * memory.
 *
 * Conventions
 *   - plain C; every function returns int: SCOUT_OK (0) or a negative error;
 *     nothing throws, aborts or takes ownership of caller memory;
 *   - "device" pointers are CUDA device addresses valid on the current device,
 *     "host" pointers are ordinary host memory;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream);
 *     work is enqueued there and, except for scout_certify, the call returns
 *     without waiting for it;
 *   - the library allocates device memory only inside a plan object;
 *   - the replica index is the position in the caller's pointer table: this is
 *     the ordered peer-to-rank map that C3 stores with its result (Sec. 5.1).
 */
#ifndef SCOUT_H
#define SCOUT_H

#include <stdint.h>

#if defined(__GNUC__)
#define SCOUT_API __attribute__((visibility("default")))
#else
#define SCOUT_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SCOUT_OK = 0,
    SCOUT_ERR_INVALID = -1,     /* bad argument (NULL, R out of range, size 0, ...)     */
    SCOUT_ERR_ALIGN = -2,       /* a tensor address is not 16-byte aligned              */
    SCOUT_ERR_UNSUPPORTED = -3, /* valid request this build does not implement (R > 64) */
    SCOUT_ERR_CUDA = -4,        /* a CUDA runtime call failed; see scout_last_cuda_error */
    SCOUT_ERR_NOMEM = -5,       /* host or device allocation failed                     */
    SCOUT_ERR_TRUNCATED = -6    /* a result list was shorter than needed; counters hold
                                   the true totals, entries beyond capacity were dropped */
};

/* Element types.  The code enters the signature (the evidence covers the dtype,
 * Sec. 5.2), so the numbering is frozen. */
enum {
    SCOUT_DT_U8 = 0, SCOUT_DT_F32 = 1, SCOUT_DT_BF16 = 2, SCOUT_DT_I64 = 3,
    SCOUT_DT_F16 = 4, SCOUT_DT_F64 = 5, SCOUT_DT_I32 = 6
};

/* The three statuses of a C3 result (Sec. 5.1): they keep an all-zero bitmap
 * from being ambiguous. */
enum { SCOUT_AGREE = 0, SCOUT_ATTRIBUTED = 1, SCOUT_INCONCLUSIVE = 2 };

/* Verdict of scout_certify over a whole replicated state. */
enum { SCOUT_CERTIFIED = 0, SCOUT_VERDICT_ATTRIBUTED = 1, SCOUT_UNDECIDED = 2 };

#define SCOUT_MAX_REPLICAS 1024 /* signing and scout_consensus_vote_wide; one-word bitmaps stop at 64 */

typedef struct scout_plan scout_plan_t; /* opaque; owns its device tables and scratch */

/* Comparable evidence of one (chunk, replica) (Sec. 5.2).  Only `hash` is
 * compared by the vote; the other fields are a diagnostic sidecar. */
typedef struct {
    uint64_t hash;      /* 64-bit position-sensitive signature of dtype, shape tag, bytes */
    uint32_t nan_count; /* elements that are NaN (0 for integer types)                   */
    uint32_t inf_count; /* elements that are +-Inf                                       */
    double sum;         /* sum of the finite elements                                    */
    double sumsq;       /* sum of squares of the finite elements                         */
} scout_sig_t;          /* 32 bytes */

typedef struct {
    uint64_t nbytes;   /* > 0, a multiple of the element size                  */
    uint32_t dtype;    /* SCOUT_DT_*                                            */
    uint32_t reserved; /* must be 0                                             */
    uint64_t meta_tag; /* caller's shape tag (scout_shape_tag), 0 allowed       */
} scout_tensor_t;

typedef struct {
    uint64_t chunk;    /* global chunk id                                       */
    uint32_t replica;  /* index of the outlier replica                          */
    uint32_t reserved;
} scout_outlier_t;     /* 16 bytes */

typedef struct {
    uint64_t n_chunks, n_agree, n_attributed, n_inconclusive;
    uint64_t n_outliers, n_undecided; /* true totals even if a list was truncated   */
    uint64_t replica_union_bitmap;    /* OR of every chunk's outlier bitmap          */
    uint64_t certificate;             /* digest of the majority hashes; 0 if UNDECIDED */
    int32_t verdict;                  /* SCOUT_CERTIFIED / _VERDICT_ATTRIBUTED / _UNDECIDED */
    int32_t reserved;
} scout_report_t;

/* ---- plan: chunking ------------------------------------------------------
 * Cuts every tensor into pieces of `chunk_bytes` (the last piece short; pieces
 * never span tensors).  The global chunk id runs over (tensor, piece).  The
 * chunk is this library's unit of evidence: C3 is applied once per chunk, so a
 * disagreement is localised to (replica, chunk) instead of (replica, tensor)
 * as in Sec. 5.2.
 *   R            number of replicas bound to this plan, 1..SCOUT_MAX_REPLICAS.
 *                2..64: everything.  65..1024: scout_sign_chunks and
 *                scout_consensus_vote_wide (multi-word bitmaps; the paper's peer
 *                groups reach degree 192); scout_certify returns
 *                SCOUT_ERR_UNSUPPORTED.  1: signing only - the local step when
 *                every GPU holds one replica and the records are gathered
 *                afterwards; a singleton has no comparison (Sec. 4 "Peer-group
 *                size"), so voting or certifying with R < 2 is SCOUT_ERR_INVALID.
 *   T, tensors   host array of T descriptors, copied
 *   chunk_bytes  a multiple of 512, at most 1 GiB
 *   out          receives the plan; destroy with scout_plan_destroy
 * Allocates the device tables and the per-tile scratch on the current device. */
SCOUT_API int scout_plan_create(uint32_t R, uint64_t T, const scout_tensor_t *tensors /*host*/,
                      uint64_t chunk_bytes, scout_plan_t **out);

/* ptrs: host array of R*T device addresses, replica-major (ptrs[r*T + t] is
 * tensor t of replica r), each 16-byte aligned (else SCOUT_ERR_ALIGN) and
 * readable for tensors[t].nbytes.  The buffers stay the caller's.  May be
 * called again to scan other buffers of the same geometry: the call first waits
 * (on the host) until the plan's most recent sign or certify has finished on
 * whatever stream it was given, so a scan in flight never sees the table change
 * under it, then copies the table synchronously.
 *
 * Every call that takes a plan must be made with the plan's device current (the
 * device that was current in scout_plan_create); with another device current it
 * returns SCOUT_ERR_INVALID and launches nothing. */
SCOUT_API int scout_plan_bind(scout_plan_t *plan, const void *const *ptrs /*host*/);

SCOUT_API int scout_plan_num_chunks(const scout_plan_t *plan, uint64_t *C);
SCOUT_API int scout_plan_chunk_info(const scout_plan_t *plan, uint64_t c, uint64_t *tensor,
                          uint64_t *index_in_tensor, uint64_t *byte_offset, uint64_t *nbytes);
SCOUT_API int scout_plan_destroy(scout_plan_t *plan);

/* ---- comparable evidence (Sec. 5.2: e_i = H_w(dtype, shape, bytes)) -------
 * Reads every byte of every bound replica once and writes one record per
 * (chunk, replica) to d_sigs[c*R + r] (device, C*R records).  The bulk fold and
 * the finalisation both run on the device (Sec. 9 folds on the device and
 * finalises on the host; here only the records leave the kernel).
 * Asynchronous on `stream`.  Results are bitwise reproducible for a given plan. */
SCOUT_API int scout_sign_chunks(scout_plan_t *plan, void *stream, scout_sig_t *d_sigs /*device [C][R]*/);

/* ---- exact consensus (Sec. 5.3; Algorithm 1, Exact branch) ----------------
 * Per chunk: the most frequent hash e* and its count c*.  If c* <= R/2 the
 * chunk is SCOUT_INCONCLUSIVE with bitmap 0 and its id is appended to
 * d_undecided; otherwise bit j of the bitmap is 1{e_j != e*}, the status is
 * SCOUT_ATTRIBUTED if any bit is set, else SCOUT_AGREE, and (chunk, j) is
 * appended to d_outliers for every set bit.
 *   d_sigs                   device [C][R] records (only .hash is compared)
 *   d_status, d_bitmap       device [C]; either may be NULL
 *   d_outliers, d_undecided  device lists of the given capacities (NULL with
 *                            capacity 0 allowed); entries are in no particular
 *                            order; entries beyond capacity are dropped
 *   d_counts                 device [6]: n_chunks, n_agree, n_attributed,
 *                            n_inconclusive, n_outliers, n_undecided (true totals)
 * Asynchronous on `stream`; overflow of a list is visible as count > capacity. */
SCOUT_API int scout_consensus_vote(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint8_t *d_status,
                         uint64_t *d_bitmap, scout_outlier_t *d_outliers, uint64_t outlier_cap,
                         uint64_t *d_undecided, uint64_t undecided_cap, uint64_t *d_counts,
                         void *stream);

/* The same rule for groups of up to SCOUT_MAX_REPLICAS peers and for records that
 * were gathered from one GPU per replica.  The record of (chunk c, replica r) is
 * d_sigs[c * chunk_stride + r * replica_stride] (strides in records):
 * (R, 1) is the chunk-major table scout_sign_chunks writes; (1, C) is the
 * rank-major table an AllGather of per-rank [C] records produces (Algorithm 1
 * line 2), so no transposition is needed.  d_bitmap: device [C][W] words with
 * W = ceil(R / 64), bit (r mod 64) of word (r / 64) for replica r; may be NULL.
 * Everything else as in scout_consensus_vote. */
SCOUT_API int scout_consensus_vote_wide(uint32_t R, uint64_t C, const scout_sig_t *d_sigs,
                                        uint64_t chunk_stride, uint64_t replica_stride,
                                        uint8_t *d_status, uint64_t *d_bitmap,
                                        scout_outlier_t *d_outliers, uint64_t outlier_cap,
                                        uint64_t *d_undecided, uint64_t undecided_cap,
                                        uint64_t *d_counts, void *stream);

/* ---- certify a replicated state -------------------------------------------
 * sign + vote + roll-up over everything bound to the plan (the optimizer-
 * boundary comparison of Sec. 9 extended from a sampled slice to the full
 * state; a checkpoint is worth promoting only if its replicas agree, Sec. 8).
 * Synchronises `stream`.  Host lists come back sorted by (chunk, replica).
 * Returns SCOUT_ERR_TRUNCATED (report still valid) if a list was too short.
 *   verdict CERTIFIED   every chunk agrees
 *           ATTRIBUTED  every chunk has a strict majority; replica_union_bitmap
 *                       names the bad replicas, the others are certified
 *           UNDECIDED   at least one chunk has no strict majority; no certificate */
SCOUT_API int scout_certify(scout_plan_t *plan, void *stream, scout_report_t *report /*host*/,
                  scout_outlier_t *h_outliers /*host*/, uint64_t outlier_cap,
                  uint64_t *h_undecided /*host*/, uint64_t undecided_cap);

/* The same run in two halves, for callers that must not block where the check is
 * enqueued (C3 runs in the progress path of a training step, Sec. 9): the first
 * call enqueues everything on `stream` and returns; the second waits for it and
 * fills the report and the sorted lists exactly as scout_certify does.  The
 * lists are cut at the capacities given to the first call (the second call's
 * capacities may be smaller, not larger).  One run may be in flight per plan:
 * a second launch, or a scout_certify, before the collect is SCOUT_ERR_INVALID. */
SCOUT_API int scout_certify_launch(scout_plan_t *plan, void *stream, uint64_t outlier_cap,
                                   uint64_t undecided_cap);
SCOUT_API int scout_certify_collect(scout_plan_t *plan, scout_report_t *report /*host*/,
                                    scout_outlier_t *h_outliers /*host*/, uint64_t outlier_cap,
                                    uint64_t *h_undecided /*host*/, uint64_t undecided_cap);

/* After scout_certify: device pointers to the plan-owned results of that run
 * (valid until the next certify or destroy).  Any output may be NULL. */
SCOUT_API int scout_plan_results(const scout_plan_t *plan, const scout_sig_t **d_sigs,
                       const uint8_t **d_status, const uint64_t **d_bitmap);
/* After scout_certify: chunks attributed to each replica, host [R]. */
SCOUT_API int scout_plan_replica_bad_counts(const scout_plan_t *plan, uint64_t *h_counts /*host [R]*/);

/* Tensor-level signatures, the granularity of Sec. 5.2: for every (tensor,
 * replica) the chunk hashes folded in order.  d_sigs: device [C][R] records;
 * d_tensor_sigs: device [T][R].  Asynchronous on `stream`. */
SCOUT_API int scout_rollup_tensors(const scout_plan_t *plan, const scout_sig_t *d_sigs,
                         uint64_t *d_tensor_sigs /*device [T][R]*/, void *stream);

/* Same as scout_certify for replicas that live in HOST memory (checkpoints kept
 * in CPU memory, Sec. 8): h_ptrs is a host array of R*T host addresses,
 * replica-major.  The data is streamed through plan-owned device staging
 * buffers in slices, copy overlapped with signing.  Pinned host memory copies
 * faster; pageable memory works.  Synchronous. */
SCOUT_API int scout_certify_host(scout_plan_t *plan, const void *const *h_ptrs /*host*/,
                       scout_report_t *report /*host*/, scout_outlier_t *h_outliers,
                       uint64_t outlier_cap, uint64_t *h_undecided, uint64_t undecided_cap);

/* ---- signing without allocating ---------------------------------------------
 * (The paper has no counterpart: this entry point exists for deployment.)
 * For callers that must not allocate device memory while they run, for example
 * a check placed inside a training step whose framework already holds nearly
 * all of HBM in its own allocator (a cudaMalloc there can fail, and it stalls
 * the device), or a handler running right after an out-of-memory error.
 * No plan is needed and nothing is allocated or freed, on the device or through
 * any library: the per-tile partial records go to a fixed 2 MiB array inside
 * the library's device image (every GPU that loads the library holds it until
 * the process exits).
 *   R             replicas, 2..64
 *   replica_ptrs  host array of R device addresses, 16-byte aligned; replica r
 *                 is ONE contiguous tensor of `nbytes` bytes at replica_ptrs[r]
 *   nbytes, dtype, meta_tag, chunk_bytes   as in scout_tensor_t / scout_plan_create
 *   d_sigs        device, caller-allocated, [C][R] with C = ceil(nbytes / chunk_bytes);
 *                 same records as scout_sign_chunks for a one-tensor plan
 *                 (hashes and counts identical; the fp64 sums may differ in the
 *                 last bits because the tile size may differ)
 * Limit: R * (number of 64 KiB tiles) <= 65536 records, i.e. about 4 GiB of
 * replica data per call; more returns SCOUT_ERR_UNSUPPORTED and launches
 * nothing.  The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current) and is the first launch of
 * this entry point's two kernels, which makes the CUDA runtime load them; that
 * loading may itself take device memory.  So make one warm-up call per device
 * at start-up, while memory is still available and before any stream capture;
 * the calls after it allocate nothing.  All calls share the one array and every call
 * overwrites the records it reads, so nothing needs clearing between calls,
 * but two calls whose kernels overlap on the GPU (different streams, or several
 * host threads) race on it: serialise them.  Asynchronous on `stream`. */
SCOUT_API int scout_sign_chunks_noalloc(uint32_t R, const void *const *replica_ptrs /*host*/,
                                        uint64_t nbytes, uint32_t dtype, uint64_t meta_tag,
                                        uint64_t chunk_bytes, scout_sig_t *d_sigs /*device*/,
                                        void *stream);

/* Diagnostic for the fixed array of scout_sign_chunks_noalloc: the array lies between two
 * 256-byte guard bands that are filled with a pattern when a device is first used; *ok
 * becomes 1 if both bands still hold it on the current device, 0 if something wrote outside
 * the array.  Synchronises the device.  Allocates nothing. */
SCOUT_API int scout_noalloc_guards_ok(int *ok /*host*/);

/* Shape tag for scout_tensor_t.meta_tag: a 64-bit digest of (ndim, dims). */
SCOUT_API uint64_t scout_shape_tag(uint32_t ndim, const uint64_t *dims /*host*/);

/* Knobs of a plan (optional).
 *   set "tile_bytes"  bytes per work item, a power of two in [2048, 262144]
 *   set "variant"     scan kernel: 1 (default) = 16-byte loads through a rotating
 *                     register pipeline, eight rows always in flight, so that a warp's
 *                     loads overlap its own arithmetic; 0 = the same loads in batches
 *                     of eight rows without that overlap (the form the one-launch
 *                     kernels use); 2 = bulk-async
 *                     copies (cp.async.bulk + mbarrier) through a per-warp ring in
 *                     shared memory; 4 = block-wide ring: a producer warp fetches
 *                     whole tiles (<= 32 KiB) with one bulk copy each and eight
 *                     consumer warps share them (needs tile_bytes <= 32768);
 *                     3 = read-only probe (measures the memory system only: the
 *                     records it leaves are NOT signatures)
 *   set "fused"       with the default scan (variants 0 and 1) and R <= 64 a call can run as
 *                     ONE kernel, in one of two forms.  1 = tickets: the warp that stores
 *                     the last tile record of a chunk finalises it (scout_sign_chunks), and
 *                     for scout_certify also votes it and folds it into the certificate
 *                     chain; the warp that folds the last chunk writes the report block
 *                     to pinned host memory.  2 = clusters (R <= 8, at most 256 tiles per
 *                     chunk, else SCOUT_ERR_UNSUPPORTED): a thread-block cluster of R
 *                     CTAs takes a chunk, CTA r scans replica r's copy and keeps its
 *                     record in shared memory, the first CTA reads the R hashes through
 *                     distributed shared memory and votes; chunks of fewer than 16 tiles
 *                     are taken several at a time.  0 = never (one kernel per stage:
 *                     scan, finalise, vote, certificate - the form scout_certify_host
 *                     always uses).  -1 (default) = whichever measured fastest:
 *                     scout_certify on plans below 1 GiB (256 MiB for plans of 16-bit
 *                     floats) uses clusters when R <= 8, no chunk has more than 64 tiles
 *                     per CTA that shares it and there are at most 1,024 chunks (or one
 *                     per 300 KiB), tickets on other plans up to 16 MiB whose
 *                     chunks have at most 64 tiles; larger plans and scout_sign_chunks
 *                     run the stages as separate kernels
 *   get "certify_form", "sign_form"  the form (0, 1, 2 as above) scout_certify /
 *                     scout_sign_chunks would use for this plan now
 *   get "cluster_ok"  1 if form 2 can run this plan with its current tile size
 *   set "dynamic"     1 (default): the scan's warps take tiles from work counters as they
 *                     become free; 0: fixed round-robin assignment
 *   set "work_streams" 1..32 (default 8): how many counters the tiles are dealt from (one
 *                     counter serves about 0.3 G tiles per second, which plans of many
 *                     small tiles exceed)
 *   set "grid"        CTAs of the scan kernel
 *   set "timing"      1: record a pair of CUDA events around every scan kernel on
 *                     the caller's stream (a ring of 256 pairs); setting it again
 *                     restarts the count
 *   get "last_sign_ns" device time of the most recent scan kernel (needs
 *                     "timing" and a synchronised stream)
 *   get "timed_sign_launches", "timed_sign_ns"  number of scan launches since
 *                     "timing" was set that the ring still holds (at most 256) and
 *                     their total device time (synchronised stream)
 *   get "device_error" 1 if a kernel's bounded wait gave up since the flag was last
 *                     cleared (synchronises); the records of such a run are not
 *                     valid.  scout_certify and scout_certify_host report it as
 *                     SCOUT_ERR_CUDA once and clear it; after scout_sign_chunks
 *                     (asynchronous, so it cannot report) read it here.
 *   set "device_error" 0 clears the flag; a non-zero value sets it from the host
 *                     (a way to exercise the error path without a GPU fault)
 *   get "debug"       1 if the plan was created with the environment variable SCOUT_DEBUG
 *                     set to something other than 0: every device buffer the plan owns then
 *                     lies between two 256-byte guard bands of a fixed pattern
 *   get "guards_ok"   debug plans only: 1 if no guard band has been written to (synchronises
 *                     the device); the check that stands in for a memory checker
 *   get "sign_kernels", "certify_kernels"  kernels one scout_sign_chunks / one
 *                     scout_certify call launches for this plan
 *   get "n_tiles", "scratch_bytes", and every settable key
 * Results do not depend on tile_bytes, variant or grid except for the rounding
 * order of the floating-point sums. */
SCOUT_API int scout_plan_set(scout_plan_t *plan, const char *key, int64_t value);
SCOUT_API int scout_plan_get(const scout_plan_t *plan, const char *key, int64_t *value);

/* Diagnostic: the bulk-async scan kernels wait for their copies with a time limit
 * (2 s) and report through "device_error" instead of hanging.  This call runs that
 * wait on a barrier nothing ever signals, with the given limit (<= 1 s):
 * d_out (device, 2 words) receives {1 if the wait gave up, nanoseconds waited}.
 * The kernel returns normally and the context stays usable.  Asynchronous. */
SCOUT_API int scout_selftest_bounded_wait(uint64_t limit_ns, uint64_t *d_out /*device [2]*/, void *stream);

SCOUT_API const char *scout_strerror(int code);
SCOUT_API int scout_version(void);
/* Name of the CUDA error behind the calling thread's most recent SCOUT_ERR_CUDA ("" if none). */
SCOUT_API const char *scout_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SCOUT_H */
