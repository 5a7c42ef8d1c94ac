/*
 * CPU oracle for the C3 sign+vote path: TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-pass restatement of what the path computes, written
 * from the paper's statement of comparable evidence (Sec. 5.2) and exact
 * consensus (Sec. 5.3, Algorithm 1, Exact branch).  It shares no code, header,
 * table or constant generator with the CUDA library.  Only tests, the smoke
 * check and the benchmark's cpu_baseline / reference legs may call it.
 *
 * Parity status of each function (what pins it besides itself):
 *   orc_hash_raw / orc_hash_final  the paper requires only a deterministic,
 *       position-sensitive 64-bit hash over dtype, shape and bytes and does not
 *       fix the function; "SF64" below is this project's reading.  Pinned to
 *       that definition by big-integer brute force, known-answer values,
 *       algebraic invariants (single-word change, word swap, segment combine),
 *       and derivations of every constant.  It cannot be pinned to a value the
 *       paper prints, because the paper prints none.
 *   orc_stats     sidecar statistics (not in the paper); pinned by correctly
 *       rounded summation, closed forms and special values.
 *   orc_vote      Algorithm 1's Exact branch; pinned by exhaustive brute force
 *       against an independently written rule and by every case the paper's
 *       prose fixes (two-rank disagreement, several distinct minorities,
 *       majority-held fault, no strict majority).
 *   orc_rollup / orc_certificate / orc_certify   project-defined roll-ups
 *       (the paper defines none): pinned by known-answer values and invariants.
 */
#ifndef SCOUT_ORACLE_H
#define SCOUT_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* dtype codes (they enter the hash, so they are frozen) */
enum { ORC_DT_U8 = 0, ORC_DT_F32 = 1, ORC_DT_BF16 = 2, ORC_DT_I64 = 3,
       ORC_DT_F16 = 4, ORC_DT_F64 = 5, ORC_DT_I32 = 6 };

/* statuses of Algorithm 1 */
enum { ORC_AGREE = 0, ORC_ATTRIBUTED = 1, ORC_INCONCLUSIVE = 2 };

typedef struct {
    uint64_t hash;
    uint32_t nan_count, inf_count;
    double sum, sumsq;
} orc_sig_t;

typedef struct {
    uint64_t nbytes;
    uint32_t dtype;
    uint32_t reserved;
    uint64_t meta_tag;
} orc_tensor_t;

typedef struct {
    uint64_t chunk;
    uint32_t replica;
    uint32_t reserved;
} orc_outlier_t;

typedef struct {
    uint64_t tensor;          /* index into the tensor table              */
    uint64_t index_in_tensor; /* k: position of the piece in its tensor   */
    uint64_t byte_offset;     /* offset of the piece inside the tensor    */
    uint64_t nbytes;          /* length of the piece (last piece short)   */
} orc_chunk_t;

typedef struct {
    uint64_t n_chunks, n_agree, n_attributed, n_inconclusive, n_outliers, n_undecided;
    uint64_t replica_union_bitmap;
    uint64_t certificate;
    int32_t verdict;
    int32_t reserved;
} orc_report_t;

uint32_t orc_dtype_size(uint32_t dtype);            /* 0 for an unknown code */
uint64_t orc_mix64(uint64_t z);
uint64_t orc_slot_multiplier(uint32_t s);           /* m_s, s in [0,128)     */
uint64_t orc_hash_raw(const uint8_t *b, uint64_t n);
uint64_t orc_hash_final(uint64_t h_raw, uint64_t n, uint64_t k, uint32_t dtype, uint64_t meta_tag);
uint64_t orc_shape_tag(uint32_t ndim, const uint64_t *dims);

/* statistics of one chunk; sum_abs may be NULL */
void orc_stats(const uint8_t *b, uint64_t n, uint32_t dtype, uint32_t *nan_count,
               uint32_t *inf_count, double *sum, double *sumsq, double *sum_abs);

void orc_sign_chunk(const uint8_t *b, uint64_t n, uint32_t dtype, uint64_t k,
                    uint64_t meta_tag, orc_sig_t *out);

/* chunk table: returns the number of chunks; fills out[] when out != NULL
 * (cap entries at most).  Returns UINT64_MAX on invalid arguments. */
uint64_t orc_chunk_table(uint64_t T, const orc_tensor_t *tensors, uint64_t chunk_bytes,
                         orc_chunk_t *out, uint64_t cap);

/* sign every chunk of one replica.  ptrs[t] = host address of tensor t.
 * Record of chunk c is written to sigs[c * stride + offset] (stride = R,
 * offset = replica index gives the chunk-major [C][R] layout).
 * nthreads <= 1: one thread; otherwise that many worker threads, each taking
 * whole chunks.  Returns 0, or -1 on invalid arguments. */
int orc_sign_replica(uint64_t T, const orc_tensor_t *tensors, const void *const *ptrs,
                     uint64_t chunk_bytes, orc_sig_t *sigs, uint64_t stride, uint64_t offset,
                     int nthreads);

/* strict-majority vote over sigs[C][R]; lists come out in ascending
 * (chunk, replica) order.  counts[6] = {n_chunks, n_agree, n_attributed,
 * n_inconclusive, n_outliers, n_undecided} (true totals even when a list is
 * shorter than needed).  Returns 0, -6 if a list was truncated, -1 invalid. */
int orc_vote(uint32_t R, uint64_t C, const orc_sig_t *sigs, uint8_t *status, uint64_t *bitmap,
             orc_outlier_t *outliers, uint64_t outlier_cap, uint64_t *undecided,
             uint64_t undecided_cap, uint64_t *counts);

/* orc_vote for any group size and strided tables: record (c, r) at
 * sigs[c*chunk_stride + r*replica_stride]; bitmap has ceil(R/64) words per chunk */
int orc_vote_wide(uint32_t R, uint64_t C, const orc_sig_t *sigs, uint64_t chunk_stride,
                  uint64_t replica_stride, uint8_t *status, uint64_t *bitmap, orc_outlier_t *outliers,
                  uint64_t outlier_cap, uint64_t *undecided, uint64_t undecided_cap, uint64_t *counts);

uint64_t orc_rollup(const uint64_t *hashes, uint64_t n);
/* certificate over the majority hash of every chunk, in order */
uint64_t orc_certificate(uint32_t R, uint64_t C, const orc_sig_t *sigs, const uint8_t *status,
                         const uint64_t *bitmap);
/* vote + roll-up into a report.  replica_bad[R] (may be NULL) receives the
 * number of chunks attributed to each replica. */
int orc_certify(uint32_t R, uint64_t C, const orc_sig_t *sigs, orc_report_t *report,
                orc_outlier_t *outliers, uint64_t outlier_cap, uint64_t *undecided,
                uint64_t undecided_cap, uint64_t *replica_bad);

#ifdef __cplusplus
}
#endif
#endif
