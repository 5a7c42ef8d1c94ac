/*
 * CPU oracle for the C3 sign+vote path: TEST INFRASTRUCTURE, not product code.
 * See scout_oracle.h for the parity status of every function.
 *
 * Everything is written as the definition states it: one word, one element,
 * one chunk at a time; no blocking, no vector intrinsics, nothing shared with
 * the CUDA library.
 */
#include "scout_oracle.h"

#include <math.h>
#include <pthread.h>
#include <stdlib.h>
#include <string.h>

/* ---- SF64 constants -------------------------------------------------------
 * The paper (Sec. 5.2) asks for a deterministic, position-sensitive 64-bit hash
 * over dtype, shape and bytes and leaves the function open.  SF64 is this
 * project's reading.  Every constant is derivable:
 *   P   = floor(2^64 / golden ratio)                 (odd, = 1 mod 4)
 *   G32 = floor(2^32 / golden ratio)
 *   C1  = frac(sqrt 2) * 2^64, lowest bit set;  C2 = frac(sqrt 3) * 2^64
 *   K0..K3 = frac(sqrt 5, 7, 11, 13) * 2^64
 */
#define SF_P   0x9E3779B97F4A7C15ull
#define SF_G32 0x9E3779B9u
#define SF_C1  0x6A09E667F3BCC909ull
#define SF_C2  0xBB67AE8584CAA73Bull
#define SF_K0  0x3C6EF372FE94F82Bull
#define SF_K1  0xA54FF53A5F1D36F1ull
#define SF_K2  0x510E527FADE682D1ull
#define SF_K3  0x9B05688C2B3E6C1Full
#define SF_ROW 128u /* words per row */

uint32_t orc_dtype_size(uint32_t dtype)
{
    switch (dtype) {
    case ORC_DT_U8:   return 1;
    case ORC_DT_F32:  return 4;
    case ORC_DT_BF16: return 2;
    case ORC_DT_I64:  return 8;
    case ORC_DT_F16:  return 2;
    case ORC_DT_F64:  return 8;
    case ORC_DT_I32:  return 4;
    default:          return 0;
    }
}

/* 64-bit finaliser: xor-shift, multiply, xor-shift, multiply, xor-shift. */
uint64_t orc_mix64(uint64_t z)
{
    z ^= z >> 32;
    z *= SF_C1;
    z ^= z >> 29;
    z *= SF_C2;
    z ^= z >> 32;
    return z;
}

/* m_s = (((s+1) * G32) mod 2^32) | 1 : 128 distinct odd 32-bit multipliers. */
uint64_t orc_slot_multiplier(uint32_t s)
{
    uint32_t m = (uint32_t)((s + 1u) * SF_G32);
    return (uint64_t)(m | 1u);
}

/* Little-endian 32-bit word i of the chunk; bytes at or past n read as 0. */
static uint32_t word_at(const uint8_t *b, uint64_t n, uint64_t i)
{
    uint32_t w = 0;
    for (unsigned j = 0; j < 4; ++j) {
        uint64_t pos = 4 * i + j;
        if (pos < n) w |= (uint32_t)b[pos] << (8 * j);
    }
    return w;
}

/* H_raw: rows of 128 words; row sum S_q = sum_s m_s * w[q*128+s];
 * h_0 = 0, h_{q+1} = h_q * P + S_q; H_raw = h_Q.  All mod 2^64. */
uint64_t orc_hash_raw(const uint8_t *b, uint64_t n)
{
    uint64_t W = (n + 3) / 4;
    uint64_t Q = (W + SF_ROW - 1) / SF_ROW;
    uint64_t h = 0;
    for (uint64_t q = 0; q < Q; ++q) {
        uint64_t S = 0;
        for (uint32_t s = 0; s < SF_ROW; ++s) {
            uint64_t i = q * SF_ROW + s;
            if (i < W) S += orc_slot_multiplier(s) * (uint64_t)word_at(b, n, i);
        }
        h = h * SF_P + S;
    }
    return h;
}

/* Metadata mix: byte length, index of the piece in its tensor, dtype code and
 * the caller's shape tag all enter the signature (the paper's evidence covers
 * dtype and shape besides the bytes). */
uint64_t orc_hash_final(uint64_t h_raw, uint64_t n, uint64_t k, uint32_t dtype, uint64_t meta_tag)
{
    uint64_t t = orc_mix64(SF_K0 ^ n);
    t = orc_mix64(t ^ k);
    t = orc_mix64(t ^ (uint64_t)dtype);
    t = orc_mix64(t ^ meta_tag);
    return orc_mix64(h_raw + t);
}

uint64_t orc_shape_tag(uint32_t ndim, const uint64_t *dims)
{
    uint64_t a = orc_mix64(SF_K2 ^ (uint64_t)ndim);
    for (uint32_t i = 0; i < ndim; ++i) a = orc_mix64(a ^ dims[i]);
    return a;
}

/* ---- statistics -------------------------------------------------------- */

/* Compensated (Neumaier) accumulator in extended precision: the result is the
 * real-number sum to well below one unit in the last place of a double. */
typedef struct { long double s, c; } acc_t;

static void acc_add(acc_t *a, long double x)
{
    long double t = a->s + x;
    if (fabsl(a->s) >= fabsl(x)) a->c += (a->s - t) + x;
    else                         a->c += (x - t) + a->s;
    a->s = t;
}

static double half_to_double(uint16_t h)
{
    uint32_t sign = h >> 15, e = (h >> 10) & 0x1F, m = h & 0x3FF;
    double v;
    if (e == 0)       v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else              v = ldexp((double)(m + 1024), (int)e - 25);
    return sign ? -v : v;
}

/* Value of element i as a double (exact for every supported float type and
 * for integers below 2^53; larger integers round to nearest). */
static double element_value(const uint8_t *b, uint64_t i, uint32_t dtype)
{
    switch (dtype) {
    case ORC_DT_F32: { float f;    memcpy(&f, b + 4 * i, 4); return (double)f; }
    case ORC_DT_BF16: {
        uint16_t h; memcpy(&h, b + 2 * i, 2);
        uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return (double)f;
    }
    case ORC_DT_F16: { uint16_t h; memcpy(&h, b + 2 * i, 2); return half_to_double(h); }
    case ORC_DT_F64: { double d;   memcpy(&d, b + 8 * i, 8); return d; }
    case ORC_DT_I64: { int64_t v;  memcpy(&v, b + 8 * i, 8); return (double)v; }
    case ORC_DT_I32: { int32_t v;  memcpy(&v, b + 4 * i, 4); return (double)v; }
    default: return 0.0;
    }
}

/* nan/inf: exact element counts.  sum, sumsq: over the FINITE elements only,
 * as real numbers, rounded once to double.  Bytes (u8) carry no statistics. */
void orc_stats(const uint8_t *b, uint64_t n, uint32_t dtype, uint32_t *nan_count,
               uint32_t *inf_count, double *sum, double *sumsq, double *sum_abs)
{
    acc_t s = {0, 0}, q = {0, 0}, a = {0, 0};
    uint32_t nn = 0, ni = 0;
    uint32_t es = orc_dtype_size(dtype);
    if (dtype != ORC_DT_U8 && es != 0) {
        uint64_t count = n / es;
        for (uint64_t i = 0; i < count; ++i) {
            double x = element_value(b, i, dtype);
            if (isnan(x)) { ++nn; continue; }
            if (isinf(x)) { ++ni; continue; }
            long double xl = (long double)x;
            acc_add(&s, xl);
            acc_add(&q, xl * xl);
            acc_add(&a, fabsl(xl));
        }
    }
    *nan_count = nn;
    *inf_count = ni;
    *sum = (double)(s.s + s.c);
    *sumsq = (double)(q.s + q.c);
    if (sum_abs) *sum_abs = (double)(a.s + a.c);
}

void orc_sign_chunk(const uint8_t *b, uint64_t n, uint32_t dtype, uint64_t k,
                    uint64_t meta_tag, orc_sig_t *out)
{
    out->hash = orc_hash_final(orc_hash_raw(b, n), n, k, dtype, meta_tag);
    orc_stats(b, n, dtype, &out->nan_count, &out->inf_count, &out->sum, &out->sumsq, NULL);
}

/* ---- chunking ---------------------------------------------------------- */

/* Each tensor is cut into pieces of chunk_bytes, the last one short; pieces
 * never span tensors; the global chunk id runs over (tensor, piece). */
uint64_t orc_chunk_table(uint64_t T, const orc_tensor_t *tensors, uint64_t chunk_bytes,
                         orc_chunk_t *out, uint64_t cap)
{
    if (chunk_bytes == 0 || chunk_bytes % 512 != 0) return UINT64_MAX;
    uint64_t c = 0;
    for (uint64_t t = 0; t < T; ++t) {
        uint32_t es = orc_dtype_size(tensors[t].dtype);
        if (es == 0 || tensors[t].nbytes == 0 || tensors[t].nbytes % es != 0) return UINT64_MAX;
        uint64_t k = 0;
        for (uint64_t off = 0; off < tensors[t].nbytes; off += chunk_bytes, ++k, ++c) {
            if (out && c < cap) {
                uint64_t left = tensors[t].nbytes - off;
                out[c].tensor = t;
                out[c].index_in_tensor = k;
                out[c].byte_offset = off;
                out[c].nbytes = left < chunk_bytes ? left : chunk_bytes;
            }
        }
    }
    return c;
}

typedef struct {
    const orc_tensor_t *tensors;
    const void *const *ptrs;
    const orc_chunk_t *chunks;
    uint64_t C;
    orc_sig_t *sigs;
    uint64_t stride, offset;
    uint64_t first, step;
} sign_job_t;

static void *sign_worker(void *arg)
{
    sign_job_t *j = (sign_job_t *)arg;
    for (uint64_t c = j->first; c < j->C; c += j->step) {
        const orc_chunk_t *ch = &j->chunks[c];
        const orc_tensor_t *tn = &j->tensors[ch->tensor];
        const uint8_t *base = (const uint8_t *)j->ptrs[ch->tensor] + ch->byte_offset;
        orc_sign_chunk(base, ch->nbytes, tn->dtype, ch->index_in_tensor, tn->meta_tag,
                       &j->sigs[c * j->stride + j->offset]);
    }
    return NULL;
}

int orc_sign_replica(uint64_t T, const orc_tensor_t *tensors, const void *const *ptrs,
                     uint64_t chunk_bytes, orc_sig_t *sigs, uint64_t stride, uint64_t offset,
                     int nthreads)
{
    uint64_t C = orc_chunk_table(T, tensors, chunk_bytes, NULL, 0);
    if (C == UINT64_MAX) return -1;
    orc_chunk_t *chunks = (orc_chunk_t *)malloc((C ? C : 1) * sizeof(orc_chunk_t));
    if (!chunks) return -1;
    orc_chunk_table(T, tensors, chunk_bytes, chunks, C);
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 1024) nthreads = 1024;
    sign_job_t *jobs = (sign_job_t *)malloc((size_t)nthreads * sizeof(sign_job_t));
    pthread_t *tids = (pthread_t *)malloc((size_t)nthreads * sizeof(pthread_t));
    for (int i = 0; i < nthreads; ++i) {
        sign_job_t job = {tensors, ptrs, chunks, C, sigs, stride, offset, (uint64_t)i,
                          (uint64_t)nthreads};
        jobs[i] = job;
    }
    if (nthreads == 1) {
        sign_worker(&jobs[0]);
    } else {
        for (int i = 0; i < nthreads; ++i) pthread_create(&tids[i], NULL, sign_worker, &jobs[i]);
        for (int i = 0; i < nthreads; ++i) pthread_join(tids[i], NULL);
    }
    free(tids);
    free(jobs);
    free(chunks);
    return 0;
}

/* ---- exact consensus (Algorithm 1, Exact branch) ------------------------ */

/* One chunk: the most frequent value e* and its count c*; c* <= N/2 gives
 * Inconclusive with a zero bitmap; otherwise B[j] = 1{e_j != e*}, and the
 * status is Attributed when any bit is set, else Agree.  Only the 64-bit hash
 * is compared.  Returns the status; *majority receives e* (0 if none). */
static int vote_one(uint32_t R, const orc_sig_t *e, uint64_t *bitmap, uint64_t *majority)
{
    uint32_t best_count = 0;
    uint64_t best_value = 0;
    for (uint32_t j = 0; j < R; ++j) {
        uint32_t cnt = 0;
        for (uint32_t i = 0; i < R; ++i)
            if (e[i].hash == e[j].hash) ++cnt;
        if (cnt > best_count) { best_count = cnt; best_value = e[j].hash; }
    }
    *bitmap = 0;
    *majority = 0;
    if (2ull * best_count <= (uint64_t)R) return ORC_INCONCLUSIVE;
    uint64_t B = 0;
    for (uint32_t j = 0; j < R; ++j)
        if (e[j].hash != best_value) B |= 1ull << j;
    *bitmap = B;
    *majority = best_value;
    return B ? ORC_ATTRIBUTED : ORC_AGREE;
}

int orc_vote(uint32_t R, uint64_t C, const orc_sig_t *sigs, uint8_t *status, uint64_t *bitmap,
             orc_outlier_t *outliers, uint64_t outlier_cap, uint64_t *undecided,
             uint64_t undecided_cap, uint64_t *counts)
{
    if (R < 2 || R > 64) return -1;
    uint64_t n_agree = 0, n_attr = 0, n_inc = 0, n_out = 0, n_und = 0;
    for (uint64_t c = 0; c < C; ++c) {
        uint64_t B, maj;
        int s = vote_one(R, sigs + c * R, &B, &maj);
        if (status) status[c] = (uint8_t)s;
        if (bitmap) bitmap[c] = B;
        if (s == ORC_AGREE) ++n_agree;
        else if (s == ORC_ATTRIBUTED) {
            ++n_attr;
            for (uint32_t j = 0; j < R; ++j) {
                if ((B >> j) & 1) {
                    if (outliers && n_out < outlier_cap) {
                        outliers[n_out].chunk = c;
                        outliers[n_out].replica = j;
                        outliers[n_out].reserved = 0;
                    }
                    ++n_out;
                }
            }
        } else {
            ++n_inc;
            if (undecided && n_und < undecided_cap) undecided[n_und] = c;
            ++n_und;
        }
    }
    if (counts) {
        counts[0] = C; counts[1] = n_agree; counts[2] = n_attr; counts[3] = n_inc;
        counts[4] = n_out; counts[5] = n_und;
    }
    return (n_out > outlier_cap || n_und > undecided_cap) ? -6 : 0;
}

/* The same rule for groups of any size and for strided record tables: the
 * record of (chunk c, replica r) is sigs[c * chunk_stride + r * replica_stride];
 * bitmap holds W = ceil(R / 64) words per chunk. */
int orc_vote_wide(uint32_t R, uint64_t C, const orc_sig_t *sigs, uint64_t chunk_stride,
                  uint64_t replica_stride, uint8_t *status, uint64_t *bitmap, orc_outlier_t *outliers,
                  uint64_t outlier_cap, uint64_t *undecided, uint64_t undecided_cap, uint64_t *counts)
{
    if (R < 2) return -1;
    uint32_t W = (R + 63) / 64;
    uint64_t n_agree = 0, n_attr = 0, n_inc = 0, n_out = 0, n_und = 0;
    for (uint64_t c = 0; c < C; ++c) {
        const orc_sig_t *row = sigs + c * chunk_stride;
        uint32_t best_count = 0;
        uint64_t best_value = 0;
        for (uint32_t j = 0; j < R; ++j) {
            uint32_t cnt = 0;
            for (uint32_t i = 0; i < R; ++i)
                if (row[i * replica_stride].hash == row[j * replica_stride].hash) ++cnt;
            if (cnt > best_count) { best_count = cnt; best_value = row[j * replica_stride].hash; }
        }
        for (uint32_t w = 0; w < W; ++w) bitmap[c * W + w] = 0;
        if (2ull * best_count <= (uint64_t)R) {
            status[c] = ORC_INCONCLUSIVE;
            ++n_inc;
            if (n_und < undecided_cap) undecided[n_und] = c;
            ++n_und;
            continue;
        }
        uint32_t marked = 0;
        for (uint32_t j = 0; j < R; ++j) {
            if (row[j * replica_stride].hash != best_value) {
                bitmap[c * W + j / 64] |= 1ull << (j % 64);
                if (n_out < outlier_cap) {
                    outliers[n_out].chunk = c;
                    outliers[n_out].replica = j;
                    outliers[n_out].reserved = 0;
                }
                ++n_out;
                ++marked;
            }
        }
        status[c] = marked ? ORC_ATTRIBUTED : ORC_AGREE;
        if (marked) ++n_attr; else ++n_agree;
    }
    counts[0] = C; counts[1] = n_agree; counts[2] = n_attr; counts[3] = n_inc;
    counts[4] = n_out; counts[5] = n_und;
    return (n_out > outlier_cap || n_und > undecided_cap) ? -6 : 0;
}

/* ---- roll-ups ------------------------------------------------------------ */

/* Tensor-level signature from the chunk hashes of one replica, in order. */
uint64_t orc_rollup(const uint64_t *hashes, uint64_t n)
{
    uint64_t a = orc_mix64(SF_K1 ^ n);
    for (uint64_t i = 0; i < n; ++i) a = orc_mix64(a ^ hashes[i]);
    return a;
}

uint64_t orc_certificate(uint32_t R, uint64_t C, const orc_sig_t *sigs, const uint8_t *status,
                         const uint64_t *bitmap)
{
    uint64_t a = orc_mix64(SF_K3 ^ C);
    for (uint64_t c = 0; c < C; ++c) {
        if (status[c] == ORC_INCONCLUSIVE) return 0;
        /* the majority hash is held by any replica whose bit is clear */
        uint32_t j = 0;
        while (j < R && ((bitmap[c] >> j) & 1)) ++j;
        a = orc_mix64(a ^ sigs[c * R + j].hash);
    }
    return a;
}

/* verdict 0 = every chunk agrees; 1 = every chunk has a strict majority and at
 * least one replica is attributed; 2 = at least one chunk has no strict
 * majority, so nothing is certified (certificate 0). */
int orc_certify(uint32_t R, uint64_t C, const orc_sig_t *sigs, orc_report_t *report,
                orc_outlier_t *outliers, uint64_t outlier_cap, uint64_t *undecided,
                uint64_t undecided_cap, uint64_t *replica_bad)
{
    if (R < 2 || R > 64 || !report) return -1;
    uint8_t *status = (uint8_t *)malloc(C ? C : 1);
    uint64_t *bitmap = (uint64_t *)malloc((C ? C : 1) * sizeof(uint64_t));
    uint64_t counts[6];
    int rc = orc_vote(R, C, sigs, status, bitmap, outliers, outlier_cap, undecided,
                      undecided_cap, counts);
    if (rc == -1) { free(status); free(bitmap); return rc; }
    memset(report, 0, sizeof(*report));
    report->n_chunks = counts[0];
    report->n_agree = counts[1];
    report->n_attributed = counts[2];
    report->n_inconclusive = counts[3];
    report->n_outliers = counts[4];
    report->n_undecided = counts[5];
    if (replica_bad) memset(replica_bad, 0, R * sizeof(uint64_t));
    for (uint64_t c = 0; c < C; ++c) {
        report->replica_union_bitmap |= bitmap[c];
        if (replica_bad)
            for (uint32_t j = 0; j < R; ++j)
                if ((bitmap[c] >> j) & 1) ++replica_bad[j];
    }
    if (counts[3] > 0)      report->verdict = 2;
    else if (counts[2] > 0) report->verdict = 1;
    else                    report->verdict = 0;
    report->certificate = report->verdict <= 1 ? orc_certificate(R, C, sigs, status, bitmap) : 0;
    free(status);
    free(bitmap);
    return rc;
}
