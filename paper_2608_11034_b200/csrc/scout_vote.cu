// Exact consensus (Sec. 5.3; Algorithm 1, Exact branch) over the gathered
// evidence of every chunk, the compaction of disagreements into lists, and the
// roll-ups built on top of it.
#include "scout_internal.h"
#include "scout_vote_device.cuh"

namespace scout {
namespace {

constexpr int VOTE_THREADS = 256;

// One warp per chunk; the rule itself is vote_chunk() (scout_vote_device.cuh).
__global__ void __launch_bounds__(VOTE_THREADS) vote_chunks(
    uint32_t R, uint64_t C, const scout_sig_t *__restrict__ sigs, uint8_t *status_out,
    uint64_t *bitmap_out, scout_outlier_t *outliers, uint64_t outlier_cap, uint64_t *undecided,
    uint64_t undecided_cap, uint64_t *counts, uint64_t *majority_out, CertifyOut *cert) {
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (VOTE_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (VOTE_THREADS / 32);
    uint32_t n_agree = 0, n_attr = 0, n_inc = 0;  // per warp, identical in all lanes
    uint64_t union_bits = 0;
    const VoteSinks sinks = {status_out, bitmap_out, majority_out, outliers, outlier_cap,
                             undecided, undecided_cap, counts, cert};

    for (uint64_t c = warp; c < C; c += n_warps) {
        const scout_sig_t *e = sigs + c * R;
        const uint64_t e0 = lane < R ? e[lane].hash : 0ull;
        const uint64_t e1 = lane + 32u < R ? e[lane + 32u].hash : 0ull;
        uint64_t bitmap, majority;
        const uint32_t st = vote_chunk(R, c, e0, e1, lane, sinks, bitmap, majority);
        if (st == SCOUT_INCONCLUSIVE) ++n_inc;
        else if (st == SCOUT_ATTRIBUTED) ++n_attr;
        else ++n_agree;
        union_bits |= bitmap;
    }

    // block-level aggregation of the status counters: one atomic per counter per CTA
    __shared__ uint32_t sh[3];
    __shared__ unsigned long long sh_union;
    if (threadIdx.x == 0) { sh[0] = sh[1] = sh[2] = 0u; sh_union = 0ull; }
    __syncthreads();
    if (lane == 0) {
        if (n_agree) atomicAdd(&sh[0], n_agree);
        if (n_attr) atomicAdd(&sh[1], n_attr);
        if (n_inc) atomicAdd(&sh[2], n_inc);
        if (union_bits) atomicOr(&sh_union, (unsigned long long)union_bits);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (sh[0]) atomicAdd((unsigned long long *)&counts[1], (unsigned long long)sh[0]);
        if (sh[1]) atomicAdd((unsigned long long *)&counts[2], (unsigned long long)sh[1]);
        if (sh[2]) atomicAdd((unsigned long long *)&counts[3], (unsigned long long)sh[2]);
        if (cert && sh_union) atomicOr((unsigned long long *)&cert->union_bitmap, sh_union);
        if (blockIdx.x == 0) counts[0] = C;
    }
}

// Wide groups (up to SCOUT_MAX_REPLICAS peers) and strided record tables: one CTA
// per chunk.  The R hashes go to shared memory; thread j counts the peers that
// hold e_j; a block-wide maximum gives c*; 2 c* <= R is Inconclusive; otherwise
// the value of any thread whose count is c* is e* and the bitmap words are
// assembled from warp ballots.
constexpr int WIDE_THREADS = 128;

__global__ void __launch_bounds__(WIDE_THREADS) vote_chunks_wide(
    uint32_t R, uint64_t C, const scout_sig_t *__restrict__ sigs, uint64_t chunk_stride,
    uint64_t replica_stride, uint8_t *status_out, uint64_t *bitmap_out, scout_outlier_t *outliers,
    uint64_t outlier_cap, uint64_t *undecided, uint64_t undecided_cap, uint64_t *counts) {
    __shared__ uint64_t e[SCOUT_MAX_REPLICAS];
    __shared__ uint32_t bits[SCOUT_MAX_REPLICAS / 32];
    __shared__ uint32_t best_count, n_set;
    __shared__ unsigned long long best_value, list_base;
    const uint32_t tid = threadIdx.x, lane = tid & 31u;
    const uint32_t W = (R + 63u) / 64u;
    uint32_t n_agree = 0, n_attr = 0, n_inc = 0;  // kept by thread 0

    for (uint64_t c = blockIdx.x; c < C; c += gridDim.x) {
        for (uint32_t r = tid; r < R; r += WIDE_THREADS)
            e[r] = sigs[c * chunk_stride + (uint64_t)r * replica_stride].hash;
        if (tid == 0) { best_count = 0; n_set = 0; }
        for (uint32_t w = tid; w < SCOUT_MAX_REPLICAS / 32; w += WIDE_THREADS) bits[w] = 0u;
        __syncthreads();
        uint32_t mine = 0;
        uint64_t mine_value = 0;
        for (uint32_t r = tid; r < R; r += WIDE_THREADS) {
            const uint64_t v = e[r];
            uint32_t cnt = 0;
            for (uint32_t i = 0; i < R; ++i) cnt += (e[i] == v);
            if (cnt > mine) { mine = cnt; mine_value = v; }
        }
        atomicMax(&best_count, mine);
        __syncthreads();
        const uint32_t best = best_count;
        const bool decided = 2u * best > R;
        if (decided && mine == best) best_value = mine_value;  // every writer holds the same e*
        __syncthreads();
        if (decided) {
            const uint64_t majority = best_value;
            for (uint32_t r0 = 0; r0 < R; r0 += WIDE_THREADS) {  // uniform trip count: ballots are safe
                const uint32_t r = r0 + tid;
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, r < R && e[r] != majority);
                if (lane == 0 && b) {
                    bits[r >> 5] = b;
                    atomicAdd(&n_set, (uint32_t)__popc(b));
                }
            }
        }
        __syncthreads();
        const uint32_t total = n_set;
        if (tid == 0) {
            const uint32_t st = !decided ? SCOUT_INCONCLUSIVE : (total ? SCOUT_ATTRIBUTED : SCOUT_AGREE);
            if (status_out) status_out[c] = (uint8_t)st;
            if (st == SCOUT_INCONCLUSIVE) {
                ++n_inc;
                const unsigned long long pos = atomicAdd((unsigned long long *)&counts[5], 1ull);
                if (pos < undecided_cap) undecided[pos] = c;
            } else if (total) {
                ++n_attr;
                list_base = atomicAdd((unsigned long long *)&counts[4], (unsigned long long)total);
            } else {
                ++n_agree;
            }
        }
        if (bitmap_out)
            for (uint32_t w = tid; w < W; w += WIDE_THREADS)
                bitmap_out[c * W + w] = ((uint64_t)bits[2 * w + 1] << 32) | bits[2 * w];
        __syncthreads();
        if (total) {  // block-aggregated append: one atomic per chunk, offsets from the bit words
            for (uint32_t r = tid; r < R; r += WIDE_THREADS) {
                if ((bits[r >> 5] >> (r & 31u)) & 1u) {
                    uint32_t before = __popc(bits[r >> 5] & ((1u << (r & 31u)) - 1u));
                    for (uint32_t w = 0; w < (r >> 5); ++w) before += __popc(bits[w]);
                    const uint64_t pos = list_base + before;
                    if (pos < outlier_cap) outliers[pos] = scout_outlier_t{c, r, 0u};
                }
            }
        }
        __syncthreads();
    }
    if (tid == 0) {
        if (n_agree) atomicAdd((unsigned long long *)&counts[1], (unsigned long long)n_agree);
        if (n_attr) atomicAdd((unsigned long long *)&counts[2], (unsigned long long)n_attr);
        if (n_inc) atomicAdd((unsigned long long *)&counts[3], (unsigned long long)n_inc);
        if (blockIdx.x == 0) counts[0] = C;
    }
}

// Certificate: a <- mix64(seed ^ C); a <- mix64(a ^ majority_c) for every chunk
// in order.  The chain is sequential by construction; one warp streams the
// hashes in coalesced groups of 32 (the next group is in flight while this one
// is folded) and every lane runs the same chain.  A full group is folded by an
// unrolled loop, so that the 32 broadcasts are issued ahead of the dependent mix
// steps instead of one per step.
__global__ void certificate_chain(uint64_t C, const uint64_t *__restrict__ majority, CertifyOut *out) {
    pdl_wait();
    const uint32_t lane = threadIdx.x;
    uint64_t a = mix64(SEED_CERT ^ C);
    uint64_t next = lane < C ? majority[lane] : 0ull;
    for (uint64_t base = 0; base < C; base += 32) {
        const uint64_t cur = next;
        const uint64_t nb = base + 32 + lane;
        next = nb < C ? majority[nb] : 0ull;
        if (C - base >= 32) {
#pragma unroll
            for (uint32_t i = 0; i < 32; ++i) a = mix64(a ^ __shfl_sync(0xFFFFFFFFu, cur, i));
        } else {
            const uint32_t n = (uint32_t)(C - base);
            for (uint32_t i = 0; i < n; ++i) a = mix64(a ^ __shfl_sync(0xFFFFFFFFu, cur, i));
        }
    }
    if (lane == 0) {
        out->certificate = out->counts[3] ? 0ull : a;
    }
}

// Tensor-level signature (the granularity of Sec. 5.2): chunk hashes of one
// (tensor, replica) folded in order.  One thread per (tensor, replica).
__global__ void rollup_tensors(const uint64_t *__restrict__ tensor_chunk0, uint64_t T, uint32_t R,
                               const scout_sig_t *__restrict__ sigs, uint64_t *out) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T * R) return;
    const uint64_t t = i / R;
    const uint32_t r = (uint32_t)(i - t * R);
    const uint64_t c0 = tensor_chunk0[t], c1 = tensor_chunk0[t + 1];
    uint64_t a = mix64(SEED_TENSOR ^ (c1 - c0));
    for (uint64_t c = c0; c < c1; ++c) a = mix64(a ^ sigs[c * R + r].hash);
    out[i] = a;
}

}  // namespace

int launch_vote(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint8_t *d_status,
                uint64_t *d_bitmap, scout_outlier_t *d_outliers, uint64_t outlier_cap,
                uint64_t *d_undecided, uint64_t undecided_cap, uint64_t *d_counts,
                uint64_t *d_majority, CertifyOut *d_out, bool counters_already_zero,
                cudaStream_t stream) {
    if (!counters_already_zero) {
        if (d_out) SCOUT_CUDA(cudaMemsetAsync(d_out, 0, sizeof(CertifyOut), stream));
        if ((void *)d_counts != (void *)d_out)
            SCOUT_CUDA(cudaMemsetAsync(d_counts, 0, 6 * sizeof(uint64_t), stream));
    }
    uint64_t blocks = (C + VOTE_THREADS / 32 - 1) / (VOTE_THREADS / 32);
    if (blocks > 148ull * 8) blocks = 148ull * 8;
    if (blocks == 0) blocks = 1;
    if (counters_already_zero) {  // follows the finalise kernel directly: dependent launch
        SCOUT_CUDA(launch_dependent(vote_chunks, dim3((unsigned)blocks), dim3(VOTE_THREADS), stream, R, C,
                                    d_sigs, d_status, d_bitmap, d_outliers, outlier_cap, d_undecided,
                                    undecided_cap, d_counts, d_majority, d_out));
    } else {
        vote_chunks<<<(int)blocks, VOTE_THREADS, 0, stream>>>(R, C, d_sigs, d_status, d_bitmap, d_outliers,
                                                             outlier_cap, d_undecided, undecided_cap,
                                                             d_counts, d_majority, d_out);
        SCOUT_CUDA(cudaGetLastError());
    }
    return SCOUT_OK;
}

int launch_vote_wide(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint64_t chunk_stride,
                     uint64_t replica_stride, uint8_t *d_status, uint64_t *d_bitmap,
                     scout_outlier_t *d_outliers, uint64_t outlier_cap, uint64_t *d_undecided,
                     uint64_t undecided_cap, uint64_t *d_counts, cudaStream_t stream) {
    SCOUT_CUDA(cudaMemsetAsync(d_counts, 0, 6 * sizeof(uint64_t), stream));
    uint64_t blocks = C < 148ull * 8 ? C : 148ull * 8;
    if (blocks == 0) blocks = 1;
    vote_chunks_wide<<<(int)blocks, WIDE_THREADS, 0, stream>>>(R, C, d_sigs, chunk_stride, replica_stride,
                                                               d_status, d_bitmap, d_outliers, outlier_cap,
                                                               d_undecided, undecided_cap, d_counts);
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}

int launch_certificate(uint64_t C, const uint64_t *d_majority, CertifyOut *d_out, cudaStream_t stream) {
    SCOUT_CUDA(launch_dependent(certificate_chain, dim3(1), dim3(32), stream, C, d_majority, d_out));
    return SCOUT_OK;
}

int launch_rollup_tensors(const ChunkDesc *, const uint64_t *tensor_chunk0, uint64_t T, uint32_t R,
                          const scout_sig_t *d_sigs, uint64_t *d_tensor_sigs, cudaStream_t stream) {
    const uint64_t n = T * R;
    if (n == 0) return SCOUT_OK;
    rollup_tensors<<<(unsigned)((n + 127) / 128), 128, 0, stream>>>(tensor_chunk0, T, R, d_sigs,
                                                                   d_tensor_sigs);
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}

}  // namespace scout
