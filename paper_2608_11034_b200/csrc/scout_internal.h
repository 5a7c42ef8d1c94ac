// Internal declarations of the sm_100a sign+vote library (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "scout.h"

namespace scout {

// ---- SF64 signature constants ----------------------------------------------
// The evidence of Sec. 5.2 is "a deterministic, position-sensitive 64-bit hash
// over dtype, shape and bytes"; the function itself is left open there.  This
// library's function: rows of 128 little-endian 32-bit words, row sum
// S_q = sum_s m_s * w[128 q + s], h <- h * P + S_q, then a metadata mix.
//   P   = floor(2^64 / golden ratio), G32 = floor(2^32 / golden ratio),
//   MIX_A / MIX_B = fractional bits of sqrt 2 (made odd) / sqrt 3,
//   SEED_* = fractional bits of sqrt 5, 7, 11, 13.
constexpr uint64_t HASH_P = 0x9E3779B97F4A7C15ull;
constexpr uint32_t HASH_G32 = 0x9E3779B9u;
constexpr uint64_t MIX_A = 0x6A09E667F3BCC909ull;
constexpr uint64_t MIX_B = 0xBB67AE8584CAA73Bull;
constexpr uint64_t SEED_CHUNK = 0x3C6EF372FE94F82Bull;
constexpr uint64_t SEED_TENSOR = 0xA54FF53A5F1D36F1ull;
constexpr uint64_t SEED_SHAPE = 0x510E527FADE682D1ull;
constexpr uint64_t SEED_CERT = 0x9B05688C2B3E6C1Full;
constexpr uint32_t ROW_BYTES = 512;  // 128 words: one 16-byte vector per lane of a warp

__host__ __device__ inline uint64_t mix64(uint64_t z) {
    z ^= z >> 32;
    z *= MIX_A;
    z ^= z >> 29;
    z *= MIX_B;
    z ^= z >> 32;
    return z;
}

// P^e mod 2^64 by square and multiply.
__host__ __device__ inline uint64_t pow_p(uint64_t e) {
    uint64_t r = 1, b = HASH_P;
    for (; e; e >>= 1) {  // a select, not a branch: the lanes of a warp come with different exponents
        r *= (e & 1) ? b : 1ull;
        b *= b;
    }
    return r;
}

__host__ __device__ inline uint64_t finalize_hash(uint64_t h_raw, uint64_t nbytes, uint64_t k,
                                                  uint32_t dtype, uint64_t meta) {
    uint64_t t = mix64(SEED_CHUNK ^ nbytes);
    t = mix64(t ^ k);
    t = mix64(t ^ (uint64_t)dtype);
    t = mix64(t ^ meta);
    return mix64(h_raw + t);
}

// ---- device tables -----------------------------------------------------------
// One work item of the scan: a run of whole rows of one chunk.
struct TileDesc {
    uint64_t off;     // byte offset inside the tensor
    uint64_t poff;    // byte offset inside the packed (staged) image of one replica
    uint32_t tensor;  // tensor index
    uint32_t nbytes;  // bytes in this tile (<= tile_bytes; only a chunk's last tile is short)
    uint32_t chunk;   // global chunk id
    uint32_t dtype : 8;         // SCOUT_DT_*
    uint32_t chunk_tiles : 24;  // tiles of this tile's chunk (at most 2^19: 1 GiB in 2 KiB tiles)
};
static_assert(sizeof(TileDesc) == 32, "TileDesc layout");

struct ChunkDesc {
    uint64_t nbytes;
    uint64_t k;        // index of the chunk inside its tensor
    uint64_t meta;     // caller's shape tag
    uint64_t tile0;    // first tile of the chunk
    uint32_t ntiles;
    uint32_t dtype;
    uint32_t tensor;
    uint32_t pad;
    uint64_t byte_offset;
};
static_assert(sizeof(ChunkDesc) == 56, "ChunkDesc layout");

// Partial evidence of one (replica, tile).
struct TileRec {
    uint64_t h;       // sum over the tile's rows of P^(rows after it in the tile) * S_q
    double sum, sumsq;
    uint32_t nan_count, inf_count;
};
static_assert(sizeof(TileRec) == 32, "TileRec layout");

// Results of the roll-up kernels, copied to the host by scout_certify.
struct CertifyOut {
    uint64_t counts[6];
    uint64_t union_bitmap;
    uint64_t certificate;
    uint64_t replica_bad[64];
};

// What scout_certify brings back to the host in one piece: the counters, the device
// error flag and the first CERTIFY_HEAD entries of both lists.  The one-launch certify
// kernel writes it straight into pinned host memory; the multi-kernel path copies it.
constexpr uint64_t CERTIFY_HEAD = 64;
struct CertifyHost {
    CertifyOut out;
    uint32_t dev_err, pad;
    scout_outlier_t outliers[CERTIFY_HEAD];
    uint64_t undecided[CERTIFY_HEAD];
};

// Where a vote leaves its results (all device memory).
struct VoteSinks {
    uint8_t *status;            // [C] or null
    uint64_t *bitmap;           // [C] or null
    uint64_t *majority;         // [C] or null: e* of every decided chunk (0 if Inconclusive)
    scout_outlier_t *outliers;  // list, capacity outlier_cap
    uint64_t outlier_cap;
    uint64_t *undecided;        // list, capacity undecided_cap
    uint64_t undecided_cap;
    uint64_t *counts;           // [6]: the two list counters (4, 5) are advanced by vote_chunk()
    CertifyOut *cert;           // per-replica bad-chunk counts, or null
};

// Progress of the certificate chain inside a one-launch certify (device, zero between launches).
struct ChainState {
    uint32_t lock;  // 1 while a warp is folding chunks into the chain
    uint32_t pad;
    uint64_t next;  // chunks folded so far
    uint64_t a;     // chain value after `next` chunks
};

// ---- error plumbing ------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char *what);
#define SCOUT_CUDA(call)                                  \
    do {                                                  \
        cudaError_t e__ = (call);                         \
        if (e__ != cudaSuccess) {                         \
            ::scout::set_cuda_error(e__, #call);          \
            return SCOUT_ERR_CUDA;                        \
        }                                                 \
    } while (0)

// ---- programmatic dependent launch ------------------------------------------------
// The small kernels that follow the scan (finalise, vote, certificate) are launched
// with programmatic stream serialisation: their CTAs may be scheduled while the
// previous kernel drains, and wait at griddepcontrol.wait until that kernel has
// completed and its writes are visible.  Without the launch attribute both
// instructions are no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream,
                                    Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- kernel launchers (defined in the .cu files) ------------------------------
struct SignLaunch {
    const TileDesc *tiles;        // device
    uint64_t tile_begin;          // first tile of this launch
    uint64_t n_tiles;             // tiles per replica in this launch
    uint64_t tiles_per_replica;   // stride of the record array
    uint32_t replica_begin;       // first replica of this launch
    uint32_t n_replicas;          // replicas in this launch
    const uint8_t *const *ptrs;   // device table [R][T], or nullptr in staged mode
    uint64_t T;
    const uint8_t *stage;         // staged mode: device image of packed bytes [slice_begin, ...)
    uint64_t slice_begin;         // packed offset held at stage[0]
    TileRec *recs;                // device [R][tiles_per_replica]
    uint32_t *error;              // device flag set when a bounded wait gave up (may be null)
    int variant;                  // 0 direct, 1 direct + register prefetch, 2 bulk-async ring, 3 read probe
    int uniform_dtype;            // dtype shared by every tile of the launch, or -1 if they differ
    unsigned long long *work;     // device [2][work_streams] work counters of the direct scan, 128 bytes
                                  // apart (null: fixed round-robin)
    uint32_t work_parity;         // which of the two this launch uses (successive launches alternate)
    uint32_t work_streams;        // counters the items are dealt from (0 or 1: one), 128 bytes apart
    int grid;                     // CTAs to launch
};
int launch_sign_tiles(const SignLaunch &a, cudaStream_t stream);

// One launch for scan + finalise (mode 0), or scan + finalise + vote + certificate +
// report (mode 1): see certify_tiles and certify_clusters in scout_one_launch.cu.
struct FusedLaunch {
    SignLaunch sign;            // the whole plan: tile_begin 0, every tile, every replica, ptrs set
    const ChunkDesc *chunks;    // device [C]
    uint64_t C;
    uint32_t R;
    uint32_t tile_rows;
    scout_sig_t *sigs;          // device [C][R]
    int mode;                   // 0 sign only, 1 certify
    VoteSinks vote;             // mode 1
    CertifyOut *out;            // mode 1: device counters, zero on entry; left zero on exit
    uint32_t *tickets;          // device [C*R + C], zero on entry; left zero on exit
    uint32_t *done;             // mode 1: device [C] launch stamps
    uint32_t epoch;             // this launch's stamp (never 0); successive launches alternate its parity
    unsigned long long *work;   // device [2]: dynamic work counters, zero on entry (see certify_tiles)
    uint32_t one_level;         // 1: every chunk has at most 64 (tile, replica) items: chunk tickets only
    ChainState *chain;          // mode 1: zero on entry; left zero on exit
    CertifyHost *host;          // mode 1: pinned host memory (device-accessible address)
    int cluster;                // 1: one thread-block cluster per chunk (certify_clusters) instead of tickets
    uint32_t cluster_batch;     // cluster form: chunks a cluster takes at once (cluster_form_possible)
    uint32_t cluster_split;     // cluster form: CTAs per replica of a chunk
};
int launch_fused(const FusedLaunch &l, cudaStream_t stream);
int fused_grid_size(int uniform_dtype, int device, int *grid);
int cluster_form_possible(int uniform_dtype, uint32_t R, uint32_t max_tiles, uint64_t C, int *ok,
                          uint32_t *batch, uint32_t *split);
int sign_grid_size(int variant, int uniform_dtype, int device, int *grid);
int launch_bounded_wait_selftest(uint64_t limit_ns, uint64_t *d_out, cudaStream_t stream);

// zero_out (may be null): a CertifyOut the finalise kernel clears for the vote that follows
int launch_finalize(const ChunkDesc *chunks, uint64_t C, uint32_t R, const TileRec *recs,
                    uint64_t tiles_per_replica, uint32_t tile_rows, uint32_t max_chunk_tiles,
                    scout_sig_t *d_sigs, CertifyOut *zero_out, cudaStream_t stream);

int launch_vote(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint8_t *d_status,
                uint64_t *d_bitmap, scout_outlier_t *d_outliers, uint64_t outlier_cap,
                uint64_t *d_undecided, uint64_t undecided_cap, uint64_t *d_counts,
                uint64_t *d_majority, CertifyOut *d_out, bool counters_already_zero,
                cudaStream_t stream);
int launch_vote_wide(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint64_t chunk_stride,
                     uint64_t replica_stride, uint8_t *d_status, uint64_t *d_bitmap,
                     scout_outlier_t *d_outliers, uint64_t outlier_cap, uint64_t *d_undecided,
                     uint64_t undecided_cap, uint64_t *d_counts, cudaStream_t stream);
int launch_certificate(uint64_t C, const uint64_t *d_majority, CertifyOut *d_out,
                       cudaStream_t stream);
int launch_rollup_tensors(const ChunkDesc *chunks, const uint64_t *tensor_chunk0, uint64_t T,
                          uint32_t R, const scout_sig_t *d_sigs, uint64_t *d_tensor_sigs,
                          cudaStream_t stream);

}  // namespace scout
