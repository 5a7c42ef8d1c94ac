// The whole sign + vote + certify path as ONE kernel, in two forms: tickets
// (certify_tiles) and a thread-block cluster per chunk (certify_clusters).  Both use
// the row routine of the staged scan (scout_scan.cuh), its combine (scout_combine.cuh)
// and the vote of the vote kernel (scout_vote_device.cuh): Algorithm 1, exact branch,
// per chunk; then the job-wide counters, the certificate chain and the report.
#include "scout_combine.cuh"
#include "scout_scan.cuh"
#include "scout_vote_device.cuh"

namespace scout {
namespace {

// ---- one launch for the whole path --------------------------------------------------
// certify_tiles = the direct scan + a per-chunk ticket.  Work items are taken tile-major
// (item = tile * R + replica), so the chunks of the plan complete roughly in order.  The
// warp that stores the last tile record of a chunk (atomic ticket; nobody waits for
// anybody) finalises the chunk's R records and, in certify mode, votes the chunk, then
// tries to advance the certificate chain: the chain is a strictly sequential fold over
// the majority hashes in chunk order, so one warp at a time (a try-lock) folds whatever
// prefix of chunks is complete and leaves; whoever completes the next chunk continues.
// The warp that folds the last chunk writes the report block to pinned host memory and
// returns the device state to zero for the next launch.  Nothing in the kernel spins.
struct FusedArgs {
    SignArgs s;
    const ChunkDesc *chunks;
    uint64_t C;
    uint32_t R, tile_rows;
    uint64_t p_stride;
    scout_sig_t *sigs;
    int mode;
    VoteSinks v;
    CertifyOut *out;
    uint32_t *tickets;
    uint32_t *done;
    uint32_t epoch;
    ChainState *chain;
    CertifyHost *host;
    unsigned long long *work;  // two work counters, used alternately by successive launches
    uint32_t one_level;        // tickets: chunk counters only (chunks with few items)
    uint32_t cluster_batch;    // certify_clusters: chunks a cluster takes at once
    uint32_t cluster_split;    // certify_clusters: CTAs that share one replica's copy of a chunk
};

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

constexpr uint64_t SMALL_CHAIN = 256;  // plans with at most this many chunks fold the chain in one go

// The whole warp folds the complete prefix of chunks into the chain.  Returns true in
// every lane if this warp folded the last chunk (it then still holds the lock and must
// publish); chain_value is the finished chain in that case.
__device__ __noinline__ bool advance_chain(const FusedArgs &a, uint32_t lane, uint64_t &chain_value) {
    ChainState *ch = a.chain;
    for (;;) {
        uint32_t owner = 0;
        if (lane == 0) owner = atomicCAS(&ch->lock, 0u, 1u) == 0u;
        if (!__shfl_sync(0xFFFFFFFFu, owner, 0)) return false;  // another warp is folding; it re-checks after it
        __threadfence();
        uint64_t n = *(volatile uint64_t *)&ch->next;
        uint64_t x = n ? *(volatile uint64_t *)&ch->a : mix64(SEED_CERT ^ a.C);
        for (;;) {
            const uint64_t c = n + lane;
            uint64_t m = 0;
            bool ready = false;
            if (c < a.C && ld_acquire_u32(a.done + c) == a.epoch) {
                ready = true;
                m = __ldcg(a.v.majority + c);
            }
            const uint32_t mask = __ballot_sync(0xFFFFFFFFu, ready);
            const uint32_t run = mask == 0xFFFFFFFFu ? 32u : (uint32_t)__ffs((int)~mask) - 1u;
            if (run == 32u) {  // unrolled: the broadcasts are issued ahead of the dependent mix steps
#pragma unroll
                for (uint32_t i = 0; i < 32; ++i) x = mix64(x ^ __shfl_sync(0xFFFFFFFFu, m, i));
            } else {
                for (uint32_t i = 0; i < run; ++i) x = mix64(x ^ __shfl_sync(0xFFFFFFFFu, m, i));
            }
            n += run;
            if (run < 32u) break;
        }
        if (n == a.C) {
            chain_value = x;
            return true;
        }
        if (lane == 0) {
            *(volatile uint64_t *)&ch->a = x;
            *(volatile uint64_t *)&ch->next = n;
            __threadfence();
            atomicExch(&ch->lock, 0u);
            __threadfence();
        }
        // a chunk may have completed between the last look and the release: look once more
        uint32_t again = 0;
        if (lane == 0) again = ld_acquire_u32(a.done + n) == a.epoch;
        if (!__shfl_sync(0xFFFFFFFFu, again, 0)) return false;
    }
}

// Every chunk has been voted and folded: finish the counters, write the report block to
// the host and leave the device state zero.  Called by one warp, which holds the chain lock.
__device__ __noinline__ void publish_report(const FusedArgs &a, uint32_t lane, uint64_t chain_value) {
    uint64_t *dev = reinterpret_cast<uint64_t *>(a.out);
    volatile uint64_t *host = reinterpret_cast<volatile uint64_t *>(&a.host->out);
    constexpr uint32_t WORDS = sizeof(CertifyOut) / sizeof(uint64_t);
    const uint64_t n_inconclusive = __ldcg(&a.out->counts[3]);
    const uint64_t n_out = __ldcg(&a.out->counts[4]), n_und = __ldcg(&a.out->counts[5]);
    for (uint32_t i = lane; i < WORDS; i += 32) {
        uint64_t w = __ldcg(dev + i);
        if (i == 0) w = a.C;                                           // counts[0]
        if (i == 7) w = n_inconclusive ? 0ull : chain_value;           // certificate
        host[i] = w;
        dev[i] = 0ull;                                                 // zero for the next launch
    }
    static_assert(offsetof(CertifyOut, certificate) == 7 * sizeof(uint64_t), "word 7 is the certificate");
    const uint64_t head_out = min(min(n_out, a.v.outlier_cap), CERTIFY_HEAD);
    const uint64_t head_und = min(min(n_und, a.v.undecided_cap), CERTIFY_HEAD);
    for (uint64_t i = lane; i < 2 * head_out; i += 32)
        reinterpret_cast<volatile uint64_t *>(a.host->outliers)[i] =
            __ldcg(reinterpret_cast<const uint64_t *>(a.v.outliers) + i);
    for (uint64_t i = lane; i < head_und; i += 32)
        reinterpret_cast<volatile uint64_t *>(a.host->undecided)[i] = __ldcg(a.v.undecided + i);
    if (lane == 0) {
        *reinterpret_cast<volatile uint32_t *>(&a.host->dev_err) = a.s.error ? __ldcg(a.s.error) : 0u;
        *(volatile uint64_t *)&a.chain->next = 0ull;
        *(volatile uint64_t *)&a.chain->a = 0ull;
        __threadfence();   // the host reads the report after the stream has completed: no system fence needed
        atomicExch(&a.chain->lock, 0u);
    }
}

__device__ __noinline__ void chunk_vote_and_fold(const FusedArgs &a, uint32_t c, uint64_t e0, uint64_t e1,
                                                 uint32_t lane);

// The last tile record of chunk c has been stored: finalise, vote, fold.
__device__ __noinline__ void chunk_complete(const FusedArgs &a, uint32_t c, uint32_t lane) {
    __threadfence();  // the records the other warps released before their tickets are visible now
    const ChunkDesc cd = a.chunks[c];
    uint64_t e0 = 0, e1 = 0;
    const uint64_t weight = combine_weight(cd.ntiles, cd.nbytes, a.tile_rows, lane);
    const TileRec *tr = a.s.recs + cd.tile0;
    if (cd.ntiles <= 32u) {
        for (uint32_t r0 = 0; r0 < a.R; r0 += COMBINE_BATCH) {
            scout_sig_t o[COMBINE_BATCH];
            const uint32_t n_rep = min((uint32_t)COMBINE_BATCH, a.R - r0);
            combine_small(tr + (uint64_t)r0 * a.s.tiles_per_replica, a.s.tiles_per_replica, n_rep, cd.ntiles,
                          cd.nbytes, cd.k, cd.dtype, cd.meta, weight, lane, o);
#pragma unroll
            for (int j = 0; j < COMBINE_BATCH; ++j) {
                const uint32_t r = r0 + j;
                if (r < a.R) {
                    if (lane == 0) a.sigs[(uint64_t)c * a.R + r] = o[j];
                    if (lane == (r & 31u)) {
                        if (r < 32u) e0 = o[j].hash; else e1 = o[j].hash;
                    }
                }
            }
        }
    } else {
        for (uint32_t r = 0; r < a.R; ++r) {
            const scout_sig_t o = combine_tiles(tr + (uint64_t)r * a.s.tiles_per_replica, cd.ntiles, cd.nbytes,
                                                cd.k, cd.dtype, cd.meta, a.p_stride, weight, lane);
            if (lane == 0) a.sigs[(uint64_t)c * a.R + r] = o;
            const uint64_t h = __shfl_sync(0xFFFFFFFFu, o.hash, 0);
            if (lane == (r & 31u)) {
                if (r < 32u) e0 = h; else e1 = h;
            }
        }
    }
    // both ticket levels of this chunk go back to zero for the next launch
    for (uint32_t r = lane; r <= a.R; r += 32) a.tickets[r < a.R ? (uint64_t)c * a.R + r : a.C * a.R + c] = 0u;
    if (a.mode == 0) return;
    chunk_vote_and_fold(a, c, e0, e1, lane);
}

// The R records of chunk c exist and lane j holds the hashes of replicas j and j + 32:
// vote the chunk, count it, and fold the certificate chain as far as it can be folded.
__device__ __noinline__ void chunk_vote_and_fold(const FusedArgs &a, uint32_t c, uint64_t e0, uint64_t e1,
                                                 uint32_t lane) {
    uint64_t bitmap, majority;
    const uint32_t st = vote_chunk(a.R, c, e0, e1, lane, a.v, bitmap, majority);
    if (a.C <= SMALL_CHAIN) {
        // Few chunks: no incremental folding.  The warp that votes the last chunk folds the
        // whole chain at once (C mix steps after one round of loads).
        uint32_t finisher = 0;
        if (lane == 0) {
            atomicAdd((unsigned long long *)&a.out->counts[1 + st], 1ull);  // AGREE, ATTRIBUTED, INCONCLUSIVE
            if (bitmap) atomicOr((unsigned long long *)&a.out->union_bitmap, (unsigned long long)bitmap);
            __threadfence();
            finisher = atomicAdd((unsigned long long *)&a.chain->next, 1ull) + 1ull == a.C;
        }
        if (!__shfl_sync(0xFFFFFFFFu, finisher, 0)) return;
        __threadfence();
        uint64_t x = mix64(SEED_CERT ^ a.C);
        for (uint64_t base = 0; base < a.C; base += 32) {
            const uint64_t m = base + lane < a.C ? __ldcg(a.v.majority + base + lane) : 0ull;
            const uint32_t n = (uint32_t)min((uint64_t)32, a.C - base);
            for (uint32_t i = 0; i < n; ++i) x = mix64(x ^ __shfl_sync(0xFFFFFFFFu, m, i));
        }
        publish_report(a, lane, x);
        return;
    }
    if (lane == 0) {
        atomicAdd((unsigned long long *)&a.out->counts[1 + st], 1ull);
        if (bitmap) atomicOr((unsigned long long *)&a.out->union_bitmap, (unsigned long long)bitmap);
        __threadfence();
        st_release_u32(a.done + c, a.epoch);
        __threadfence();
    }
    __syncwarp();
    uint64_t chain_value = 0;
    if (advance_chain(a, lane, chain_value)) publish_report(a, lane, chain_value);
}

// Tickets.  First level: one counter per (chunk, replica), advanced once per tile; the warp
// that brings it to the chunk's tile count advances the second level, one counter per
// chunk, and the warp that brings that one to R has completed the chunk.  Two levels keep
// the number of atomics per address small (same-address atomics serialise in L2); plans
// whose chunks have few (tile, replica) items use the chunk counter alone (one round trip
// less on the way to the result).  The result of a tile's atomic is looked at one tile
// later, after the next tile has been scanned, so no warp waits for an atomic's round trip.
__device__ __forceinline__ void resolve_ticket(const FusedArgs &a, uint32_t lane, uint32_t returned,
                                               uint32_t tiles_of_chunk, uint32_t chunk) {
    uint32_t last = 0;
    if (a.one_level) {
        last = lane == 0 && returned + 1u == tiles_of_chunk * a.R;
    } else if (lane == 0 && returned + 1u == tiles_of_chunk) {
        last = atomicAdd(&a.tickets[a.C * a.R + chunk], 1u) + 1u == a.R;
    }
    if (__shfl_sync(0xFFFFFFFFu, last, 0)) chunk_complete(a, chunk, lane);
}

template <int DTSEL>
__global__ void __launch_bounds__(SIGN_THREADS, SCOUT_MINBLOCKS) certify_tiles(const __grid_constant__ FusedArgs a) {
    const uint32_t lane = threadIdx.x & 31u;
    // Work items are handed out dynamically (a warp that stops to finalise a chunk simply
    // takes fewer tiles afterwards): every warp starts with item `warp`, later items come
    // from a counter.  The counter of this launch is work[epoch & 1]; the other one is
    // zeroed here for the next launch.  The next item is requested before the current tile
    // is scanned and looked at after it, so the atomic's round trip is never waited for.
    // Few values live across the scan of a tile (what can be recomputed from the launch
    // arguments is): the answers of the two atomics must stay in registers, a spill of
    // either would wait for its round trip.
#define N_WARPS ((uint64_t)gridDim.x * (SIGN_THREADS / 32))
#define N_ITEMS (a.s.n_tiles * a.R)
    uint64_t item = (uint64_t)blockIdx.x * (SIGN_THREADS / 32) + (threadIdx.x >> 5);
    if (item == 0 && lane == 0) a.work[(a.epoch & 1u) ^ 1u] = 0ull;
    // the previous tile's ticket: value its atomic returned (lane 0), tiles of its chunk, its chunk
    uint32_t prev_returned = 0, prev_tiles = 0, prev_chunk = 0;
    while (item < N_ITEMS) {
        unsigned long long next = N_ITEMS;  // "nothing left" unless the counter says otherwise
        if (N_ITEMS > N_WARPS && lane == 0) next = atomicAdd(a.work + (a.epoch & 1u), 1ull);
        const uint64_t t = item / a.R;
        const uint32_t r = (uint32_t)(item - t * a.R);
        const TileDesc td = a.s.tiles[t];
        const uint8_t *tile = a.s.ptrs[(uint64_t)r * a.s.T + td.tensor] + td.off;
        TileRec *const out = &a.s.recs[(uint64_t)r * a.s.tiles_per_replica + t];
        uint32_t *const ticket = &a.tickets[a.one_level ? a.C * a.R + td.chunk : (uint64_t)td.chunk * a.R + r];
        // whoever completes this chunk reads its descriptor: have it in L2 by then
        if (lane == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.chunks + td.chunk));
        TileRec rec;
        if constexpr (DTSEL >= 0) scan_tile<DTSEL, true>(tile, td.nbytes, lane, rec);
        else                      scan_dispatch(td.dtype, tile, td.nbytes, lane, rec);
        if (prev_tiles) resolve_ticket(a, lane, prev_returned, prev_tiles, prev_chunk);
        if (lane == 0) {
            store_record(out, rec);
            __threadfence();
            prev_returned = atomicAdd(ticket, 1u);
        }
        prev_tiles = td.chunk_tiles;
        prev_chunk = td.chunk;
        item = N_WARPS + __shfl_sync(0xFFFFFFFFu, next, 0);
    }
    if (prev_tiles) resolve_ticket(a, lane, prev_returned, prev_tiles, prev_chunk);
#undef N_WARPS
#undef N_ITEMS
}

// ---- one launch, one thread-block cluster per chunk -----------------------------------
// certify_clusters: the same path for plans made of many small chunks.  A cluster of
// R * split CTAs takes chunk c; `split` CTAs share replica r's copy of the chunk (one warp
// per tile, the tile geometry of the plan).  Tile records are stored straight into the
// shared memory of the replica's first CTA, which combines them after a barrier and
// stores the finished hash into the shared memory of the cluster's first CTA; that one
// votes after a second barrier.  No tile record, ticket or fence goes through global
// memory on the way to the vote: from the arrival of a chunk's last byte to its vote
// there are two barriers and no L2 round trip.  Only the job-wide steps (counters,
// certificate chain, report) use global atomics, once per chunk.  The tile table is not
// read: a chunk's tiles follow from its descriptor.  Chunks of fewer than 16 tiles are
// taken `batch` at a time, so that every warp of a CTA has a tile.
constexpr int CLUSTER_THREADS = 512;          // 256-thread CTAs measured equal or slower on every shape tried
constexpr int CLUSTER_CTAS_PER_SM = 1024 / CLUSTER_THREADS;
constexpr uint32_t CLUSTER_MAX_TILES = 512;   // records of one (chunk, replica) held in shared memory
constexpr uint32_t CLUSTER_MAX_CTAS = 8;      // portable cluster size: R * split

__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The address of `local` (a shared-memory object of this CTA) in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_address(const void *local, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
    return remote;
}
__device__ __forceinline__ void st_cluster_u64(uint32_t addr, uint64_t v) {
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_record(uint32_t addr, const TileRec &rec) {
    asm volatile("st.shared::cluster.v2.u64 [%0], {%1, %2};" ::"r"(addr), "l"(rec.h),
                 "l"((uint64_t)__double_as_longlong(rec.sum)) : "memory");
    asm volatile("st.shared::cluster.v2.u64 [%0], {%1, %2};" ::"r"(addr + 16u),
                 "l"((uint64_t)__double_as_longlong(rec.sumsq)),
                 "l"((uint64_t)rec.nan_count | ((uint64_t)rec.inf_count << 32)) : "memory");
}

template <int DTSEL>
__global__ void __launch_bounds__(CLUSTER_THREADS, CLUSTER_CTAS_PER_SM) certify_clusters(const __grid_constant__ FusedArgs a) {
    constexpr uint32_t WARPS = CLUSTER_THREADS / 32;
    __shared__ __align__(16) TileRec s_rec[CLUSTER_MAX_TILES];
    __shared__ uint64_t s_hash[WARPS][CLUSTER_MAX_CTAS];   // first CTA: hash of (chunk of the batch, replica)
    __shared__ ChunkDesc s_chunk[WARPS];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t split = a.cluster_split, batch = a.cluster_batch;
    const uint32_t rank = cluster_cta_rank();         // cluster dimension = R * split
    const uint32_t r = rank / split, part = rank - r * split;
    const bool remote = split > 1 || a.mode != 0;     // does anything cross CTAs in this launch?
    // Stores into another CTA's shared memory need that CTA to have started: arrive now,
    // wait when the first loads are on their way.
    if (remote) cluster_arrive();
    const uint32_t warps_per_chunk = WARPS / batch;   // batch > 1 only with split == 1
    const uint64_t c_first = (uint64_t)(blockIdx.x / (a.R * split)) * batch;
    const uint32_t tile_bytes = a.tile_rows * ROW_BYTES;
    const uint32_t b = warp / warps_per_chunk, j0 = warp - b * warps_per_chunk;
    const uint64_t c_scan = c_first + b;
    ChunkDesc cd;
    cd.ntiles = 0;
    const uint8_t *base = nullptr;
    if (c_scan < a.C) {
        cd = a.chunks[c_scan];
        base = a.s.ptrs[(uint64_t)r * a.s.T + cd.tensor] + cd.byte_offset;
    }
    if (remote) cluster_wait();
    if (c_scan < a.C) {
        if (part == 0 && j0 == 0 && lane == 0) s_chunk[b] = cd;
        const uint32_t slot0 = batch > 1 ? b * warps_per_chunk : 0u;
        const uint32_t home = split > 1 ? cluster_address(s_rec, r * split) : 0u;
        for (uint32_t j = part * warps_per_chunk + j0; j < cd.ntiles; j += split * warps_per_chunk) {
            const uint64_t off = (uint64_t)j * tile_bytes;
            const uint32_t nbytes = (uint32_t)min((uint64_t)tile_bytes, cd.nbytes - off);
            TileRec rec;
            if constexpr (DTSEL >= 0) scan_tile<DTSEL, true>(base + off, nbytes, lane, rec);
            else                      scan_dispatch(cd.dtype, base + off, nbytes, lane, rec);
            if (lane == 0) {
                if (split > 1) st_cluster_record(home + (slot0 + j) * (uint32_t)sizeof(TileRec), rec);
                else           s_rec[slot0 + j] = rec;
            }
        }
    }
    // every record of (chunk, replica r) is in the shared memory of the replica's first CTA
    if (split > 1) {
        cluster_arrive();
        cluster_wait();
    } else {
        __syncthreads();
    }
    const uint64_t c = c_first + warp;                // from here on warp b works on chunk b of the batch
    const bool mine = warp < batch && c < a.C;
    if (mine && part == 0) {
        const ChunkDesc my = s_chunk[warp];
        const scout_sig_t o = combine_tiles<true>(s_rec + (batch > 1 ? warp * warps_per_chunk : 0u), my.ntiles,
                                                  my.nbytes, my.k, my.dtype, my.meta, a.p_stride,
                                                  combine_weight(my.ntiles, my.nbytes, a.tile_rows, lane), lane);
        if (lane == 0) {
            a.sigs[c * a.R + r] = o;
            if (a.mode != 0) st_cluster_u64(cluster_address(&s_hash[warp][r], 0), o.hash);
        }
    }
    if (a.mode == 0) return;
    cluster_arrive();
    cluster_wait();      // the R hashes of every chunk of the batch are in the first CTA
    if (rank == 0 && mine) chunk_vote_and_fold(a, (uint32_t)c, lane < a.R ? s_hash[warp][lane] : 0ull, 0ull, lane);
}

using FusedKernel = void (*)(const FusedArgs);
FusedKernel cluster_kernel(int uniform) {
    if (uniform == SCOUT_DT_F32) return certify_clusters<SCOUT_DT_F32>;
    if (uniform == SCOUT_DT_BF16) return certify_clusters<SCOUT_DT_BF16>;
    return certify_clusters<-1>;
}

FusedKernel fused_kernel(int uniform) {
    if (uniform == SCOUT_DT_F32) return certify_tiles<SCOUT_DT_F32>;
    if (uniform == SCOUT_DT_BF16) return certify_tiles<SCOUT_DT_BF16>;
    return certify_tiles<-1>;
}

}  // namespace

int fused_grid_size(int uniform_dtype, int device, int *grid) {
    int sms = 0, per_sm = 0;
    SCOUT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    SCOUT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_kernel(uniform_dtype), SIGN_THREADS, 0));
    if (per_sm < 1) per_sm = 1;
    *grid = sms * per_sm;
    return SCOUT_OK;
}

// Whether the cluster form can run a plan of R replicas whose chunks have at most max_tiles
// tiles on this device, and with which geometry.  Chunks with few tiles are taken `batch`
// at a time, so that every warp of a CTA has a tile; chunks with many tiles are shared by
// `split` CTAs per replica while the cluster stays within its size, every CTA keeps at
// least a tile per warp ...
int cluster_form_possible(int uniform_dtype, uint32_t R, uint32_t max_tiles, uint64_t C, int *ok,
                          uint32_t *batch_out, uint32_t *split_out) {
    *ok = 0;
    constexpr uint32_t WARPS = CLUSTER_THREADS / 32;
    uint32_t batch = 1, split = 1;
    while (batch < WARPS && 2 * batch * max_tiles <= WARPS) batch *= 2;
    // ... and only while all CTAs of the launch are resident at once (two per SM): a second
    // wave of CTAs costs more than the finer split gains (measured: 201 MB in 1 MiB chunks,
    // R = 3, 59 us with 201 CTAs, 68 us with 402)
    int device = 0, sms = 0;
    SCOUT_CUDA(cudaGetDevice(&device));
    SCOUT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    const uint64_t clusters = (C + batch - 1) / batch;
    while (2 * split * R <= CLUSTER_MAX_CTAS && max_tiles >= 2 * split * WARPS &&
           clusters * R * 2 * split <= (uint64_t)CLUSTER_CTAS_PER_SM * (uint64_t)sms)
        split *= 2;
    *batch_out = batch;
    *split_out = split;
    if (R < 1 || R > CLUSTER_MAX_CTAS || max_tiles > CLUSTER_MAX_TILES || C * CLUSTER_MAX_CTAS > 0x7FFFFFFFull || C == 0)
        return SCOUT_OK;
    uint32_t ctas = R;                     // the largest cluster launch_fused may ask for
    while (2 * ctas <= CLUSTER_MAX_CTAS) ctas *= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(CLUSTER_THREADS);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ctas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, cluster_kernel(uniform_dtype), &cfg) != cudaSuccess) {
        cudaGetLastError();
        return SCOUT_OK;
    }
    *ok = n > 0;
    return SCOUT_OK;
}

int launch_fused(const FusedLaunch &l, cudaStream_t stream) {
    if (l.sign.n_tiles == 0 || l.R == 0) return SCOUT_OK;
    FusedArgs a;
    a.s.tiles = l.sign.tiles;
    a.s.tile_begin = 0;
    a.s.n_tiles = l.sign.n_tiles;
    a.s.tiles_per_replica = l.sign.tiles_per_replica;
    a.s.replica_begin = 0;
    a.s.n_replicas = l.R;
    a.s.ptrs = l.sign.ptrs;
    a.s.T = l.sign.T;
    a.s.stage = nullptr;
    a.s.slice_begin = 0;
    a.s.recs = l.sign.recs;
    a.s.error = l.sign.error;
    a.s.work = nullptr;
    a.s.work_parity = 0;
    a.s.work_streams = 1;
    a.chunks = l.chunks;
    a.C = l.C;
    a.R = l.R;
    a.tile_rows = l.tile_rows;
    a.p_stride = pow_p(32ull * l.tile_rows);
    a.sigs = l.sigs;
    a.mode = l.mode;
    a.v = l.vote;
    a.out = l.out;
    a.tickets = l.tickets;
    a.done = l.done;
    a.epoch = l.epoch;
    a.chain = l.chain;
    a.host = l.host;
    a.work = l.work;
    a.one_level = l.one_level;
    a.cluster_batch = 1;
    a.cluster_split = 1;
    if (l.cluster) {
        const uint32_t batch = l.cluster_batch, split = l.cluster_split;
        a.cluster_batch = batch;
        a.cluster_split = split;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(((l.C + batch - 1) / batch) * l.R * split));
        cfg.blockDim = dim3(CLUSTER_THREADS);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = l.R * split;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        SCOUT_CUDA(cudaLaunchKernelEx(&cfg, cluster_kernel(l.sign.uniform_dtype), a));
        return SCOUT_OK;
    }
    const uint64_t items = l.sign.n_tiles * l.R;
    const uint64_t want = (items + SIGN_THREADS / 32 - 1) / (SIGN_THREADS / 32);
    int grid = l.sign.grid;
    if ((uint64_t)grid > want) grid = (int)want;
    fused_kernel(l.sign.uniform_dtype)<<<grid, SIGN_THREADS, 0, stream>>>(a);
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}

}  // namespace scout
