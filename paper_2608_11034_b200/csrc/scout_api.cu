// Host side of the C ABI: plan construction (chunk and tile tables), argument
// validation, launch sequencing, and the certify roll-up.  All arithmetic of the
// method runs in the kernels of scout_sign.cu, scout_one_launch.cu, scout_noalloc.cu and scout_vote.cu.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>

#include "scout_internal.h"

namespace scout {

static thread_local std::string g_last_cuda_error;

void set_cuda_error(cudaError_t e, const char *what) {
    g_last_cuda_error = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " in " + what;
    (void)cudaGetLastError();  // clear the sticky-free error state
}

static uint32_t dtype_size(uint32_t d) {
    switch (d) {
        case SCOUT_DT_U8: return 1;
        case SCOUT_DT_F32: return 4;
        case SCOUT_DT_BF16: return 2;
        case SCOUT_DT_I64: return 8;
        case SCOUT_DT_F16: return 2;
        case SCOUT_DT_F64: return 8;
        case SCOUT_DT_I32: return 4;
        default: return 0;
    }
}

}  // namespace scout

using namespace scout;

constexpr uint32_t MAX_WORK_STREAMS = 32;  // work counters of the direct scan: [2][streams], 128 bytes apart
constexpr size_t WORK_BYTES = 2 * MAX_WORK_STREAMS * 128;
constexpr size_t TIMING_RING = 256;  // event pairs kept for the "timing" knob

struct scout_plan {
    uint32_t R = 0;
    uint64_t T = 0, chunk_bytes = 0;
    std::vector<scout_tensor_t> tensors;
    std::vector<ChunkDesc> chunks;
    std::vector<uint64_t> tensor_chunk0;  // [T+1]
    std::vector<uint64_t> tensor_poff;    // [T+1] packed offsets, 256-byte aligned
    std::vector<TileDesc> tiles;
    uint32_t tile_bytes = 0;
    int variant = 1, device = 0, grid = 0;   // front end of the scan (key "variant"); 1 = register prefetch
    int uniform_dtype = -1;  // dtype of every tensor, or -1 if they differ
    bool bound = false;

    TileDesc *d_tiles = nullptr;
    ChunkDesc *d_chunks = nullptr;
    uint64_t *d_tensor_chunk0 = nullptr;
    const uint8_t **d_ptrs = nullptr;
    TileRec *d_recs = nullptr;
    uint32_t *d_error = nullptr;  // set by a kernel whose bounded wait gave up

    // certify-owned results
    scout_sig_t *d_sigs = nullptr;
    uint8_t *d_status = nullptr;
    uint64_t *d_bitmap = nullptr, *d_majority = nullptr, *d_undecided = nullptr;
    scout_outlier_t *d_outliers = nullptr;
    uint64_t outlier_cap = 0, undecided_cap = 0;
    CertifyOut *d_out = nullptr;
    CertifyHost *h_out = nullptr;  // pinned
    bool have_results = false;

    // one-launch path (certify_tiles): per-chunk tickets, launch stamps, chain state
    int fused = -1;               // key "fused": 1 always, 0 never, -1 where it is the faster form (see
                                  // launch_form); the bulk-async front ends (variants 2, 4) have no one-launch form
    uint64_t total_bytes = 0;     // R * bytes per replica
    int fused_grid = 0;
    int cluster_ok = 0;           // the cluster form of the one-launch path can run this plan (upload_tables)
    uint32_t max_chunk_tiles = 0;
    uint32_t cluster_batch = 1, cluster_split = 1;   // geometry of the cluster form (cluster_form_possible)
    uint32_t *d_tickets = nullptr, *d_done = nullptr;
    ChainState *d_chain = nullptr;
    unsigned long long *d_work = nullptr;   // one-launch kernels
    unsigned long long *d_work2 = nullptr;  // direct scan kernels of the staged path
    uint64_t work_launches = 0;
    bool dynamic = true;                    // key "dynamic"
    uint32_t work_streams = 8;              // key "work_streams": counters the tiles are dealt from (one
                                            // counter hands out about 0.3 G tiles/s: 3 GB in 4 KiB chunks
                                            // scans at 1.8 TB/s with one counter, 5.9 TB/s with eight)
    CertifyHost *h_out_dev = nullptr;  // device-side address of h_out
    uint32_t epoch = 0;
    bool out_dirty = false;       // d_out was left non-zero by the multi-kernel path
    bool pending = false;         // a certify was launched and not collected yet
    cudaStream_t pending_stream = nullptr;
    uint64_t pending_ocap = 0, pending_ucap = 0;

    // host-replica staging
    uint8_t *d_stage[2] = {nullptr, nullptr};
    uint64_t stage_bytes = 0;
    cudaStream_t s_copy = nullptr, s_comp = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr};

    // recorded after the last kernel of every launch sequence: scout_plan_bind waits for it
    // before it rewrites the pointer table
    cudaEvent_t ev_last = nullptr;
    bool launched = false;

    // Debug mode (environment variable SCOUT_DEBUG=1 when the plan is created): every device
    // buffer the plan owns sits between two guard bands of a fixed byte pattern, and
    // scout_plan_get(plan, "guards_ok") checks that no kernel wrote into any of them.
    bool debug = false;
    struct Guarded { uint8_t *user; size_t bytes; };
    std::vector<Guarded> guarded;

    // optional in-stream timing of the scan kernel (key "timing")
    // a ring of event pairs, one per sign launch, so that a caller can time every launch of a
    // loop and read the durations after it
    bool timing = false;
    std::vector<cudaEvent_t> ev_t0, ev_t1;
    uint64_t timed_launches = 0;
};

namespace {

constexpr size_t GUARD_BYTES = 256;
constexpr int GUARD_PATTERN = 0xA5;

// Device allocation for a plan.  In debug mode the buffer is preceded and followed by a
// guard band; the caller gets the address between them (still 256-byte aligned).
cudaError_t plan_malloc(scout_plan *p, void **ptr, size_t bytes) {
    if (!p->debug) return cudaMalloc(ptr, bytes);
    const size_t padded = (bytes + 255) / 256 * 256;   // the rear band starts on a 256-byte boundary
    uint8_t *base = nullptr;
    cudaError_t e = cudaMalloc(&base, padded + 2 * GUARD_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaMemset(base, GUARD_PATTERN, padded + 2 * GUARD_BYTES);
    if (e != cudaSuccess) {
        cudaFree(base);
        return e;
    }
    try {
        p->guarded.push_back({base + GUARD_BYTES, bytes});
    } catch (const std::bad_alloc &) {
        cudaFree(base);
        return cudaErrorMemoryAllocation;
    }
    *ptr = base + GUARD_BYTES;
    return cudaSuccess;
}

void plan_free(scout_plan *p, void *ptr) {
    if (!ptr) return;
    if (p->debug) {
        for (size_t i = 0; i < p->guarded.size(); ++i)
            if (p->guarded[i].user == ptr) {
                p->guarded.erase(p->guarded.begin() + i);
                cudaFree((uint8_t *)ptr - GUARD_BYTES);
                return;
            }
    }
    cudaFree(ptr);
}

// Debug mode: 1 if every guard band of every buffer still holds the pattern.  The bytes
// between the end of a buffer and the next 256-byte boundary count as guard, too.
int guards_intact(const scout_plan *p, int64_t *ok) {
    SCOUT_CUDA(cudaDeviceSynchronize());
    std::vector<uint8_t> host;
    *ok = 1;
    for (const scout_plan::Guarded &g : p->guarded) {
        const size_t padded = (g.bytes + 255) / 256 * 256;
        const size_t rear = padded - g.bytes + GUARD_BYTES;
        host.resize(GUARD_BYTES + rear);
        SCOUT_CUDA(cudaMemcpy(host.data(), g.user - GUARD_BYTES, GUARD_BYTES, cudaMemcpyDeviceToHost));
        SCOUT_CUDA(cudaMemcpy(host.data() + GUARD_BYTES, g.user + g.bytes, rear, cudaMemcpyDeviceToHost));
        for (uint8_t b : host)
            if (b != (uint8_t)GUARD_PATTERN) *ok = 0;
    }
    return SCOUT_OK;
}

// A plan's tables, scratch and events live on the device that was current when it was
// created; using it with another device current would launch on the wrong GPU.
int check_device(const scout_plan *p) {
    int d = -1;
    SCOUT_CUDA(cudaGetDevice(&d));
    return d == p->device ? SCOUT_OK : SCOUT_ERR_INVALID;
}

// Marks the end of a launch sequence on `stream` (see scout_plan_bind).
int mark_launched(scout_plan *p, cudaStream_t stream) {
    SCOUT_CUDA(cudaEventRecord(p->ev_last, stream));
    p->launched = true;
    return SCOUT_OK;
}

uint32_t auto_tile_bytes(uint64_t total_bytes, int uniform_dtype) {
    // About two work items per resident warp, 4 KiB .. 32 KiB, power of two (measured:
    // 12.6 MB is fastest with 4 KiB tiles, 201 MB with 16 KiB, fp32 and mixed plans of 1 GB and
    // more with 32 KiB).  Large plans of 16-bit floats are bound by instruction issue, not by
    // HBM, and gain from fewer tile boundaries: 128 KiB (measured on 125 GB of bf16: 6,350 GB/s
    // with 32 KiB tiles, 6,450 with 64 KiB, 6,500 with 128 KiB; fp32 loses 3 % beyond 32 KiB).
    const uint64_t want_items = 148ull * 32 * 2;
    uint64_t t = total_bytes / want_items;
    uint32_t tile = 4096;
    while (tile < 32768 && (uint64_t)tile * 2 <= t) tile *= 2;
    const bool half_floats = uniform_dtype == SCOUT_DT_BF16 || uniform_dtype == SCOUT_DT_F16;
    if (half_floats && total_bytes >= (4ull << 30)) tile = 131072;
    return tile;
}

void build_tiles(scout_plan *p) {
    p->tiles.clear();
    for (uint64_t c = 0; c < p->chunks.size(); ++c) {
        ChunkDesc &cd = p->chunks[c];
        cd.tile0 = p->tiles.size();
        uint32_t n = 0;
        for (uint64_t o = 0; o < cd.nbytes; o += p->tile_bytes, ++n) {
            TileDesc td;
            td.off = cd.byte_offset + o;
            td.poff = p->tensor_poff[cd.tensor] + td.off;
            td.tensor = cd.tensor;
            td.nbytes = (uint32_t)std::min<uint64_t>(p->tile_bytes, cd.nbytes - o);
            td.chunk = (uint32_t)c;
            td.dtype = cd.dtype;
            p->tiles.push_back(td);
        }
        cd.ntiles = n;
        for (uint32_t j = 0; j < n; ++j) p->tiles[cd.tile0 + j].chunk_tiles = n;
    }
}

int upload_tables(scout_plan *p) {
    if (p->d_tiles) { plan_free(p, p->d_tiles); p->d_tiles = nullptr; }
    if (p->d_recs) { plan_free(p, p->d_recs); p->d_recs = nullptr; }
    if (p->d_chunks) { plan_free(p, p->d_chunks); p->d_chunks = nullptr; }
    const size_t nt = p->tiles.size(), nc = p->chunks.size();
    SCOUT_CUDA(plan_malloc(p, (void **)&p->d_tiles, nt * sizeof(TileDesc)));
    SCOUT_CUDA(plan_malloc(p, (void **)&p->d_chunks, nc * sizeof(ChunkDesc)));
    SCOUT_CUDA(plan_malloc(p, (void **)&p->d_recs, nt * p->R * sizeof(TileRec)));
    SCOUT_CUDA(cudaMemcpy(p->d_tiles, p->tiles.data(), nt * sizeof(TileDesc), cudaMemcpyHostToDevice));
    SCOUT_CUDA(cudaMemcpy(p->d_chunks, p->chunks.data(), nc * sizeof(ChunkDesc), cudaMemcpyHostToDevice));
    p->max_chunk_tiles = 0;
    for (const ChunkDesc &cd : p->chunks) p->max_chunk_tiles = std::max(p->max_chunk_tiles, cd.ntiles);
    return cluster_form_possible(p->uniform_dtype, p->R, p->max_chunk_tiles, nc, &p->cluster_ok,
                                 &p->cluster_batch, &p->cluster_split);
}

// How a call is launched: 0 = one kernel per stage (scan, finalise, vote, certificate chain,
// linked by programmatic dependent launch), 1 = one kernel with tickets (certify_tiles),
// 2 = one kernel with a thread-block cluster per chunk (certify_clusters).  Key "fused":
// 0, 1, 2 force a form (2 only where it can run, else 1); -1, the default, follows what was
// measured on B200 (device time of scout_certify, L2 flushed between calls):
//   * scout_certify on a plan below 1 GiB whose chunks have at most 64 tiles and which has
//     at most 1,024 chunks, R <= 8: clusters.  12.6 MB in 64 KiB chunks: 25 us against 29
//     (tickets) and 33 (per stage); 50 MB in 256 KiB chunks: 33 against 57 and 46; 201 MB in
//     1 MiB chunks: 59-68 against 74-84 and 69-73; 900 MiB in 1 MiB chunks: 188 against 204
//     and 191.  With more chunks (1,024, or one per 300 KiB of the plan if that is more) the
//     sequential certificate chain (32 ns per chunk) decides and the per-stage form is as
//     fast; with more tiles per chunk too few CTAs stream (a CTA has 64 KiB in flight, about
//     50 GB/s).  Plans of 16-bit floats above 256 MiB: per stage (their row routine bounds an
//     SM at 47-49 GB/s, so the uneven spread of CTAs over SMs costs 11 % at 900 MiB).
//   * scout_certify on other plans up to 16 MiB whose chunks have at most 64 tiles (in
//     practice: more than 8 replicas): tickets (29-35 us against 33-40).
//   * everything else: per stage.  With its work handed out dynamically the staged scan
//     reaches 7.2 TB/s on 36 GB of fp32 and 6.5 TB/s on 125 GB of bf16; the ticket kernel
//     stays 3 to 9 % below that, more than the three small launches it saves.
int launch_form(const scout_plan *p, bool certify) {
    if (p->variant > 1 || p->R > 64 || !p->d_tickets || p->fused == 0) return 0;
    if (p->fused == 2) return p->cluster_ok ? 2 : 1;
    if (p->fused == 1) return 1;
    if (!certify || p->total_bytes >= (1ull << 30)) return 0;
    const bool half_floats = p->uniform_dtype == SCOUT_DT_BF16 || p->uniform_dtype == SCOUT_DT_F16;
    const uint64_t max_chunks = std::max<uint64_t>(1024, p->total_bytes / (300ull << 10));
    if (p->cluster_ok && p->max_chunk_tiles <= 64 * p->cluster_split && p->chunks.size() <= max_chunks &&
        (!half_floats || p->total_bytes <= (256ull << 20)))
        return 2;
    return (p->total_bytes <= (16ull << 20) && p->max_chunk_tiles <= 64) ? 1 : 0;
}

void fill_sign_launch(const scout_plan *p, SignLaunch &l) {
    l.tiles = p->d_tiles;
    l.tile_begin = 0;
    l.n_tiles = p->tiles.size();
    l.tiles_per_replica = p->tiles.size();
    l.replica_begin = 0;
    l.n_replicas = p->R;
    l.ptrs = (const uint8_t *const *)p->d_ptrs;
    l.T = p->T;
    l.stage = nullptr;
    l.slice_begin = 0;
    l.recs = p->d_recs;
    l.error = p->d_error;
    l.variant = p->variant;
    l.uniform_dtype = p->uniform_dtype;
    l.grid = p->grid;
    l.work = nullptr;
    l.work_parity = 0;
    l.work_streams = 1;
}

// The direct scan kernels take their work dynamically: successive launches alternate between
// the plan's two counters (the launch that uses one zeroes the other).
void next_work_counter(scout_plan *p, SignLaunch &l) {
    l.work = p->dynamic ? p->d_work2 : nullptr;
    l.work_parity = (p->work_launches++) & 1u;
    l.work_streams = p->work_streams;
}

// One kernel: scan + finalise (certify == false), or the whole certify path.  The timing
// events bracket that kernel.
int launch_one_kernel(scout_plan *p, cudaStream_t stream, scout_sig_t *d_sigs, bool certify,
                      uint64_t outlier_cap, uint64_t undecided_cap) {
    FusedLaunch f;
    std::memset(&f, 0, sizeof(f));
    fill_sign_launch(p, f.sign);
    f.sign.grid = p->fused_grid;
    f.chunks = p->d_chunks;
    f.C = p->chunks.size();
    f.R = p->R;
    f.tile_rows = p->tile_bytes / ROW_BYTES;
    f.sigs = d_sigs;
    f.mode = certify ? 1 : 0;
    f.tickets = p->d_tickets;
    f.work = p->d_work;
    f.one_level = (uint64_t)p->max_chunk_tiles * p->R <= 64 ? 1u : 0u;
    f.cluster = launch_form(p, certify) == 2 ? 1 : 0;
    f.cluster_batch = p->cluster_batch;
    f.cluster_split = p->cluster_split;
    if (++p->epoch == 0) p->epoch = 1;  // 0 is the stamp of "never"
    f.epoch = p->epoch;
    if (certify) {
        if (p->out_dirty) {
            SCOUT_CUDA(cudaMemsetAsync(p->d_out, 0, sizeof(CertifyOut), stream));
            p->out_dirty = false;
        }
        f.vote = VoteSinks{p->d_status, p->d_bitmap, p->d_majority, p->d_outliers, outlier_cap,
                           p->d_undecided, undecided_cap, p->d_out->counts, p->d_out};
        f.out = p->d_out;
        f.done = p->d_done;
        f.chain = p->d_chain;
        f.host = p->h_out_dev;
    }
    const size_t slot = p->timing ? (size_t)(p->timed_launches % p->ev_t0.size()) : 0;
    if (p->timing) SCOUT_CUDA(cudaEventRecord(p->ev_t0[slot], stream));
    int rc = launch_fused(f, stream);
    if (rc) return rc;
    if (p->timing) {
        SCOUT_CUDA(cudaEventRecord(p->ev_t1[slot], stream));
        p->timed_launches += 1;
    }
    return mark_launched(p, stream);
}

int sign_all(scout_plan *p, cudaStream_t stream, scout_sig_t *d_sigs, CertifyOut *zero_out = nullptr) {
    if (launch_form(p, false) && !zero_out) return launch_one_kernel(p, stream, d_sigs, false, 0, 0);
    SignLaunch l;
    fill_sign_launch(p, l);
    next_work_counter(p, l);
    const size_t slot = p->timing ? (size_t)(p->timed_launches % p->ev_t0.size()) : 0;
    if (p->timing) SCOUT_CUDA(cudaEventRecord(p->ev_t0[slot], stream));
    int rc = launch_sign_tiles(l, stream);
    if (rc) return rc;
    if (p->timing) {
        SCOUT_CUDA(cudaEventRecord(p->ev_t1[slot], stream));
        p->timed_launches += 1;
    }
    rc = launch_finalize(p->d_chunks, p->chunks.size(), p->R, p->d_recs, p->tiles.size(),
                         p->tile_bytes / ROW_BYTES, p->max_chunk_tiles, d_sigs, zero_out, stream);
    if (rc) return rc;
    return mark_launched(p, stream);
}

int ensure_certify_buffers(scout_plan *p, uint64_t outlier_cap, uint64_t undecided_cap) {
    const uint64_t C = p->chunks.size();
    if (!p->d_sigs) {
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_sigs, C * p->R * sizeof(scout_sig_t)));
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_status, C));
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_bitmap, C * sizeof(uint64_t)));
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_majority, C * sizeof(uint64_t)));
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_out, sizeof(CertifyOut)));
        SCOUT_CUDA(cudaMemset(p->d_out, 0, sizeof(CertifyOut)));
        SCOUT_CUDA(cudaHostAlloc(&p->h_out, sizeof(CertifyHost), cudaHostAllocMapped));
        SCOUT_CUDA(cudaHostGetDevicePointer((void **)&p->h_out_dev, p->h_out, 0));
    }
    if (!p->d_outliers || outlier_cap > p->outlier_cap) {
        if (p->d_outliers) plan_free(p, p->d_outliers);
        p->d_outliers = nullptr;
        p->outlier_cap = std::max<uint64_t>(outlier_cap, 1);
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_outliers, p->outlier_cap * sizeof(scout_outlier_t)));
    }
    if (!p->d_undecided || undecided_cap > p->undecided_cap) {
        if (p->d_undecided) plan_free(p, p->d_undecided);
        p->d_undecided = nullptr;
        p->undecided_cap = std::max<uint64_t>(undecided_cap, 1);
        SCOUT_CUDA(plan_malloc(p, (void **)&p->d_undecided, p->undecided_cap * sizeof(uint64_t)));
    }
    return SCOUT_OK;
}

// Multi-kernel path: vote + certificate + speculative copies of the report block, after
// d_sigs is ready on `stream` (the finalise kernel that precedes this cleared d_out).
int enqueue_vote_and_copies(scout_plan *p, cudaStream_t stream, uint64_t outlier_cap, uint64_t undecided_cap) {
    const uint64_t C = p->chunks.size();
    int rc = launch_vote(p->R, C, p->d_sigs, p->d_status, p->d_bitmap, p->d_outliers, outlier_cap,
                         p->d_undecided, undecided_cap, p->d_out->counts, p->d_majority, p->d_out, true,
                         stream);
    if (rc) return rc;
    rc = launch_certificate(C, p->d_majority, p->d_out, stream);
    if (rc) return rc;
    p->out_dirty = true;
    // One round trip in the common case: the counters, the error flag and the head of
    // both lists are copied speculatively; longer lists need a second copy.
    CertifyHost *hh = p->h_out;
    const uint64_t head_out = std::min<uint64_t>(outlier_cap, CERTIFY_HEAD);
    const uint64_t head_und = std::min<uint64_t>(undecided_cap, CERTIFY_HEAD);
    SCOUT_CUDA(cudaMemcpyAsync(&hh->out, p->d_out, sizeof(CertifyOut), cudaMemcpyDeviceToHost, stream));
    SCOUT_CUDA(cudaMemcpyAsync(&hh->dev_err, p->d_error, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    if (head_out)
        SCOUT_CUDA(cudaMemcpyAsync(hh->outliers, p->d_outliers, head_out * sizeof(scout_outlier_t),
                                   cudaMemcpyDeviceToHost, stream));
    if (head_und)
        SCOUT_CUDA(cudaMemcpyAsync(hh->undecided, p->d_undecided, head_und * sizeof(uint64_t),
                                   cudaMemcpyDeviceToHost, stream));
    return SCOUT_OK;
}

// Waits for the launched certify and turns the report block (in pinned host memory, written
// by copies or by the one-launch kernel itself) into the caller's report and canonical lists.
int collect_report(scout_plan *p, cudaStream_t stream, scout_report_t *report,
                   scout_outlier_t *h_outliers, uint64_t outlier_cap, uint64_t *h_undecided,
                   uint64_t undecided_cap) {
    SCOUT_CUDA(cudaStreamSynchronize(stream));
    p->pending = false;
    CertifyHost *hh = p->h_out;
    const uint64_t head_out = std::min<uint64_t>(outlier_cap, CERTIFY_HEAD);
    const uint64_t head_und = std::min<uint64_t>(undecided_cap, CERTIFY_HEAD);
    const CertifyOut &o = hh->out;
    const uint64_t n_out = std::min<uint64_t>(o.counts[4], outlier_cap);
    const uint64_t n_und = std::min<uint64_t>(o.counts[5], undecided_cap);
    std::memcpy(h_outliers, hh->outliers, std::min(n_out, head_out) * sizeof(scout_outlier_t));
    std::memcpy(h_undecided, hh->undecided, std::min(n_und, head_und) * sizeof(uint64_t));
    if (n_out > head_out)
        SCOUT_CUDA(cudaMemcpyAsync(h_outliers + head_out, p->d_outliers + head_out,
                                   (n_out - head_out) * sizeof(scout_outlier_t), cudaMemcpyDeviceToHost,
                                   stream));
    if (n_und > head_und)
        SCOUT_CUDA(cudaMemcpyAsync(h_undecided + head_und, p->d_undecided + head_und,
                                   (n_und - head_und) * sizeof(uint64_t), cudaMemcpyDeviceToHost, stream));
    if (n_out > head_out || n_und > head_und) SCOUT_CUDA(cudaStreamSynchronize(stream));
    // device lists are in arrival order; the host lists are canonical
    std::sort(h_outliers, h_outliers + n_out, [](const scout_outlier_t &a, const scout_outlier_t &b) {
        return a.chunk != b.chunk ? a.chunk < b.chunk : a.replica < b.replica;
    });
    std::sort(h_undecided, h_undecided + n_und);
    std::memset(report, 0, sizeof(*report));
    report->n_chunks = o.counts[0];
    report->n_agree = o.counts[1];
    report->n_attributed = o.counts[2];
    report->n_inconclusive = o.counts[3];
    report->n_outliers = o.counts[4];
    report->n_undecided = o.counts[5];
    report->replica_union_bitmap = o.union_bitmap;
    report->certificate = o.certificate;
    report->verdict = o.counts[3] ? SCOUT_UNDECIDED
                                  : (o.counts[2] ? SCOUT_VERDICT_ATTRIBUTED : SCOUT_CERTIFIED);
    p->have_results = true;
    if (hh->dev_err) {
        // reported once: the flag is cleared so that the next run starts clean
        SCOUT_CUDA(cudaMemsetAsync(p->d_error, 0, sizeof(uint32_t), stream));
        SCOUT_CUDA(cudaStreamSynchronize(stream));
        set_cuda_error(cudaErrorUnknown, "scan kernel: a bounded wait for a bulk copy gave up");
        return SCOUT_ERR_CUDA;
    }
    return (o.counts[4] > outlier_cap || o.counts[5] > undecided_cap) ? SCOUT_ERR_TRUNCATED : SCOUT_OK;
}

int vote_and_report(scout_plan *p, cudaStream_t stream, scout_report_t *report,
                    scout_outlier_t *h_outliers, uint64_t outlier_cap, uint64_t *h_undecided,
                    uint64_t undecided_cap) {
    int rc = enqueue_vote_and_copies(p, stream, outlier_cap, undecided_cap);
    if (rc) return rc;
    return collect_report(p, stream, report, h_outliers, outlier_cap, h_undecided, undecided_cap);
}

// Enqueues one certify run on `stream` (either path); collect_report() finishes it.
int certify_enqueue(scout_plan *p, cudaStream_t stream, uint64_t outlier_cap, uint64_t undecided_cap) {
    int rc = ensure_certify_buffers(p, outlier_cap, undecided_cap);
    if (rc) return rc;
    if (launch_form(p, true)) {
        rc = launch_one_kernel(p, stream, p->d_sigs, true, outlier_cap, undecided_cap);
    } else {
        if ((rc = sign_all(p, stream, p->d_sigs, p->d_out))) return rc;
        rc = enqueue_vote_and_copies(p, stream, outlier_cap, undecided_cap);
    }
    if (rc) return rc;
    p->pending = true;
    p->pending_stream = stream;
    p->pending_ocap = outlier_cap;
    p->pending_ucap = undecided_cap;
    return SCOUT_OK;
}

}  // namespace

extern "C" {

int scout_plan_create(uint32_t R, uint64_t T, const scout_tensor_t *tensors, uint64_t chunk_bytes,
                      scout_plan_t **out) {
    if (!out) return SCOUT_ERR_INVALID;
    *out = nullptr;
    if (R < 1 || !tensors || T == 0) return SCOUT_ERR_INVALID;
    if (R > SCOUT_MAX_REPLICAS) return SCOUT_ERR_UNSUPPORTED;
    if (chunk_bytes == 0 || chunk_bytes % ROW_BYTES != 0 || chunk_bytes > (1ull << 30))
        return SCOUT_ERR_INVALID;
    if (T > 0xFFFFFFFFull) return SCOUT_ERR_UNSUPPORTED;
    scout_plan *p = new (std::nothrow) scout_plan;
    if (!p) return SCOUT_ERR_NOMEM;
    p->R = R;
    p->T = T;
    p->chunk_bytes = chunk_bytes;
    const char *dbg = std::getenv("SCOUT_DEBUG");
    p->debug = dbg && dbg[0] && dbg[0] != '0';
    uint64_t total = 0, poff = 0;
    try {
        p->tensors.assign(tensors, tensors + T);
        p->tensor_chunk0.resize(T + 1);
        p->tensor_poff.resize(T + 1);
        for (uint64_t t = 0; t < T; ++t) {
            const scout_tensor_t &tn = tensors[t];
            const uint32_t es = dtype_size(tn.dtype);
            if (es == 0 || tn.nbytes == 0 || tn.nbytes % es != 0 || tn.reserved != 0) {
                delete p;
                return SCOUT_ERR_INVALID;
            }
            p->tensor_chunk0[t] = p->chunks.size();
            p->tensor_poff[t] = poff;
            poff += (tn.nbytes + 255) / 256 * 256;
            total += tn.nbytes;
            uint64_t k = 0;
            for (uint64_t o = 0; o < tn.nbytes; o += chunk_bytes, ++k) {
                ChunkDesc cd;
                std::memset(&cd, 0, sizeof(cd));
                cd.nbytes = std::min<uint64_t>(chunk_bytes, tn.nbytes - o);
                cd.k = k;
                cd.meta = tn.meta_tag;
                cd.dtype = tn.dtype;
                cd.tensor = (uint32_t)t;
                cd.byte_offset = o;
                p->chunks.push_back(cd);
            }
        }
        p->uniform_dtype = (int)tensors[0].dtype;
        for (uint64_t t = 1; t < T; ++t)
            if ((int)tensors[t].dtype != p->uniform_dtype) p->uniform_dtype = -1;
        p->tensor_chunk0[T] = p->chunks.size();
        p->tensor_poff[T] = poff;
        if (p->chunks.size() > 0xFFFFFFFFull) {
            delete p;
            return SCOUT_ERR_UNSUPPORTED;
        }
        p->total_bytes = total * R;
        p->tile_bytes = auto_tile_bytes(total * R, p->uniform_dtype);
        build_tiles(p);
    } catch (const std::bad_alloc &) {
        delete p;
        return SCOUT_ERR_NOMEM;
    }
    int rc = SCOUT_OK;
    do {
        if (cudaGetDevice(&p->device) != cudaSuccess) { rc = SCOUT_ERR_CUDA; break; }
        if ((rc = sign_grid_size(p->variant, p->uniform_dtype, p->device, &p->grid))) break;
        if ((rc = upload_tables(p))) break;
        if (plan_malloc(p, (void **)&p->d_tensor_chunk0, (T + 1) * sizeof(uint64_t)) != cudaSuccess ||
            plan_malloc(p, (void **)&p->d_ptrs, (size_t)R * T * sizeof(void *)) != cudaSuccess ||
            plan_malloc(p, (void **)&p->d_error, sizeof(uint32_t)) != cudaSuccess) {
            rc = SCOUT_ERR_NOMEM;
            break;
        }
        const size_t nc = p->chunks.size();
        const size_t n_tickets = nc * R + nc;  // one per (chunk, replica), then one per chunk
        if (plan_malloc(p, (void **)&p->d_tickets, n_tickets * sizeof(uint32_t)) != cudaSuccess ||
            plan_malloc(p, (void **)&p->d_done, nc * sizeof(uint32_t)) != cudaSuccess ||
            plan_malloc(p, (void **)&p->d_chain, sizeof(ChainState)) != cudaSuccess ||
            plan_malloc(p, (void **)&p->d_work, 2 * sizeof(unsigned long long)) != cudaSuccess ||
            plan_malloc(p, (void **)&p->d_work2, WORK_BYTES) != cudaSuccess) {
            rc = SCOUT_ERR_NOMEM;
            break;
        }
        if (cudaMemset(p->d_tickets, 0, n_tickets * sizeof(uint32_t)) != cudaSuccess ||
            cudaMemset(p->d_done, 0, nc * sizeof(uint32_t)) != cudaSuccess ||
            cudaMemset(p->d_chain, 0, sizeof(ChainState)) != cudaSuccess ||
            cudaMemset(p->d_work, 0, 2 * sizeof(unsigned long long)) != cudaSuccess ||
            cudaMemset(p->d_work2, 0, WORK_BYTES) != cudaSuccess) {
            rc = SCOUT_ERR_CUDA;
            break;
        }
        if ((rc = fused_grid_size(p->uniform_dtype, p->device, &p->fused_grid))) break;
        if (cudaMemset(p->d_error, 0, sizeof(uint32_t)) != cudaSuccess ||
            cudaEventCreateWithFlags(&p->ev_last, cudaEventDisableTiming) != cudaSuccess) {
            rc = SCOUT_ERR_CUDA;
            break;
        }
        if (cudaMemcpy(p->d_tensor_chunk0, p->tensor_chunk0.data(), (T + 1) * sizeof(uint64_t),
                       cudaMemcpyHostToDevice) != cudaSuccess) {
            rc = SCOUT_ERR_CUDA;
            break;
        }
    } while (0);
    if (rc) {
        scout_plan_destroy(p);
        return rc;
    }
    *out = p;
    return SCOUT_OK;
}

int scout_plan_bind(scout_plan_t *p, const void *const *ptrs) {
    if (!p || !ptrs) return SCOUT_ERR_INVALID;
    const uint64_t n = (uint64_t)p->R * p->T;
    for (uint64_t i = 0; i < n; ++i) {
        if (!ptrs[i]) return SCOUT_ERR_INVALID;
        if ((uintptr_t)ptrs[i] & 15u) return SCOUT_ERR_ALIGN;
    }
    int rc = check_device(p);
    if (rc) return rc;
    // a scan that is still running reads the table: wait for the plan's last launch first
    if (p->launched) SCOUT_CUDA(cudaEventSynchronize(p->ev_last));
    SCOUT_CUDA(cudaMemcpy(p->d_ptrs, ptrs, n * sizeof(void *), cudaMemcpyHostToDevice));
    p->bound = true;
    return SCOUT_OK;
}

int scout_plan_num_chunks(const scout_plan_t *p, uint64_t *C) {
    if (!p || !C) return SCOUT_ERR_INVALID;
    *C = p->chunks.size();
    return SCOUT_OK;
}

int scout_plan_chunk_info(const scout_plan_t *p, uint64_t c, uint64_t *tensor, uint64_t *index_in_tensor,
                          uint64_t *byte_offset, uint64_t *nbytes) {
    if (!p || c >= p->chunks.size()) return SCOUT_ERR_INVALID;
    const ChunkDesc &cd = p->chunks[c];
    if (tensor) *tensor = cd.tensor;
    if (index_in_tensor) *index_in_tensor = cd.k;
    if (byte_offset) *byte_offset = cd.byte_offset;
    if (nbytes) *nbytes = cd.nbytes;
    return SCOUT_OK;
}

int scout_plan_destroy(scout_plan_t *p) {
    if (!p) return SCOUT_OK;
    plan_free(p, p->d_tiles);
    plan_free(p, p->d_chunks);
    plan_free(p, p->d_tensor_chunk0);
    plan_free(p, (void *)p->d_ptrs);
    plan_free(p, p->d_recs);
    plan_free(p, p->d_error);
    plan_free(p, p->d_tickets);
    plan_free(p, p->d_done);
    plan_free(p, p->d_chain);
    plan_free(p, p->d_work);
    plan_free(p, p->d_work2);
    plan_free(p, p->d_sigs);
    plan_free(p, p->d_status);
    plan_free(p, p->d_bitmap);
    plan_free(p, p->d_majority);
    plan_free(p, p->d_undecided);
    plan_free(p, p->d_outliers);
    plan_free(p, p->d_out);
    if (p->h_out) cudaFreeHost(p->h_out);
    for (int i = 0; i < 2; ++i) {
        plan_free(p, p->d_stage[i]);
        if (p->ev_copied[i]) cudaEventDestroy(p->ev_copied[i]);
        if (p->ev_done[i]) cudaEventDestroy(p->ev_done[i]);
    }
    if (p->s_copy) cudaStreamDestroy(p->s_copy);
    if (p->s_comp) cudaStreamDestroy(p->s_comp);
    if (p->ev_last) cudaEventDestroy(p->ev_last);
    for (cudaEvent_t e : p->ev_t0) cudaEventDestroy(e);
    for (cudaEvent_t e : p->ev_t1) cudaEventDestroy(e);
    (void)cudaGetLastError();
    delete p;
    return SCOUT_OK;
}

int scout_sign_chunks(scout_plan_t *p, void *stream, scout_sig_t *d_sigs) {
    if (!p || !d_sigs) return SCOUT_ERR_INVALID;
    if (!p->bound) return SCOUT_ERR_INVALID;
    int rc = check_device(p);
    if (rc) return rc;
    return sign_all(p, (cudaStream_t)stream, d_sigs);
}

int scout_consensus_vote(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint8_t *d_status,
                         uint64_t *d_bitmap, scout_outlier_t *d_outliers, uint64_t outlier_cap,
                         uint64_t *d_undecided, uint64_t undecided_cap, uint64_t *d_counts,
                         void *stream) {
    if (R < 2) return SCOUT_ERR_INVALID;
    if (R > 64) return SCOUT_ERR_UNSUPPORTED;
    if (!d_counts || (C && !d_sigs)) return SCOUT_ERR_INVALID;
    if ((outlier_cap && !d_outliers) || (undecided_cap && !d_undecided)) return SCOUT_ERR_INVALID;
    return launch_vote(R, C, d_sigs, d_status, d_bitmap, d_outliers, outlier_cap, d_undecided,
                       undecided_cap, d_counts, nullptr, nullptr, false, (cudaStream_t)stream);
}

int scout_consensus_vote_wide(uint32_t R, uint64_t C, const scout_sig_t *d_sigs, uint64_t chunk_stride,
                              uint64_t replica_stride, uint8_t *d_status, uint64_t *d_bitmap,
                              scout_outlier_t *d_outliers, uint64_t outlier_cap, uint64_t *d_undecided,
                              uint64_t undecided_cap, uint64_t *d_counts, void *stream) {
    if (R < 2) return SCOUT_ERR_INVALID;
    if (R > SCOUT_MAX_REPLICAS) return SCOUT_ERR_UNSUPPORTED;
    if (!d_counts || (C && !d_sigs) || chunk_stride == 0 || replica_stride == 0) return SCOUT_ERR_INVALID;
    if ((outlier_cap && !d_outliers) || (undecided_cap && !d_undecided)) return SCOUT_ERR_INVALID;
    return launch_vote_wide(R, C, d_sigs, chunk_stride, replica_stride, d_status, d_bitmap, d_outliers,
                            outlier_cap, d_undecided, undecided_cap, d_counts, (cudaStream_t)stream);
}

int scout_certify_launch(scout_plan_t *p, void *stream, uint64_t outlier_cap, uint64_t undecided_cap) {
    if (!p || !p->bound || p->R < 2) return SCOUT_ERR_INVALID;
    if (p->R > 64) return SCOUT_ERR_UNSUPPORTED;
    if (p->pending) return SCOUT_ERR_INVALID;  // one run in flight per plan: collect it first
    int rc = check_device(p);
    if (rc) return rc;
    return certify_enqueue(p, (cudaStream_t)stream, outlier_cap, undecided_cap);
}

int scout_certify_collect(scout_plan_t *p, scout_report_t *report, scout_outlier_t *h_outliers,
                          uint64_t outlier_cap, uint64_t *h_undecided, uint64_t undecided_cap) {
    if (!p || !report || !p->pending) return SCOUT_ERR_INVALID;
    if ((outlier_cap && !h_outliers) || (undecided_cap && !h_undecided)) return SCOUT_ERR_INVALID;
    if (outlier_cap > p->pending_ocap || undecided_cap > p->pending_ucap) return SCOUT_ERR_INVALID;
    int rc = check_device(p);
    if (rc) return rc;
    // the device lists were cut at the capacities given at launch
    return collect_report(p, p->pending_stream, report, h_outliers, outlier_cap, h_undecided, undecided_cap);
}

int scout_certify(scout_plan_t *p, void *stream, scout_report_t *report, scout_outlier_t *h_outliers,
                  uint64_t outlier_cap, uint64_t *h_undecided, uint64_t undecided_cap) {
    if (!p || !report || !p->bound || p->R < 2) return SCOUT_ERR_INVALID;
    if (p->R > 64) return SCOUT_ERR_UNSUPPORTED;
    if ((outlier_cap && !h_outliers) || (undecided_cap && !h_undecided)) return SCOUT_ERR_INVALID;
    if (p->pending) return SCOUT_ERR_INVALID;
    int rc = check_device(p);
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    if ((rc = certify_enqueue(p, s, outlier_cap, undecided_cap))) return rc;
    return collect_report(p, s, report, h_outliers, outlier_cap, h_undecided, undecided_cap);
}

int scout_certify_host(scout_plan_t *p, const void *const *h_ptrs, scout_report_t *report,
                       scout_outlier_t *h_outliers, uint64_t outlier_cap, uint64_t *h_undecided,
                       uint64_t undecided_cap) {
    if (!p || !h_ptrs || !report || p->R < 2) return SCOUT_ERR_INVALID;
    if (p->R > 64) return SCOUT_ERR_UNSUPPORTED;
    if ((outlier_cap && !h_outliers) || (undecided_cap && !h_undecided)) return SCOUT_ERR_INVALID;
    const uint64_t n = (uint64_t)p->R * p->T;
    for (uint64_t i = 0; i < n; ++i)
        if (!h_ptrs[i]) return SCOUT_ERR_INVALID;
    int rc = check_device(p);
    if (rc) return rc;
    if ((rc = ensure_certify_buffers(p, outlier_cap, undecided_cap))) return rc;
    const uint64_t packed = p->tensor_poff[p->T];
    if (!p->s_copy) {
        SCOUT_CUDA(cudaStreamCreateWithFlags(&p->s_copy, cudaStreamNonBlocking));
        SCOUT_CUDA(cudaStreamCreateWithFlags(&p->s_comp, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            SCOUT_CUDA(cudaEventCreateWithFlags(&p->ev_copied[i], cudaEventDisableTiming));
            SCOUT_CUDA(cudaEventCreateWithFlags(&p->ev_done[i], cudaEventDisableTiming));
        }
        p->stage_bytes = std::min<uint64_t>(packed, 256ull << 20);
        p->stage_bytes = std::max<uint64_t>(p->stage_bytes, (uint64_t)p->tile_bytes + 256);
        for (int i = 0; i < 2; ++i) SCOUT_CUDA(plan_malloc(p, (void **)&p->d_stage[i], p->stage_bytes));
    }
    const uint64_t NT = p->tiles.size();
    uint64_t slice = 0;
    for (uint32_t r = 0; r < p->R; ++r) {
        uint64_t t0 = 0;
        while (t0 < NT) {
            // largest run of tiles whose packed extent fits the staging buffer
            const uint64_t a = p->tiles[t0].poff;
            uint64_t t1 = t0;
            while (t1 < NT && p->tiles[t1].poff + p->tiles[t1].nbytes - a <= p->stage_bytes) ++t1;
            const uint64_t b = p->tiles[t1 - 1].poff + p->tiles[t1 - 1].nbytes;
            const int buf = (int)(slice & 1);
            if (slice >= 2) SCOUT_CUDA(cudaStreamWaitEvent(p->s_copy, p->ev_done[buf], 0));
            // One copy per run of tensors that sit in host memory exactly as in the packed
            // image (same spacing, so only alignment padding of < 256 bytes lies between
            // them): a replica kept as one flat buffer is copied slice by slice instead of
            // tensor by tensor.
            const uint8_t *run_src = nullptr;
            uint64_t run_dst = 0, run_len = 0;
            for (uint32_t t = p->tiles[t0].tensor; t <= p->tiles[t1 - 1].tensor; ++t) {
                const uint64_t lo = std::max<uint64_t>(a, p->tensor_poff[t]);
                const uint64_t hi = std::min<uint64_t>(b, p->tensor_poff[t] + p->tensors[t].nbytes);
                if (hi <= lo) continue;
                const uint8_t *src = (const uint8_t *)h_ptrs[(uint64_t)r * p->T + t] + (lo - p->tensor_poff[t]);
                const uint64_t dst = lo - a;
                if (run_len && src - run_src == (ptrdiff_t)(dst - run_dst) && dst - run_dst >= run_len &&
                    dst - run_dst - run_len < 256) {
                    run_len = dst - run_dst + (hi - lo);
                    continue;
                }
                if (run_len)
                    SCOUT_CUDA(cudaMemcpyAsync(p->d_stage[buf] + run_dst, run_src, run_len,
                                               cudaMemcpyHostToDevice, p->s_copy));
                run_src = src;
                run_dst = dst;
                run_len = hi - lo;
            }
            if (run_len)
                SCOUT_CUDA(cudaMemcpyAsync(p->d_stage[buf] + run_dst, run_src, run_len,
                                           cudaMemcpyHostToDevice, p->s_copy));
            SCOUT_CUDA(cudaEventRecord(p->ev_copied[buf], p->s_copy));
            SCOUT_CUDA(cudaStreamWaitEvent(p->s_comp, p->ev_copied[buf], 0));
            SignLaunch l;
            l.tiles = p->d_tiles;
            l.tile_begin = t0;
            l.n_tiles = t1 - t0;
            l.tiles_per_replica = NT;
            l.replica_begin = r;
            l.n_replicas = 1;
            l.ptrs = nullptr;
            l.T = p->T;
            l.stage = p->d_stage[buf];
            l.slice_begin = a;
            l.recs = p->d_recs;
            l.error = p->d_error;
            l.variant = p->variant == 3 ? 0 : p->variant;
            l.uniform_dtype = p->uniform_dtype;
            l.grid = p->grid;
            next_work_counter(p, l);
            if ((rc = launch_sign_tiles(l, p->s_comp))) return rc;
            SCOUT_CUDA(cudaEventRecord(p->ev_done[buf], p->s_comp));
            t0 = t1;
            ++slice;
        }
    }
    rc = launch_finalize(p->d_chunks, p->chunks.size(), p->R, p->d_recs, NT, p->tile_bytes / ROW_BYTES,
                         p->max_chunk_tiles, p->d_sigs, p->d_out, p->s_comp);
    if (rc) return rc;
    if ((rc = mark_launched(p, p->s_comp))) return rc;
    return vote_and_report(p, p->s_comp, report, h_outliers, outlier_cap, h_undecided, undecided_cap);
}

int scout_plan_results(const scout_plan_t *p, const scout_sig_t **d_sigs, const uint8_t **d_status,
                       const uint64_t **d_bitmap) {
    if (!p || !p->have_results) return SCOUT_ERR_INVALID;
    if (d_sigs) *d_sigs = p->d_sigs;
    if (d_status) *d_status = p->d_status;
    if (d_bitmap) *d_bitmap = p->d_bitmap;
    return SCOUT_OK;
}

int scout_plan_replica_bad_counts(const scout_plan_t *p, uint64_t *h_counts) {
    if (!p || !h_counts || !p->have_results) return SCOUT_ERR_INVALID;
    for (uint32_t r = 0; r < p->R; ++r) h_counts[r] = p->h_out->out.replica_bad[r];
    return SCOUT_OK;
}

int scout_rollup_tensors(const scout_plan_t *p, const scout_sig_t *d_sigs, uint64_t *d_tensor_sigs,
                         void *stream) {
    if (!p || !d_sigs || !d_tensor_sigs) return SCOUT_ERR_INVALID;
    if (int rc = check_device(p)) return rc;
    return launch_rollup_tensors(p->d_chunks, p->d_tensor_chunk0, p->T, p->R, d_sigs, d_tensor_sigs,
                                 (cudaStream_t)stream);
}

uint64_t scout_shape_tag(uint32_t ndim, const uint64_t *dims) {
    uint64_t a = mix64(SEED_SHAPE ^ (uint64_t)ndim);
    for (uint32_t i = 0; i < ndim; ++i) a = mix64(a ^ dims[i]);
    return a;
}

int scout_plan_set(scout_plan_t *p, const char *key, int64_t value) {
    if (!p || !key) return SCOUT_ERR_INVALID;
    if (int rc = check_device(p)) return rc;
    if (!std::strcmp(key, "device_error")) {
        // 0 clears the flag a timed-out wait left behind; a non-zero value sets it from the
        // host (how the tests produce the failure without making a GPU wait run out)
        const uint32_t v = value ? 1u : 0u;
        if (p->launched) SCOUT_CUDA(cudaEventSynchronize(p->ev_last));
        SCOUT_CUDA(cudaMemcpy(p->d_error, &v, sizeof(v), cudaMemcpyHostToDevice));
        return SCOUT_OK;
    }
    if (!std::strcmp(key, "tile_bytes")) {
        if (value < 2048 || value > 262144 || (value & (value - 1))) return SCOUT_ERR_INVALID;
        if ((uint32_t)value == p->tile_bytes) return SCOUT_OK;
        if (p->variant == 4 && value > 32768) return SCOUT_ERR_INVALID;
        if (p->launched) SCOUT_CUDA(cudaEventSynchronize(p->ev_last));  // the tables may be in use
        p->tile_bytes = (uint32_t)value;
        try {
            build_tiles(p);
        } catch (const std::bad_alloc &) {
            return SCOUT_ERR_NOMEM;
        }
        if (p->d_stage[0]) {  // staging was sized for the old tiles
            for (int i = 0; i < 2; ++i) { plan_free(p, p->d_stage[i]); p->d_stage[i] = nullptr; }
            cudaStreamDestroy(p->s_copy);
            cudaStreamDestroy(p->s_comp);
            p->s_copy = p->s_comp = nullptr;
            for (int i = 0; i < 2; ++i) {
                cudaEventDestroy(p->ev_copied[i]);
                cudaEventDestroy(p->ev_done[i]);
                p->ev_copied[i] = p->ev_done[i] = nullptr;
            }
        }
        return upload_tables(p);
    }
    if (!std::strcmp(key, "work_streams")) {
        if (value < 1 || value > (int64_t)MAX_WORK_STREAMS) return SCOUT_ERR_INVALID;
        if (p->launched) SCOUT_CUDA(cudaEventSynchronize(p->ev_last));   // the counters may be in use
        p->work_streams = (uint32_t)value;
        SCOUT_CUDA(cudaMemset(p->d_work2, 0, WORK_BYTES));
        return SCOUT_OK;
    }
    if (!std::strcmp(key, "dynamic")) {
        p->dynamic = value != 0;
        return SCOUT_OK;
    }
    if (!std::strcmp(key, "fused")) {
        if (value < -1 || value > 2) return SCOUT_ERR_INVALID;
        if (value == 2 && !p->cluster_ok) return SCOUT_ERR_UNSUPPORTED;
        p->fused = (int)value;
        return SCOUT_OK;
    }
    if (!std::strcmp(key, "variant")) {
        if (value < 0 || value > 4) return SCOUT_ERR_INVALID;
        if (value == 4 && p->tile_bytes > 32768) return SCOUT_ERR_INVALID;  // a tile must fit one stage
        p->variant = (int)value;
        return sign_grid_size(p->variant, p->uniform_dtype, p->device, &p->grid);
    }
    if (!std::strcmp(key, "timing")) {
        if (value && p->ev_t0.empty()) {
            try {
                p->ev_t0.assign(TIMING_RING, nullptr);
                p->ev_t1.assign(TIMING_RING, nullptr);
            } catch (const std::bad_alloc &) {
                return SCOUT_ERR_NOMEM;
            }
            for (size_t i = 0; i < TIMING_RING; ++i) {
                SCOUT_CUDA(cudaEventCreate(&p->ev_t0[i]));
                SCOUT_CUDA(cudaEventCreate(&p->ev_t1[i]));
            }
        }
        p->timing = value != 0;
        p->timed_launches = 0;  // (re)starts the count the two getters below refer to
        return SCOUT_OK;
    }
    if (!std::strcmp(key, "grid")) {
        if (value < 1 || value > 65535) return SCOUT_ERR_INVALID;
        p->grid = (int)value;
        return SCOUT_OK;
    }
    return SCOUT_ERR_INVALID;
}

int scout_plan_get(const scout_plan_t *p, const char *key, int64_t *value) {
    if (!p || !key || !value) return SCOUT_ERR_INVALID;
    if (!std::strcmp(key, "tile_bytes")) *value = p->tile_bytes;
    else if (!std::strcmp(key, "variant")) *value = p->variant;
    else if (!std::strcmp(key, "grid")) *value = p->grid;
    else if (!std::strcmp(key, "n_tiles")) *value = (int64_t)p->tiles.size();
    else if (!std::strcmp(key, "debug")) *value = p->debug;
    else if (!std::strcmp(key, "guards_ok")) {
        if (!p->debug) return SCOUT_ERR_INVALID;  // there are no guard bands to look at
        if (int rc = check_device(p)) return rc;
        return guards_intact(p, value);
    }
    else if (!std::strcmp(key, "fused")) *value = p->fused;
    else if (!std::strcmp(key, "work_streams")) *value = p->work_streams;
    else if (!std::strcmp(key, "certify_form")) *value = launch_form(p, true);
    else if (!std::strcmp(key, "sign_form")) *value = launch_form(p, false);
    else if (!std::strcmp(key, "cluster_ok")) *value = p->cluster_ok;
    else if (!std::strcmp(key, "dynamic")) *value = p->dynamic;
    else if (!std::strcmp(key, "sign_kernels")) *value = launch_form(p, false) ? 1 : 2;    // scan, finalise
    else if (!std::strcmp(key, "certify_kernels")) *value = launch_form(p, true) ? 1 : 4;  // + vote, certificate chain
    else if (!std::strcmp(key, "last_sign_ns")) {
        // device time of the most recent scan kernel; the stream must have been synchronised
        if (!p->timing || p->timed_launches == 0) return SCOUT_ERR_INVALID;
        const size_t slot = (size_t)((p->timed_launches - 1) % TIMING_RING);
        float ms = 0.f;
        SCOUT_CUDA(cudaEventElapsedTime(&ms, p->ev_t0[slot], p->ev_t1[slot]));
        *value = (int64_t)((double)ms * 1e6);
    }
    else if (!std::strcmp(key, "timed_sign_launches")) {
        // scan launches the ring still holds (all of them, up to its size) since "timing" was set
        if (!p->timing) return SCOUT_ERR_INVALID;
        *value = (int64_t)std::min<uint64_t>(p->timed_launches, TIMING_RING);
    }
    else if (!std::strcmp(key, "timed_sign_ns")) {
        // their total device time; the stream must have been synchronised
        if (!p->timing) return SCOUT_ERR_INVALID;
        const uint64_t n = std::min<uint64_t>(p->timed_launches, TIMING_RING);
        double total_ms = 0.0;
        for (uint64_t i = 0; i < n; ++i) {
            const size_t slot = (size_t)((p->timed_launches - 1 - i) % TIMING_RING);
            float ms = 0.f;
            SCOUT_CUDA(cudaEventElapsedTime(&ms, p->ev_t0[slot], p->ev_t1[slot]));
            total_ms += ms;
        }
        *value = (int64_t)(total_ms * 1e6);
    }
    else if (!std::strcmp(key, "device_error")) {
        if (int rc = check_device(p)) return rc;
        uint32_t e = 0;
        SCOUT_CUDA(cudaMemcpy(&e, p->d_error, sizeof(e), cudaMemcpyDeviceToHost));
        *value = e;
    }
    else if (!std::strcmp(key, "scratch_bytes")) *value = (int64_t)(p->tiles.size() * p->R * sizeof(TileRec));
    else return SCOUT_ERR_INVALID;
    return SCOUT_OK;
}

int scout_selftest_bounded_wait(uint64_t limit_ns, uint64_t *d_out, void *stream) {
    if (!d_out || limit_ns == 0 || limit_ns > 1000000000ull) return SCOUT_ERR_INVALID;
    return launch_bounded_wait_selftest(limit_ns, d_out, (cudaStream_t)stream);
}

const char *scout_strerror(int code) {
    switch (code) {
        case SCOUT_OK: return "ok";
        case SCOUT_ERR_INVALID: return "invalid argument";
        case SCOUT_ERR_ALIGN: return "tensor address not 16-byte aligned";
        case SCOUT_ERR_UNSUPPORTED: return "unsupported (more than 64 replicas, or a table too large)";
        case SCOUT_ERR_CUDA: return "CUDA runtime error";
        case SCOUT_ERR_NOMEM: return "out of memory";
        case SCOUT_ERR_TRUNCATED: return "result list truncated (counters hold the true totals)";
        default: return "unknown error";
    }
}

int scout_version(void) { return 100; }

const char *scout_last_cuda_error(void) { return g_last_cuda_error.c_str(); }

}  // extern "C"
