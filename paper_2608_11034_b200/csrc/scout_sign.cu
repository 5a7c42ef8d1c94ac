// Comparable evidence (Sec. 5.2) as separate kernels: the bulk fold of replica bytes
// into per-tile partial records (the direct scan and its alternative front ends, the
// read-only probe) and the kernel that finalises them into one record per
// (chunk, replica).  The row routine is in scout_scan.cuh, the combine in
// scout_combine.cuh.
#include "scout_combine.cuh"
#include "scout_scan.cuh"

namespace scout {
namespace {

// Work distribution of the direct scan and of the read probe.  Every warp starts with item
// `warp`; the items after the first n_warps are handed out as warps become free (tiles differ
// in size and dtype, and SMs differ in how the memory system serves them, so a fixed
// round-robin ends with its slowest warp).  They are dealt from `streams` counters, 128 bytes
// apart: counter j hands out the items n_warps + j, n_warps + j + streams, ... in order, and a
// warp draws from counter (warp mod streams) until that one has run out, then from the next.
// One counter is one address, served by one L2 slice at about one atomic per 3 ns, which is
// about the rate at which a B200 finishes 32 KiB tiles; several counters keep the hand-out
// off that limit while the tiles in flight stay one contiguous window of the input (claiming
// several consecutive tiles per atomic was tried instead and cost 2-5 %).  The request for the
// next item is made before the current tile is scanned and its answer is read after it.  The
// counters of this launch are those of work_parity; the others are zeroed here for the launch
// that follows.
constexpr uint32_t WORK_STRIDE = 16;   // 64-bit words between two counters (128 bytes)
struct WorkQueue {
    unsigned long long *ctr;   // this launch's counters, or null: fixed round-robin
    uint64_t n_warps, n_items, n_rest;
    uint32_t streams, stream, empty_seen;

    __device__ __forceinline__ void begin(const SignArgs &a, uint64_t warp, uint64_t warps, uint64_t items,
                                          uint32_t lane) {
        n_warps = warps;
        n_items = items;
        n_rest = items > warps ? items - warps : 0;
        streams = a.work_streams;
        ctr = (a.work && n_rest) ? a.work + (uint64_t)a.work_parity * streams * WORK_STRIDE : nullptr;
        if (a.work && warp == 0 && lane < streams)
            a.work[((uint64_t)(a.work_parity ^ 1u) * streams + lane) * WORK_STRIDE] = 0ull;
        stream = (uint32_t)(warp % streams);
        empty_seen = 0;
    }
    // lane 0: ask for the next item (the answer is used by next_item)
    __device__ __forceinline__ unsigned long long request(uint32_t lane) const {
        unsigned long long k = 0;
        if (ctr && lane == 0) k = atomicAdd(ctr + stream * WORK_STRIDE, 1ull);
        return k;
    }
    // the item that follows `item`, given the answer to the request made before it was scanned
    __device__ __forceinline__ uint64_t next_item(uint64_t item, unsigned long long answer, uint32_t lane) {
        if (!ctr) return item + n_warps;
        uint64_t i = __shfl_sync(0xFFFFFFFFu, answer, 0) * streams + stream;
        while (i >= n_rest) {   // this counter has run out: the next one (only at the very end of a launch)
            if (++empty_seen >= streams) return n_items;
            stream = stream + 1 == streams ? 0 : stream + 1;
            unsigned long long k = 0;
            if (lane == 0) k = atomicAdd(ctr + stream * WORK_STRIDE, 1ull);
            i = __shfl_sync(0xFFFFFFFFu, k, 0) * streams + stream;
        }
        return n_warps + i;
    }
};

// Persistent grid; every warp takes whole tiles, replica-major, round-robin.
// DTSEL >= 0: every tile of the launch has that dtype (the element path is fixed at
// compile time, so the register allocation is that path's, not the union of all
// seven); DTSEL < 0: the dtype is read from the tile table.
template <int PREFETCH, int DTSEL>
__global__ void __launch_bounds__(SIGN_THREADS, PREFETCH ? SCOUT_MINBLOCKS_PF : SCOUT_MINBLOCKS) sign_tiles_direct(const SignArgs a) {
    pdl_launch_dependents();
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (SIGN_THREADS / 32) + (threadIdx.x >> 5);
    WorkQueue q;
    q.begin(a, warp, (uint64_t)gridDim.x * (SIGN_THREADS / 32), a.n_tiles * a.n_replicas, lane);
    uint64_t item = warp;
    while (item < q.n_items) {
        const unsigned long long answer = q.request(lane);
        const uint32_t rr = (uint32_t)(item / a.n_tiles);
        const uint64_t t = a.tile_begin + (item - (uint64_t)rr * a.n_tiles);
        const uint32_t r = a.replica_begin + rr;
        const TileDesc td = a.tiles[t];
        const uint8_t *tile = tile_address(a, td, r);
        TileRec rec;
        if constexpr (DTSEL >= 0) {
            if (PREFETCH) scan_tile_prefetch<DTSEL, true>(tile, td.nbytes, lane, rec);
            else          scan_tile<DTSEL, true>(tile, td.nbytes, lane, rec);
        } else {
            if (PREFETCH) scan_dispatch_prefetch(td.dtype, tile, td.nbytes, lane, rec);
            else          scan_dispatch(td.dtype, tile, td.nbytes, lane, rec);
        }
        if (lane == 0) store_record(&a.recs[(uint64_t)r * a.tiles_per_replica + t], rec);
        item = q.next_item(item, answer, lane);
    }
}

using SignKernel = void (*)(const SignArgs);
// The direct-scan kernel for a front end (0 direct, 1 register prefetch) and a launch
// whose tiles all have dtype `uniform` (specialised for fp32, bf16 and fp16), or mixed (-1).
SignKernel direct_kernel(int prefetch, int uniform) {
    if (prefetch) {
        if (uniform == SCOUT_DT_F32) return sign_tiles_direct<1, SCOUT_DT_F32>;
        if (uniform == SCOUT_DT_BF16) return sign_tiles_direct<1, SCOUT_DT_BF16>;
        return sign_tiles_direct<1, -1>;
    }
    if (uniform == SCOUT_DT_F32) return sign_tiles_direct<0, SCOUT_DT_F32>;
    if (uniform == SCOUT_DT_BF16) return sign_tiles_direct<0, SCOUT_DT_BF16>;
    if (uniform == SCOUT_DT_F16) return sign_tiles_direct<0, SCOUT_DT_F16>;
    return sign_tiles_direct<0, -1>;
}

// ---- front end 2: bulk-async ring ----------------------------------------------
// Every warp owns RING_STAGES pieces of RING_PIECE bytes in shared memory and one
// mbarrier per piece.  Lane 0 asks the copy engine for whole rows
// (cp.async.bulk global -> shared, completion counted in bytes on the piece's
// mbarrier); the warp waits for a piece, folds its rows from shared memory, and
// immediately asks for the piece RING_STAGES ahead, across tile boundaries, so
// the bytes in flight do not depend on how long the arithmetic takes.  There is
// no block-wide synchronisation: warps are independent.  Only whole rows go
// through the ring; a chunk's ragged last row is read with plain loads.
#ifndef SCOUT_RING_PIECE
#define SCOUT_RING_PIECE 4096
#endif
#ifndef SCOUT_RING_STAGES
#define SCOUT_RING_STAGES 3
#endif
#ifndef SCOUT_RING_BLOCKS
#define SCOUT_RING_BLOCKS 2
#endif
constexpr int RING_PIECE = SCOUT_RING_PIECE;  // bytes per piece: whole rows
constexpr int RING_STAGES = SCOUT_RING_STAGES;
constexpr int RING_ROWS = RING_PIECE / (int)ROW_BYTES;
constexpr int RING_WARPS = SIGN_THREADS / 32;
constexpr int RING_SMEM = RING_WARPS * RING_STAGES * RING_PIECE + RING_WARPS * RING_STAGES * 8;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // a wait on a copy gives up after 2 s

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Wait for an mbarrier phase, but never longer than limit_ns: the clock is read every
// 256 polls; false means the wait gave up (the caller reports it and returns).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  unsigned long long limit_ns = WAIT_LIMIT_NS) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t polls = 1;; ++polls) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((polls & 255u) == 0u && global_ns() - t0 > limit_ns) return false;
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ uint4 lds16(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr));
    return v;
}

// What the ring needs to know about one work item.
struct RingTile {
    const uint8_t *base;
    TileRec *rec;
    uint32_t nbytes, dtype;
};

struct RingCtx {
    const SignArgs &a;
    uint64_t n_items, n_warps;
    uint32_t lane, data0, bar0;
    uint32_t issued, consumed;
    // producer side: the tile whose pieces are being requested, and the one after it
    RingTile p_cur, p_next;
    uint64_t p_item;       // item id of p_next
    uint32_t p_off, p_full;
    bool p_valid;
    bool gave_up;

    __device__ __forceinline__ RingTile describe(uint64_t item) const {
        RingTile t;
        t.base = nullptr; t.rec = nullptr; t.nbytes = 0; t.dtype = 0;
        if (item < n_items) {
            const uint32_t rr = (uint32_t)(item / a.n_tiles);
            const uint64_t ti = a.tile_begin + (item - (uint64_t)rr * a.n_tiles);
            const uint32_t r = a.replica_begin + rr;
            const TileDesc td = a.tiles[ti];
            t.base = tile_address(a, td, r);
            t.rec = &a.recs[(uint64_t)r * a.tiles_per_replica + ti];
            t.nbytes = td.nbytes;
            t.dtype = td.dtype;
        }
        return t;
    }
    // make p_cur the next tile that has whole rows; p_next is read one tile early so
    // that its descriptor has arrived by the time the producer needs it
    __device__ __forceinline__ void producer_advance() {
        for (;;) {
            p_cur = p_next;
            p_valid = p_item < n_items;
            if (!p_valid) return;
            p_item += n_warps;
            p_next = describe(p_item);
            p_off = 0;
            p_full = (p_cur.nbytes / ROW_BYTES) * ROW_BYTES;
            if (p_full) return;
        }
    }
    __device__ __forceinline__ void request() {
        const uint32_t stage = issued % RING_STAGES;
        const uint32_t bytes = min((uint32_t)RING_PIECE, p_full - p_off);
        if (lane == 0) {
            mbar_expect_tx(bar0 + 8 * stage, bytes);
            bulk_g2s(data0 + stage * RING_PIECE, p_cur.base + p_off, bytes, bar0 + 8 * stage);
        }
        ++issued;
        p_off += bytes;
        if (p_off >= p_full) producer_advance();
    }
    // wait for the oldest outstanding piece; false if the bounded wait gave up
    __device__ __forceinline__ bool acquire(uint32_t &saddr) {
        const uint32_t stage = consumed % RING_STAGES;
        const uint32_t parity = (consumed / RING_STAGES) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * stage, parity)) { gave_up = true; return false; }
        saddr = data0 + stage * RING_PIECE + 16u * lane;
        return true;
    }
    __device__ __forceinline__ void release() {
        __syncwarp();  // every lane has read the piece before it is requested again
        ++consumed;
        if (p_valid) request();
    }
};

template <int DT>
__device__ __forceinline__ void ring_tile(RingCtx &c, const RingTile &t, TileRec &rec) {
    TileScan<DT> st;
    st.begin(c.lane);
    uint32_t rows = t.nbytes / ROW_BYTES;
#pragma unroll 1
    for (; rows >= RING_ROWS; rows -= RING_ROWS) {
        uint32_t saddr;
        if (!c.acquire(saddr)) return;
        uint4 v[RING_ROWS];
#pragma unroll
        for (int r = 0; r < RING_ROWS; ++r) v[r] = lds16(saddr + r * ROW_BYTES);
#pragma unroll
        for (int r = 0; r < RING_ROWS; ++r) st.row(v[r]);
        c.release();
    }
    if (rows) {
        uint32_t saddr;
        if (!c.acquire(saddr)) return;
        for (uint32_t r = 0; r < rows; ++r) st.row(lds16(saddr + r * ROW_BYTES));
        c.release();
    }
    st.finish(t.base, t.nbytes, c.lane, rec);
}

__global__ void __launch_bounds__(SIGN_THREADS, SCOUT_RING_BLOCKS) sign_tiles_ring(const SignArgs a) {
    extern __shared__ __align__(128) uint8_t ring_smem[];
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wib = threadIdx.x >> 5;
    const uint64_t warp = (uint64_t)blockIdx.x * RING_WARPS + wib;
    RingCtx c{a};
    c.n_items = a.n_tiles * a.n_replicas;
    c.n_warps = (uint64_t)gridDim.x * RING_WARPS;
    c.lane = lane;
    c.data0 = smem_u32(ring_smem) + wib * (RING_STAGES * RING_PIECE);
    c.bar0 = smem_u32(ring_smem) + RING_WARPS * RING_STAGES * RING_PIECE + wib * (RING_STAGES * 8);
    c.issued = c.consumed = 0;
    c.gave_up = false;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < RING_STAGES; ++s) mbar_init(c.bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    c.p_item = warp;
    c.p_next = c.describe(warp);
    c.producer_advance();
    for (int s = 0; s < RING_STAGES && c.p_valid; ++s) c.request();

    RingTile next = c.describe(warp);
#pragma unroll 1
    for (uint64_t item = warp; item < c.n_items && !c.gave_up; item += c.n_warps) {
        const RingTile t = next;
        next = c.describe(item + c.n_warps);  // in flight while this tile is folded
        TileRec rec;
        switch (t.dtype) {
            case SCOUT_DT_F32:  ring_tile<SCOUT_DT_F32>(c, t, rec); break;
            case SCOUT_DT_BF16: ring_tile<SCOUT_DT_BF16>(c, t, rec); break;
            case SCOUT_DT_I64:  ring_tile<SCOUT_DT_I64>(c, t, rec); break;
            case SCOUT_DT_F16:  ring_tile<SCOUT_DT_F16>(c, t, rec); break;
            case SCOUT_DT_F64:  ring_tile<SCOUT_DT_F64>(c, t, rec); break;
            case SCOUT_DT_I32:  ring_tile<SCOUT_DT_I32>(c, t, rec); break;
            default:            ring_tile<SCOUT_DT_U8>(c, t, rec); break;
        }
        if (!c.gave_up && lane == 0) store_record(t.rec, rec);
    }
    if (c.gave_up) {
        // A copy never completed.  Report it, give the copies still in flight one more
        // bounded chance to land (shared memory must not be released under them), return.
        if (lane == 0 && a.error) atomicExch(a.error, 1u);
        for (uint32_t n = c.consumed; n < c.issued; ++n) {
            const uint32_t stage = n % RING_STAGES, parity = (n / RING_STAGES) & 1u;
            mbar_wait_bounded(c.bar0 + 8 * stage, parity);
        }
    }
}

// ---- front end 4: block-wide bulk-async ring --------------------------------------
// One CTA = 8 consumer warps + 1 producer warp.  The producer's lane 0 walks the
// CTA's tiles and fetches each WHOLE tile (<= 32 KiB of whole rows) with one
// cp.async.bulk into one of CTA_STAGES shared-memory stages, after the stage's
// "empty" mbarrier says all eight consumers are done with its previous tile.  The
// consumers wait on the stage's "full" mbarrier; warp w folds rows [8w, 8w+8) of
// the tile; every lane weights its hash share by the rows that follow its warp's
// block and leaves (h, sum, sumsq) in shared memory; the last warp to finish a tile
// (an atomic ticket in shared memory, nobody waits) adds the eight warps' shares
// lane by lane in warp order, runs the one butterfly of the tile and writes the
// record.  Large copies keep the copy engine efficient and the bytes
// in flight (CTA_STAGES x 32 KiB per CTA, 2 CTAs per SM) do not depend on the
// arithmetic.  Every wait is bounded; a wait that gives up sets the error flag.
constexpr int CTA_STAGE_BYTES = 32768;
constexpr int CTA_STAGES = 3;
constexpr int CTA_CONSUMERS = 8;
constexpr int CTA_THREADS = (CTA_CONSUMERS + 1) * 32;
constexpr int CTA_ROWS_PER_WARP = CTA_STAGE_BYTES / (int)ROW_BYTES / CTA_CONSUMERS;  // 8

struct CtaStageInfo {      // written by the producer before the copy, read after the full barrier
    const uint8_t *tile;
    TileRec *rec;
    uint32_t nbytes, dtype;
};
// One consumer LANE's part of a tile (no per-warp reduction).  The shares are kept
// in the stage itself: once warp w has folded its rows, the first kilobyte of its
// own 4 KiB block (which no other warp reads) holds its 32 lanes' shares.
struct CtaShare {
    uint64_t h;
    double s, q;
    uint64_t pad;
};
static_assert(sizeof(CtaShare) * 32 <= CTA_ROWS_PER_WARP * ROW_BYTES, "shares fit the warp's block");
struct CtaShared {
    unsigned long long full[CTA_STAGES], empty[CTA_STAGES];
    CtaStageInfo info[CTA_STAGES];
    uint64_t weight[CTA_CONSUMERS];  // P^(rows after warp w's block) in a full tile
    uint32_t suspect[CTA_STAGES];
    uint32_t ticket[CTA_STAGES];
    uint32_t abort_flag;
};
constexpr int CTA_SMEM = CTA_STAGES * CTA_STAGE_BYTES + (int)sizeof(CtaShared);

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
template <int DT>
__device__ __forceinline__ void cta_consume(const CtaStageInfo &info, uint32_t data, uint32_t warp,
                                            uint32_t lane, uint64_t weight, CtaShare &out, bool &suspect) {
    TileScan<DT> st;
    st.begin(lane);
    const uint32_t full_rows = info.nbytes / ROW_BYTES;
    const uint32_t total_rows = (info.nbytes + ROW_BYTES - 1) / ROW_BYTES;
    const uint32_t row0 = warp * CTA_ROWS_PER_WARP;
    const uint32_t row1 = min(row0 + CTA_ROWS_PER_WARP, total_rows);
    const uint32_t saddr = data + row0 * ROW_BYTES + 16u * lane;
    if (row0 + CTA_ROWS_PER_WARP <= full_rows) {
        uint4 v[CTA_ROWS_PER_WARP];
#pragma unroll
        for (int r = 0; r < CTA_ROWS_PER_WARP; ++r) v[r] = lds16(saddr + r * ROW_BYTES);
#pragma unroll
        for (int r = 0; r < CTA_ROWS_PER_WARP; ++r) st.row(v[r]);
    } else {
        for (uint32_t r = row0; r < row1; ++r) {
            if (r < full_rows) st.row(lds16(data + r * ROW_BYTES + 16u * lane));
            else st.row(ld_masked16(info.tile, r * ROW_BYTES + 16u * lane, info.nbytes));  // ragged row
        }
    }
    // the warp's rows are followed by (total_rows - row1) rows of the tile
    uint64_t h = st.h;
    if (row1 > row0) h *= total_rows == (uint32_t)(CTA_STAGE_BYTES / ROW_BYTES) ? weight : pow_p(total_rows - row1);
    out.h = h;
    out.q = st.a.q0 + st.a.q1;
    if constexpr (DT == SCOUT_DT_BF16 && BF16_BITROUTE > 0) out.s = fma(st.a.s1, 0x1p896, st.a.s0);
    else out.s = st.a.s0 + st.a.s1;
    suspect = may_hold_nonfinite<DT>(st.a);
}

template <int DT>
__device__ __forceinline__ void cta_rescan(const CtaStageInfo &info, uint32_t lane, TileRec &rec) {
    if constexpr (DT == SCOUT_DT_F32 || DT == SCOUT_DT_BF16 || DT == SCOUT_DT_F16 || DT == SCOUT_DT_F64)
        rescan_classifying<DT>(info.tile, info.nbytes, lane, rec.sum, rec.sumsq, rec.nan_count, rec.inf_count);
}

__global__ void __launch_bounds__(CTA_THREADS, 2) sign_tiles_cta_ring(const SignArgs a) {
    extern __shared__ __align__(128) uint8_t cta_smem[];
    CtaShared &sh = *reinterpret_cast<CtaShared *>(cta_smem + CTA_STAGES * CTA_STAGE_BYTES);
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint64_t n_items = a.n_tiles * a.n_replicas;
    const uint32_t data0 = smem_u32(cta_smem);
    pdl_launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < CTA_STAGES; ++s) {
            mbar_init(smem_u32(&sh.full[s]), 1);
            mbar_init(smem_u32(&sh.empty[s]), CTA_CONSUMERS);
            sh.ticket[s] = 0;
            sh.suspect[s] = 0;
        }
        for (int w = 0; w < CTA_CONSUMERS; ++w)
            sh.weight[w] = pow_p((uint64_t)CTA_ROWS_PER_WARP * (CTA_CONSUMERS - 1 - w));
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == CTA_CONSUMERS) {
        // ---- producer ----
        if (lane == 0) {
            uint32_t n = 0;
            for (uint64_t item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
                const uint32_t stage = n % CTA_STAGES;
                // wait until the consumers have released this stage's previous tile
                // (the first CTA_STAGES uses find the barrier's "previous" phase complete)
                if (!mbar_wait_bounded(smem_u32(&sh.empty[stage]), ((n / CTA_STAGES) & 1u) ^ 1u) ||
                    *(volatile uint32_t *)&sh.abort_flag) {
                    atomicExch(&sh.abort_flag, 1u);
                    if (a.error) atomicExch(a.error, 1u);
                    break;
                }
                const uint32_t rr = (uint32_t)(item / a.n_tiles);
                const uint64_t t = a.tile_begin + (item - (uint64_t)rr * a.n_tiles);
                const uint32_t r = a.replica_begin + rr;
                const TileDesc td = a.tiles[t];
                CtaStageInfo info;
                info.tile = tile_address(a, td, r);
                info.rec = &a.recs[(uint64_t)r * a.tiles_per_replica + t];
                info.nbytes = td.nbytes;
                info.dtype = td.dtype;
                sh.info[stage] = info;
                const uint32_t bytes = (td.nbytes / ROW_BYTES) * ROW_BYTES;
                const uint32_t bar = smem_u32(&sh.full[stage]);
                if (bytes) {
                    mbar_expect_tx(bar, bytes);
                    bulk_g2s(data0 + stage * CTA_STAGE_BYTES, info.tile, bytes, bar);
                } else {
                    mbar_arrive(bar);  // a tile shorter than one row: nothing to copy
                }
            }
        }
        return;
    }

    // ---- consumers ----
    uint32_t n = 0;
    for (uint64_t item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
        const uint32_t stage = n % CTA_STAGES;
        if (!mbar_wait_bounded(smem_u32(&sh.full[stage]), (n / CTA_STAGES) & 1u) ||
            *(volatile uint32_t *)&sh.abort_flag) {
            if (lane == 0) {
                atomicExch(&sh.abort_flag, 1u);
                if (a.error) atomicExch(a.error, 1u);
            }
            break;  // copies already issued are awaited below, before shared memory is released
        }
        const CtaStageInfo info = sh.info[stage];
        const uint32_t data = data0 + stage * CTA_STAGE_BYTES;
        CtaShare mine;
        bool sus = false;
        const uint64_t wgt = sh.weight[warp];
        switch (info.dtype) {
            case SCOUT_DT_F32:  cta_consume<SCOUT_DT_F32>(info, data, warp, lane, wgt, mine, sus); break;
            case SCOUT_DT_BF16: cta_consume<SCOUT_DT_BF16>(info, data, warp, lane, wgt, mine, sus); break;
            case SCOUT_DT_I64:  cta_consume<SCOUT_DT_I64>(info, data, warp, lane, wgt, mine, sus); break;
            case SCOUT_DT_F16:  cta_consume<SCOUT_DT_F16>(info, data, warp, lane, wgt, mine, sus); break;
            case SCOUT_DT_F64:  cta_consume<SCOUT_DT_F64>(info, data, warp, lane, wgt, mine, sus); break;
            case SCOUT_DT_I32:  cta_consume<SCOUT_DT_I32>(info, data, warp, lane, wgt, mine, sus); break;
            default:            cta_consume<SCOUT_DT_U8>(info, data, warp, lane, wgt, mine, sus); break;
        }
        CtaShare *shares = reinterpret_cast<CtaShare *>(cta_smem + stage * CTA_STAGE_BYTES);
        __syncwarp();  // every lane of this warp has read its rows: the block may be reused
        shares[warp * (CTA_ROWS_PER_WARP * ROW_BYTES / sizeof(CtaShare)) + lane] = mine;
        if (__any_sync(0xFFFFFFFFu, sus) && lane == 0) atomicOr(&sh.suspect[stage], 1u);
        uint32_t last = 0;
        __syncwarp();
        if (lane == 0) {
            __threadfence_block();
            last = atomicAdd(&sh.ticket[stage], 1u) == CTA_CONSUMERS - 1;
        }
        last = __shfl_sync(0xFFFFFFFFu, last, 0);
        if (last) {  // every share of this tile is in shared memory: add them in warp order
            __threadfence_block();
            uint64_t h = 0;
            double sum = 0.0, sumsq = 0.0;
            for (int w = 0; w < CTA_CONSUMERS; ++w) {
                const volatile CtaShare &x = shares[w * (CTA_ROWS_PER_WARP * ROW_BYTES / sizeof(CtaShare)) + lane];
                h += x.h;
                sum += x.s;
                sumsq += x.q;
            }
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                h += __shfl_xor_sync(0xFFFFFFFFu, h, d);
                sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
                sumsq += __shfl_xor_sync(0xFFFFFFFFu, sumsq, d);
            }
            TileRec rec;
            rec.h = h;
            rec.sum = sum;
            rec.sumsq = sumsq;
            rec.nan_count = rec.inf_count = 0;
            const uint32_t suspect = *(volatile uint32_t *)&sh.suspect[stage];
            if (suspect) {
                switch (info.dtype) {
                    case SCOUT_DT_F32:  cta_rescan<SCOUT_DT_F32>(info, lane, rec); break;
                    case SCOUT_DT_BF16: cta_rescan<SCOUT_DT_BF16>(info, lane, rec); break;
                    case SCOUT_DT_F16:  cta_rescan<SCOUT_DT_F16>(info, lane, rec); break;
                    case SCOUT_DT_F64:  cta_rescan<SCOUT_DT_F64>(info, lane, rec); break;
                    default: break;
                }
            }
            if (lane == 0) {
                store_record(info.rec, rec);
                sh.ticket[stage] = 0;
                sh.suspect[stage] = 0;
            }
        }
        __syncwarp();
        if (lane == 0) {
            // the shares were written with ordinary stores; order them before the next bulk copy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(smem_u32(&sh.empty[stage]));  // this warp is done with the stage
        }
    }
    if (*(volatile uint32_t *)&sh.abort_flag) {
        // give copies that may still be in flight a bounded chance to land before exit
        for (int s = 0; s < CTA_STAGES; ++s)
            for (uint32_t par = 0; par < 2; ++par) mbar_wait_bounded(smem_u32(&sh.full[s]), par);
    }
}

// Self-test of the bounded wait: an mbarrier that nothing ever arrives on.  The wait
// must give up after limit_ns and the kernel must return normally; out[0] = 1 if it
// gave up, out[1] = nanoseconds waited.
__global__ void bounded_wait_selftest(unsigned long long limit_ns, unsigned long long *out) {
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const unsigned long long t0 = global_ns();
    const bool arrived = mbar_wait_bounded(smem_u32(&bar), 0, limit_ns);
    const unsigned long long dt = global_ns() - t0;
    if (threadIdx.x == 0) {
        out[0] = arrived ? 0ull : 1ull;
        out[1] = dt;
    }
}

// Read-only probe: the same tiles and the same loads as the direct scan, with an
// XOR as the only arithmetic.  It measures what the memory system delivers to
// this access pattern (the ceiling the scan is compared with).
__global__ void __launch_bounds__(SIGN_THREADS) read_probe(const SignArgs a) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (SIGN_THREADS / 32) + (threadIdx.x >> 5);
    WorkQueue q;   // the same work distribution as the scan
    q.begin(a, warp, (uint64_t)gridDim.x * (SIGN_THREADS / 32), a.n_tiles * a.n_replicas, lane);
    uint64_t item = warp;
    while (item < q.n_items) {
        const unsigned long long answer = q.request(lane);
        const uint32_t rr = (uint32_t)(item / a.n_tiles);
        const uint64_t t = a.tile_begin + (item - (uint64_t)rr * a.n_tiles);
        const uint32_t r = a.replica_begin + rr;
        const TileDesc td = a.tiles[t];
        const uint8_t *p = tile_address(a, td, r) + 16u * lane;
        const uint32_t full = td.nbytes / ROW_BYTES;
        uint4 x = make_uint4(0u, 0u, 0u, 0u);
        uint32_t row = 0;
        for (; row + 8 <= full; row += 8) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = ld_stream16(p + (size_t)(row + u) * ROW_BYTES);
#pragma unroll
            for (int u = 0; u < 8; ++u) { x.x ^= v[u].x; x.y ^= v[u].y; x.z ^= v[u].z; x.w ^= v[u].w; }
        }
        for (; row < full; ++row) {
            uint4 v = ld_stream16(p + (size_t)row * ROW_BYTES);
            x.x ^= v.x; x.y ^= v.y; x.z ^= v.z; x.w ^= v.w;
        }
        uint32_t y = x.x ^ x.y ^ x.z ^ x.w;
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) y ^= __shfl_xor_sync(0xFFFFFFFFu, y, d);
        if (lane == 0) a.recs[(uint64_t)r * a.tiles_per_replica + t].h = y;
        item = q.next_item(item, answer, lane);
    }
}

__global__ void __launch_bounds__(FIN_THREADS) finalize_chunks(const ChunkDesc *chunks, uint64_t C,
                                                               uint32_t R, const TileRec *recs,
                                                               uint64_t tiles_per_replica,
                                                               uint32_t tile_rows, uint64_t p_stride,
                                                               scout_sig_t *sigs, CertifyOut *zero_out,
                                                               uint32_t rep_batch) {
    pdl_launch_dependents();
    pdl_wait();
    if (zero_out && blockIdx.x == 0 && threadIdx.x < sizeof(CertifyOut) / sizeof(uint64_t))
        reinterpret_cast<uint64_t *>(zero_out)[threadIdx.x] = 0ull;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (FIN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (FIN_THREADS / 32);
    // One item = one chunk and up to rep_batch replicas of it (COMBINE_BATCH when no chunk of the
    // plan has more than 32 tiles, else 1): the chunk's geometry (its descriptor, the lanes'
    // weights) is worked out once for them and their record loads are in flight together.  A
    // warp's items are a chain of dependent memory round trips, so for chunks of few tiles fewer
    // and wider items shorten the kernel (24,320 chunks x 16 replicas: 231 -> 109 us); chunks of
    // many tiles keep one item per replica (717 chunks of 512 tiles x 3: 13 us, 21 us if grouped).
    const uint32_t groups = (R + rep_batch - 1) / rep_batch;
    for (uint64_t item = warp; item < C * groups; item += n_warps) {
        const uint64_t c = item / groups;
        const uint32_t r0 = (uint32_t)(item - c * groups) * rep_batch;
        const uint32_t n_rep = min(rep_batch, R - r0);
        const ChunkDesc cd = chunks[c];
        const uint64_t weight = combine_weight(cd.ntiles, cd.nbytes, tile_rows, lane);
        const TileRec *tr = recs + (uint64_t)r0 * tiles_per_replica + cd.tile0;
        if (rep_batch > 1) {   // every chunk of the plan has at most 32 tiles
            scout_sig_t o[COMBINE_BATCH];
            combine_small(tr, tiles_per_replica, n_rep, cd.ntiles, cd.nbytes, cd.k, cd.dtype, cd.meta, weight, lane, o);
#pragma unroll
            for (int j = 0; j < COMBINE_BATCH; ++j)
                if ((uint32_t)j < n_rep && lane == 0) sigs[c * R + r0 + j] = o[j];
        } else {
            for (uint32_t j = 0; j < n_rep; ++j) {
                const scout_sig_t o = combine_tiles(tr + (uint64_t)j * tiles_per_replica, cd.ntiles, cd.nbytes, cd.k,
                                                    cd.dtype, cd.meta, p_stride, weight, lane);
                if (lane == 0) sigs[c * R + r0 + j] = o;
            }
        }
    }
}


}  // namespace

int sign_grid_size(int variant, int uniform_dtype, int device, int *grid) {
    int sms = 0, per_sm = 0;
    SCOUT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    if (variant == 4) {
        SCOUT_CUDA(cudaFuncSetAttribute(sign_tiles_cta_ring, cudaFuncAttributeMaxDynamicSharedMemorySize, CTA_SMEM));
        SCOUT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sign_tiles_cta_ring, CTA_THREADS, CTA_SMEM));
    } else if (variant == 2) {
        SCOUT_CUDA(cudaFuncSetAttribute(sign_tiles_ring, cudaFuncAttributeMaxDynamicSharedMemorySize, RING_SMEM));
        SCOUT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sign_tiles_ring, SIGN_THREADS, RING_SMEM));
    } else {
        SCOUT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, direct_kernel(variant == 1, uniform_dtype),
                                                                 SIGN_THREADS, 0));
    }
    if (per_sm < 1) per_sm = 1;
    *grid = sms * per_sm;
    return SCOUT_OK;
}

int launch_sign_tiles(const SignLaunch &l, cudaStream_t stream) {
    if (l.n_tiles == 0 || l.n_replicas == 0) return SCOUT_OK;
    SignArgs a;
    a.tiles = l.tiles;
    a.tile_begin = l.tile_begin;
    a.n_tiles = l.n_tiles;
    a.tiles_per_replica = l.tiles_per_replica;
    a.replica_begin = l.replica_begin;
    a.n_replicas = l.n_replicas;
    a.ptrs = l.ptrs;
    a.T = l.T;
    a.stage = l.stage;
    a.slice_begin = l.slice_begin;
    a.recs = l.recs;
    a.error = l.error;
    a.work = l.work;
    a.work_parity = l.work_parity;
    a.work_streams = l.work_streams ? l.work_streams : 1u;
    const uint64_t items = l.n_tiles * l.n_replicas;
    const uint64_t want = (items + SIGN_THREADS / 32 - 1) / (SIGN_THREADS / 32);
    int grid = l.grid;
    if ((uint64_t)grid > want) grid = (int)want;
    if (l.variant == 4) {  // one CTA per tile at a time
        int g = l.grid;
        if ((uint64_t)g > items) g = (int)items;
        sign_tiles_cta_ring<<<g, CTA_THREADS, CTA_SMEM, stream>>>(a);
        SCOUT_CUDA(cudaGetLastError());
        return SCOUT_OK;
    }
    switch (l.variant) {
        case 3: read_probe<<<grid, SIGN_THREADS, 0, stream>>>(a); break;
        case 2: sign_tiles_ring<<<grid, SIGN_THREADS, RING_SMEM, stream>>>(a); break;
        default: direct_kernel(l.variant == 1, l.uniform_dtype)<<<grid, SIGN_THREADS, 0, stream>>>(a); break;
    }
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}

int launch_bounded_wait_selftest(uint64_t limit_ns, uint64_t *d_out, cudaStream_t stream) {
    bounded_wait_selftest<<<1, 32, 0, stream>>>(limit_ns, (unsigned long long *)d_out);
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}

int launch_finalize(const ChunkDesc *chunks, uint64_t C, uint32_t R, const TileRec *recs,
                    uint64_t tiles_per_replica, uint32_t tile_rows, uint32_t max_chunk_tiles,
                    scout_sig_t *d_sigs, CertifyOut *zero_out, cudaStream_t stream) {
    if (C == 0) return SCOUT_OK;
    const uint32_t rep_batch = max_chunk_tiles <= 32u ? (uint32_t)COMBINE_BATCH : 1u;
    const uint64_t items = C * ((R + rep_batch - 1) / rep_batch);
    uint64_t blocks = (items + FIN_THREADS / 32 - 1) / (FIN_THREADS / 32);
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    static_assert(sizeof(CertifyOut) / sizeof(uint64_t) <= FIN_THREADS, "one thread per word clears it");
    SCOUT_CUDA(launch_dependent(finalize_chunks, dim3((unsigned)blocks), dim3(FIN_THREADS), stream, chunks, C,
                                R, recs, tiles_per_replica, tile_rows, pow_p(32ull * tile_rows), d_sigs,
                                zero_out, rep_batch));
    return SCOUT_OK;
}

}  // namespace scout
