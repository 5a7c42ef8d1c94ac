// Finalisation of comparable evidence (Sec. 5.2): the per-tile partial records of one
// (chunk, replica) combined into its 32-byte signature record.  Shared by the finalise
// kernel, the one-launch kernels and the no-allocation entry point, so that every path
// produces bitwise the same record.
#pragma once

#include "scout_internal.h"

namespace scout {
namespace {

// ---- finalise: tile partials -> one record per (chunk, replica) --------------
// Segment combine: for a split after some rows, H_raw = H_raw(left) * P^(rows
// right) + H_raw(right).  A lane walks tiles lane, lane+32, ... with the
// multiplier P^(32 * tile_rows), then weights its value by the rows that follow
// its last tile; the chunk's last tile (the only one that can be short) is added
// with weight one; the lane values add up to H_raw.  The fp64 partials are added
// per lane in ascending tile order and then through a fixed butterfly.
constexpr int FIN_THREADS = 128;

// One warp turns the tile records of one (chunk, replica) into its signature record
// (valid in lane 0).  tr: the chunk's nt records in order; every tile but the last
// has tile_rows rows; p_stride = P^(32 * tile_rows).
// A tile record as another SM wrote it: read through L2.  (L1 is not coherent, and a
// 128-byte line holds four records, so a line fetched while a neighbouring chunk was being
// finalised may hold records that had not been written yet.)
__device__ __forceinline__ TileRec load_record(const TileRec *p) {
    const uint4 lo = __ldcg(reinterpret_cast<const uint4 *>(p));
    const uint4 hi = __ldcg(reinterpret_cast<const uint4 *>(p) + 1);
    TileRec r;
    r.h = ((uint64_t)lo.y << 32) | lo.x;
    r.sum = __hiloint2double((int)lo.w, (int)lo.z);
    r.sumsq = __hiloint2double((int)hi.y, (int)hi.x);
    r.nan_count = hi.z;
    r.inf_count = hi.w;
    return r;
}

// Weight of a lane's share in combine_tiles: P^(rows that follow the last full tile the
// lane walks).  It depends on the chunk's geometry only, so it is computed once per chunk
// and reused for every replica.
__device__ __forceinline__ uint64_t combine_weight(uint32_t nt, uint64_t nbytes, uint32_t tile_rows,
                                                   uint32_t lane) {
    const uint32_t n_full = nt - 1;  // every tile but the chunk's last has tile_rows rows
    if (lane >= n_full) return 1ull;
    const uint64_t rows_total = (nbytes + ROW_BYTES - 1) / ROW_BYTES;
    const uint64_t rows_last = rows_total - (uint64_t)n_full * tile_rows;
    const uint32_t last_t = lane + ((n_full - 1 - lane) / 32u) * 32u;
    return pow_p(rows_last + (uint64_t)tile_rows * (n_full - 1 - last_t));
}

// SHARED: the records sit in this CTA's shared memory (plain loads) instead of global memory.
template <bool SHARED = false>
__device__ __forceinline__ scout_sig_t combine_tiles(const TileRec *tr, uint32_t nt, uint64_t nbytes,
                                                     uint64_t k, uint32_t dtype, uint64_t meta,
                                                     uint64_t p_stride, uint64_t weight, uint32_t lane) {
    uint64_t h = 0;
    double s = 0.0, q = 0.0;
    uint32_t nan_count = 0, inf_count = 0;
    const uint32_t n_full = nt - 1;
    for (uint32_t t = lane; t < n_full; t += 32) {
        const TileRec x = SHARED ? tr[t] : load_record(tr + t);
        h = h * p_stride + x.h;
        s += x.sum;
        q += x.sumsq;
        nan_count += x.nan_count;
        inf_count += x.inf_count;
    }
    if (lane < n_full) h *= weight;
    if (lane == (n_full & 31u)) {  // the last (possibly short) tile: nothing follows it
        const TileRec x = SHARED ? tr[n_full] : load_record(tr + n_full);
        h += x.h;
        s += x.sum;
        q += x.sumsq;
        nan_count += x.nan_count;
        inf_count += x.inf_count;
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        h += __shfl_xor_sync(0xFFFFFFFFu, h, d);
        s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
        q += __shfl_xor_sync(0xFFFFFFFFu, q, d);
        nan_count += __shfl_xor_sync(0xFFFFFFFFu, nan_count, d);
        inf_count += __shfl_xor_sync(0xFFFFFFFFu, inf_count, d);
    }
    scout_sig_t o;
    o.hash = finalize_hash(h, nbytes, k, dtype, meta);
    o.nan_count = nan_count;
    o.inf_count = inf_count;
    o.sum = s;
    o.sumsq = q;
    return o;
}

// The same combine for a chunk of at most 32 tiles (lane t holds tile t), four replicas
// at a time: their record loads are independent, so they are in flight together.  The
// arithmetic and its order are those of combine_tiles, so the records are identical.
constexpr int COMBINE_BATCH = 4;
__device__ __forceinline__ void combine_small(const TileRec *tr, uint64_t replica_stride, uint32_t n_rep,
                                              uint32_t nt, uint64_t nbytes, uint64_t k, uint32_t dtype,
                                              uint64_t meta, uint64_t weight, uint32_t lane,
                                              scout_sig_t (&o)[COMBINE_BATCH]) {
    TileRec x[COMBINE_BATCH];
#pragma unroll
    for (int j = 0; j < COMBINE_BATCH; ++j) {
        x[j].h = 0; x[j].sum = 0.0; x[j].sumsq = 0.0; x[j].nan_count = 0; x[j].inf_count = 0;
        if ((uint32_t)j < n_rep && lane < nt) x[j] = load_record(tr + (uint64_t)j * replica_stride + lane);
    }
#pragma unroll
    for (int j = 0; j < COMBINE_BATCH; ++j) {
        uint64_t h = lane < nt - 1 ? x[j].h * weight : x[j].h;
        double s = x[j].sum, q = x[j].sumsq;
        uint32_t nan_count = x[j].nan_count, inf_count = x[j].inf_count;
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            h += __shfl_xor_sync(0xFFFFFFFFu, h, d);
            s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
            q += __shfl_xor_sync(0xFFFFFFFFu, q, d);
            nan_count += __shfl_xor_sync(0xFFFFFFFFu, nan_count, d);
            inf_count += __shfl_xor_sync(0xFFFFFFFFu, inf_count, d);
        }
        o[j].hash = finalize_hash(h, nbytes, k, dtype, meta);
        o[j].nan_count = nan_count;
        o[j].inf_count = inf_count;
        o[j].sum = s;
        o[j].sumsq = q;
    }
}


}  // namespace
}  // namespace scout
