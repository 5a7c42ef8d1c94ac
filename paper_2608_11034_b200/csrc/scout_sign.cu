// Comparable evidence (Sec. 5.2): the bulk fold of replica bytes into per-tile
// partial records, and their finalisation into one record per (chunk, replica).
//
// Layout of the scan.  A row is 128 little-endian 32-bit words = 512 bytes =
// one 16-byte vector per lane of a warp.  Lane l always holds words 4l..4l+3 of
// a row, so its four slot multipliers m_{4l..4l+3} are loop constants, and the
// row recurrence h <- h*P + S_q distributes over lanes: every lane runs its own
// recurrence on its share of S_q and the shares are added once per tile
// (integer addition mod 2^64 is order-free).  The fp64 sums use a fixed
// lane -> element mapping and a fixed butterfly, so results are bitwise
// reproducible.
//
// Non-finite values.  The hot loop does not classify elements.  Every finite
// fp32/bf16/fp16 square is below 2^256 and every non-finite element pushes the
// naive sum of squares to at least 2^256 (or NaN), so "!(sumsq < 2^256)" is a
// necessary condition for a non-finite element in the tile.  A tile that trips
// it is scanned again (it is still in L2) by a loop that classifies every
// element, counts NaN/Inf and sums the finite ones only.
#include <cuda_fp16.h>

#include <mutex>
#include <type_traits>

#include <cstddef>

#include "scout_internal.h"
#include "scout_vote_device.cuh"

namespace scout {
namespace {

constexpr int SIGN_THREADS = 256;
// Compile-time settings (the defaults are the measured optimum on B200; build.py
// can compile a copy with others, selected at run time by the SCOUT_LIB variable):
//   SCOUT_UNROLL         rows (16 B per lane each) a warp has in flight, direct scan
//   SCOUT_MINBLOCKS      CTAs per SM the direct scan is compiled for (caps registers)
//   SCOUT_MINBLOCKS_PF   the same for the register-prefetch front end
//   SCOUT_BF16_BITROUTE  see below
//   SCOUT_RING_PIECE / _STAGES / _BLOCKS   geometry of the per-warp bulk-async ring
#ifndef SCOUT_MINBLOCKS
#define SCOUT_MINBLOCKS 4
#endif
#ifndef SCOUT_MINBLOCKS_PF
#define SCOUT_MINBLOCKS_PF 3
#endif
#ifndef SCOUT_UNROLL
#define SCOUT_UNROLL 8
#endif


constexpr int UNROLL = SCOUT_UNROLL;
// bf16: how many of a word-quad's four high halves are widened by bit placement
// instead of the conversion pipe (see stats_fast).  Default 0: every instruction costs about
// 1.6 issue cycles whatever its pipe, so the route with the fewest instructions wins even
// though it keeps the conversion pipe busiest (measured on 125 GB of bf16: 6,361 GB/s with 0,
// 6,282 with 1, 6,223 with 2, 6,016 with 3).
#ifndef SCOUT_BF16_BITROUTE
#define SCOUT_BF16_BITROUTE 0
#endif

constexpr int BF16_BITROUTE = SCOUT_BF16_BITROUTE;

struct Acc {
    double s0, s1, q0, q1;
};

// Streaming 16-byte load: read-only path, no L1 allocation (the data is used once).
// .cs, L2::256B prefetch and evict-first hints measured the same on B200.
__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 16 bytes at tile[byte_off..], bytes at or past nbytes read as zero.  Only
// the last row of a chunk can be ragged, so the byte loop is off the hot path.
__device__ __noinline__ uint4 ld_masked16(const uint8_t *tile, uint32_t byte_off, uint32_t nbytes) {
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (byte_off + 16u <= nbytes) {
        uint4 v = ld_stream16(tile + byte_off);
        return v;
    }
    if (byte_off < nbytes) {
        uint32_t n = nbytes - byte_off;
        for (uint32_t i = 0; i < n; ++i) w[i >> 2] |= (uint32_t)tile[byte_off + i] << (8u * (i & 3u));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void acc2(Acc &a, double x0, double x1) {
    a.s0 += x0;
    a.q0 = fma(x0, x0, a.q0);
    a.s1 += x1;
    a.q1 = fma(x1, x1, a.q1);
}

// ---- per-dtype element paths: fast (no classification) -----------------------
template <int DT>
__device__ __forceinline__ void stats_fast(const uint4 &v, Acc &a) {
    if constexpr (DT == SCOUT_DT_F32) {
        acc2(a, (double)__uint_as_float(v.x), (double)__uint_as_float(v.y));
        acc2(a, (double)__uint_as_float(v.z), (double)__uint_as_float(v.w));
    } else if constexpr (DT == SCOUT_DT_BF16) {
        // Two widening routes, mixed so that the conversion pipe (16 lanes/clk/SM)
        // does not carry all eight elements of a vector.
        //  (A) cvt.f64.bf16 straight from either half of the word; accumulators
        //      s0, q0 hold true values.
        //  (B) bit placement, no conversion: the bf16 pattern dropped into the top
        //      of a double's exponent/mantissa gives u = x * 2^-896 exactly for
        //      every finite x (zeros and subnormals included); OR-ing 0x700 into
        //      the exponent field gives v = x * 2^+896 for every NORMAL x (garbage
        //      but finite for zeros and subnormals), so u*v = x^2 exactly for
        //      normal x and for zero.  s1 sums u (rescaled once per tile), q1 sums
        //      u*v.  A subnormal x contributes a wrong but tiny (< 2^-252) term to
        //      q1; lanes with 0 < q1 < 2^-180 send the tile to the exact rescan, so
        //      the error that can remain is below 2^-58 relative.
        //      Inf/NaN give v = Inf/NaN: the usual "sum of squares not finite" flag.
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint16_t l16, h16;
            asm("mov.b32 {%0,%1}, %2;" : "=h"(l16), "=h"(h16) : "r"(w[i]));
            double lo;
            asm("cvt.f64.bf16 %0, %1;" : "=d"(lo) : "h"(l16));
            a.s0 += lo;
            a.q0 = fma(lo, lo, a.q0);
            if (i < BF16_BITROUTE) {
                const uint32_t uh = (uint32_t)((int)w[i] >> 3) & 0x8FFFE000u;
                const double u = __hiloint2double((int)uh, 0);
                const double x2 = __hiloint2double((int)(uh | 0x70000000u), 0);
                a.s1 += u;
                a.q1 = fma(u, x2, a.q1);
            } else {
                double hi;
                asm("cvt.f64.bf16 %0, %1;" : "=d"(hi) : "h"(h16));
                if (BF16_BITROUTE > 0) {
                    a.s0 += hi;
                    a.q0 = fma(hi, hi, a.q0);
                } else {
                    a.s1 += hi;
                    a.q1 = fma(hi, hi, a.q1);
                }
            }
        }
    } else if constexpr (DT == SCOUT_DT_F16) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint16_t l16, h16;
            double lo, hi;
            asm("mov.b32 {%0,%1}, %2;" : "=h"(l16), "=h"(h16) : "r"(w[i]));
            asm("cvt.f64.f16 %0, %1;" : "=d"(lo) : "h"(l16));
            asm("cvt.f64.f16 %0, %1;" : "=d"(hi) : "h"(h16));
            acc2(a, lo, hi);
        }
    } else if constexpr (DT == SCOUT_DT_F64) {
        acc2(a, __hiloint2double((int)v.y, (int)v.x), __hiloint2double((int)v.w, (int)v.z));
    } else if constexpr (DT == SCOUT_DT_I64) {
        acc2(a, (double)(long long)(((uint64_t)v.y << 32) | v.x),
             (double)(long long)(((uint64_t)v.w << 32) | v.z));
    } else if constexpr (DT == SCOUT_DT_I32) {
        acc2(a, (double)(int)v.x, (double)(int)v.y);
        acc2(a, (double)(int)v.z, (double)(int)v.w);
    }
}

template <int DT>
__device__ __forceinline__ bool may_hold_nonfinite(const Acc &a) {
    if constexpr (DT == SCOUT_DT_BF16) {
        // non-finite element, or a subnormal one on the bit-placement route
        return !(a.q0 + a.q1 < 1.157920892373162e77) ||                    // 2^256
               (BF16_BITROUTE > 0 && a.q1 > 0.0 && a.q1 < 6.525304467998525e-55);  // 2^-180
    } else if constexpr (DT == SCOUT_DT_F32 || DT == SCOUT_DT_F16) {
        return !(a.q0 + a.q1 < 1.157920892373162e77);  // 2^256
    } else if constexpr (DT == SCOUT_DT_F64) {
        return !(a.q0 + a.q1 < __longlong_as_double(0x7FF0000000000000ll));
    } else {
        return false;
    }
}

// ---- per-dtype element paths: classifying (slow) ------------------------------
struct SlowAcc {
    double s, q;
    uint32_t nan_count, inf_count;
};

__device__ __forceinline__ void slow_add(SlowAcc &a, double x, bool nonfinite, bool is_nan) {
    if (nonfinite) {
        if (is_nan) ++a.nan_count; else ++a.inf_count;
    } else {
        a.s += x;
        a.q = fma(x, x, a.q);
    }
}

template <int DT>
__device__ __forceinline__ void stats_slow(const uint4 &v, SlowAcc &a) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if constexpr (DT == SCOUT_DT_F32) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            slow_add(a, (double)__uint_as_float(w[i]), (w[i] & 0x7F800000u) == 0x7F800000u,
                     (w[i] & 0x007FFFFFu) != 0u);
    } else if constexpr (DT == SCOUT_DT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t lo = w[i] << 16, hi = w[i] & 0xFFFF0000u;
            slow_add(a, (double)__uint_as_float(lo), (lo & 0x7F800000u) == 0x7F800000u, (lo & 0x007F0000u) != 0u);
            slow_add(a, (double)__uint_as_float(hi), (hi & 0x7F800000u) == 0x7F800000u, (hi & 0x007F0000u) != 0u);
        }
    } else if constexpr (DT == SCOUT_DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            uint32_t lo = w[i] & 0xFFFFu, hi = w[i] >> 16;
            slow_add(a, (double)f.x, (lo & 0x7C00u) == 0x7C00u, (lo & 0x03FFu) != 0u);
            slow_add(a, (double)f.y, (hi & 0x7C00u) == 0x7C00u, (hi & 0x03FFu) != 0u);
        }
    } else if constexpr (DT == SCOUT_DT_F64) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            uint32_t lo = w[2 * i], hi = w[2 * i + 1];
            slow_add(a, __hiloint2double((int)hi, (int)lo), (hi & 0x7FF00000u) == 0x7FF00000u,
                     ((hi & 0x000FFFFFu) | lo) != 0u);
        }
    }
}

template <int DT>
__device__ __noinline__ void rescan_classifying(const uint8_t *tile, uint32_t nbytes, uint32_t lane,
                                                double &sum, double &sumsq, uint32_t &nan_count,
                                                uint32_t &inf_count) {
    SlowAcc a = {0.0, 0.0, 0u, 0u};
    const uint32_t rows = (nbytes + ROW_BYTES - 1) / ROW_BYTES;
    for (uint32_t row = 0; row < rows; ++row) {
        uint4 v = ld_masked16(tile, row * ROW_BYTES + 16u * lane, nbytes);
        stats_slow<DT>(v, a);
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        a.s += __shfl_xor_sync(0xFFFFFFFFu, a.s, d);
        a.q += __shfl_xor_sync(0xFFFFFFFFu, a.q, d);
        a.nan_count += __shfl_xor_sync(0xFFFFFFFFu, a.nan_count, d);
        a.inf_count += __shfl_xor_sync(0xFFFFFFFFu, a.inf_count, d);
    }
    sum = a.s;
    sumsq = a.q;
    nan_count = a.nan_count;
    inf_count = a.inf_count;
}

// h <- h * P + (m0 w0 + m1 w1 + m2 w2 + m3 w3) mod 2^64.  Starting the chain from
// h * P lets every product be a 32x32+64 multiply-add (measured: fewest
// instructions of the forms tried; a 64-bit accumulate costs two issue slots).
__device__ __forceinline__ void fold_row(uint64_t &h, const uint4 &v, const uint32_t (&m)[4]) {
    uint64_t t = h * HASH_P;
    t += (uint64_t)m[0] * v.x;
    t += (uint64_t)m[1] * v.y;
    t += (uint64_t)m[2] * v.z;
    t += (uint64_t)m[3] * v.w;
    h = t;
}

// Per-lane state of one tile's scan: the lane's four slot multipliers, its share
// of the hash recurrence, and its fp64 accumulators.  Rows may be fed from
// registers (direct loads) or from shared memory (bulk-async ring); the
// arithmetic is the same.
template <int DT>
struct TileScan {
    uint32_t m[4];
    uint64_t h;
    Acc a;

    __device__ __forceinline__ void begin(uint32_t lane) {
#pragma unroll
        for (int j = 0; j < 4; ++j) m[j] = ((4u * lane + j + 1u) * HASH_G32) | 1u;
        h = 0;
        a = Acc{0.0, 0.0, 0.0, 0.0};
    }
    // the two halves of a row's work, separately (the cost microbenchmark times each alone)
    __device__ __forceinline__ void row_hash(const uint4 &v) { fold_row(h, v, m); }
    __device__ __forceinline__ void row_stats(const uint4 &v) { stats_fast<DT>(v, a); }
    __device__ __forceinline__ void row(const uint4 &v) {
        fold_row(h, v, m);
        stats_fast<DT>(v, a);
    }
    // Warp reduction of what the lanes hold: hash share, sums, and whether any lane
    // suspects a non-finite (or, for bf16, subnormal) element.
    __device__ __forceinline__ void reduce(uint64_t &h_out, double &s, double &q, bool &suspect) const {
        q = a.q0 + a.q1;
        if constexpr (DT == SCOUT_DT_BF16 && BF16_BITROUTE > 0)
            s = fma(a.s1, 0x1p896, a.s0);  // s1 holds x * 2^-896: exact power-of-two rescale
        else
            s = a.s0 + a.s1;
        suspect = __any_sync(0xFFFFFFFFu, may_hold_nonfinite<DT>(a));
        h_out = h;
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            h_out += __shfl_xor_sync(0xFFFFFFFFu, h_out, d);
            s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
            q += __shfl_xor_sync(0xFFFFFFFFu, q, d);
        }
    }
    // Ragged last row of a chunk (missing words are zero), warp reduction, and the
    // classifying rescan if the tile may hold a non-finite element.
    __device__ __forceinline__ void finish(const uint8_t *tile, uint32_t nbytes, uint32_t lane,
                                           TileRec &out) {
        if (nbytes % ROW_BYTES) {
            uint4 v = ld_masked16(tile, (nbytes / ROW_BYTES) * ROW_BYTES + 16u * lane, nbytes);
            row(v);
        }
        double s, q;
        bool suspect;
        uint64_t h_tile;
        reduce(h_tile, s, q, suspect);
        uint32_t nan_count = 0, inf_count = 0;
        if constexpr (DT == SCOUT_DT_F32 || DT == SCOUT_DT_BF16 || DT == SCOUT_DT_F16 ||
                      DT == SCOUT_DT_F64) {
            if (suspect) rescan_classifying<DT>(tile, nbytes, lane, s, q, nan_count, inf_count);
        }
        out.h = h_tile;
        out.sum = s;
        out.sumsq = q;
        out.nan_count = nan_count;
        out.inf_count = inf_count;
    }
};

// Front end 0: one warp scans one tile with direct 16-byte loads, UNROLL rows in
// flight, no overlap of a warp's own loads with its own arithmetic.
template <int DT>
__device__ __forceinline__ void scan_tile(const uint8_t *tile, uint32_t nbytes, uint32_t lane,
                                          TileRec &out) {
    TileScan<DT> st;
    st.begin(lane);
    const uint32_t full = nbytes / ROW_BYTES;
    const uint8_t *p = tile + 16u * lane;
#pragma unroll 1
    for (uint32_t b = full / UNROLL; b != 0; --b, p += UNROLL * ROW_BYTES) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream16(p + u * ROW_BYTES);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) st.row(v[u]);
    }
#pragma unroll 1
    for (uint32_t b = full % UNROLL; b != 0; --b, p += ROW_BYTES) st.row(ld_stream16(p));
    st.finish(tile, nbytes, lane, out);
}

// Front end 1: rotating register pipeline.  PF_ROWS rows are always in flight:
// as soon as a row has been folded its registers are reloaded with the row
// PF_ROWS ahead, so a warp's loads overlap its own arithmetic.
#ifndef SCOUT_PF_ROWS
#define SCOUT_PF_ROWS 4
#endif
constexpr int PF_ROWS = SCOUT_PF_ROWS;

template <int DT>
__device__ __forceinline__ void scan_tile_prefetch(const uint8_t *tile, uint32_t nbytes, uint32_t lane,
                                                   TileRec &out) {
    TileScan<DT> st;
    st.begin(lane);
    const uint32_t full = nbytes / ROW_BYTES;
    const uint8_t *p = tile + 16u * lane;
    const uint8_t *const end_full = p + (size_t)full * ROW_BYTES;
    if (full >= PF_ROWS) {
        // rows [p, p + PF_ROWS) are in registers; the loop reloads each register with
        // the row PF_ROWS further on while there are at least PF_ROWS more rows
        const uint8_t *const end_steady = p + (size_t)(full / PF_ROWS - 1) * (PF_ROWS * ROW_BYTES);
        uint4 v[PF_ROWS];
#pragma unroll
        for (int u = 0; u < PF_ROWS; ++u) v[u] = ld_stream16(p + u * ROW_BYTES);
#pragma unroll 1
        for (; p != end_steady; p += PF_ROWS * ROW_BYTES) {
#pragma unroll
            for (int u = 0; u < PF_ROWS; ++u) {
                st.row(v[u]);
                v[u] = ld_stream16(p + (PF_ROWS + u) * ROW_BYTES);
            }
        }
#pragma unroll
        for (int u = 0; u < PF_ROWS; ++u) st.row(v[u]);
        p += PF_ROWS * ROW_BYTES;
    }
    for (; p != end_full; p += ROW_BYTES) st.row(ld_stream16(p));
    st.finish(tile, nbytes, lane, out);
}

struct SignArgs {
    const TileDesc *tiles;
    uint64_t tile_begin, n_tiles, tiles_per_replica;
    uint32_t replica_begin, n_replicas;
    const uint8_t *const *ptrs;
    uint64_t T;
    const uint8_t *stage;
    uint64_t slice_begin;
    TileRec *recs;
    uint32_t *error;  // device flag: set if a bounded wait gave up
    // dynamic work distribution of the direct scan: two counters used alternately by
    // successive launches (null: static round-robin), and this launch's parity
    unsigned long long *work;
    uint32_t work_parity;
};

__device__ __forceinline__ void scan_dispatch(uint32_t dtype, const uint8_t *tile, uint32_t nbytes,
                                              uint32_t lane, TileRec &rec) {
    switch (dtype) {
        case SCOUT_DT_F32:  scan_tile<SCOUT_DT_F32>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_BF16: scan_tile<SCOUT_DT_BF16>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_I64:  scan_tile<SCOUT_DT_I64>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_F16:  scan_tile<SCOUT_DT_F16>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_F64:  scan_tile<SCOUT_DT_F64>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_I32:  scan_tile<SCOUT_DT_I32>(tile, nbytes, lane, rec); break;
        default:            scan_tile<SCOUT_DT_U8>(tile, nbytes, lane, rec); break;
    }
}

__device__ __forceinline__ void scan_dispatch_prefetch(uint32_t dtype, const uint8_t *tile,
                                                       uint32_t nbytes, uint32_t lane, TileRec &rec) {
    switch (dtype) {
        case SCOUT_DT_F32:  scan_tile_prefetch<SCOUT_DT_F32>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_BF16: scan_tile_prefetch<SCOUT_DT_BF16>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_I64:  scan_tile_prefetch<SCOUT_DT_I64>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_F16:  scan_tile_prefetch<SCOUT_DT_F16>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_F64:  scan_tile_prefetch<SCOUT_DT_F64>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_I32:  scan_tile_prefetch<SCOUT_DT_I32>(tile, nbytes, lane, rec); break;
        default:            scan_tile_prefetch<SCOUT_DT_U8>(tile, nbytes, lane, rec); break;
    }
}

__device__ __forceinline__ const uint8_t *tile_address(const SignArgs &a, const TileDesc &td, uint32_t r) {
    return a.ptrs ? a.ptrs[(uint64_t)r * a.T + td.tensor] + td.off : a.stage + (td.poff - a.slice_begin);
}

__device__ __forceinline__ void store_record(TileRec *dst_rec, const TileRec &rec) {
    uint4 *dst = reinterpret_cast<uint4 *>(dst_rec);
    dst[0] = make_uint4((uint32_t)rec.h, (uint32_t)(rec.h >> 32), (uint32_t)__double2loint(rec.sum),
                        (uint32_t)__double2hiint(rec.sum));
    dst[1] = make_uint4((uint32_t)__double2loint(rec.sumsq), (uint32_t)__double2hiint(rec.sumsq),
                        rec.nan_count, rec.inf_count);
}

// Persistent grid; every warp takes whole tiles, replica-major, round-robin.
// DTSEL >= 0: every tile of the launch has that dtype (the element path is fixed at
// compile time, so the register allocation is that path's, not the union of all
// seven); DTSEL < 0: the dtype is read from the tile table.
template <int PREFETCH, int DTSEL>
__global__ void __launch_bounds__(SIGN_THREADS, PREFETCH ? SCOUT_MINBLOCKS_PF : SCOUT_MINBLOCKS) sign_tiles_direct(const SignArgs a) {
    pdl_launch_dependents();
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (SIGN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (SIGN_THREADS / 32);
    const uint64_t n_items = a.n_tiles * a.n_replicas;
    // Every warp starts with item `warp`.  With a work counter the later items are handed out
    // in order as warps become free (tiles differ in size and dtype, so a fixed round-robin
    // leaves some warps with more bytes than others); the request for the next item is made
    // before the current tile is scanned and its answer is read after it.  The counter of this
    // launch is work[parity]; the other one is zeroed here for the launch that follows.
    unsigned long long *work = a.work ? a.work + a.work_parity : nullptr;
    if (work && warp == 0 && lane == 0) a.work[a.work_parity ^ 1u] = 0ull;
    const bool dynamic = work != nullptr && n_items > n_warps;
    uint64_t item = warp;
    while (item < n_items) {
        unsigned long long next = 0;
        if (dynamic) {
            if (lane == 0) next = atomicAdd(work, 1ull);
        }
        const uint32_t rr = (uint32_t)(item / a.n_tiles);
        const uint64_t t = a.tile_begin + (item - (uint64_t)rr * a.n_tiles);
        const uint32_t r = a.replica_begin + rr;
        const TileDesc td = a.tiles[t];
        const uint8_t *tile = tile_address(a, td, r);
        TileRec rec;
        if constexpr (DTSEL >= 0) {
            if (PREFETCH) scan_tile_prefetch<DTSEL>(tile, td.nbytes, lane, rec);
            else          scan_tile<DTSEL>(tile, td.nbytes, lane, rec);
        } else {
            if (PREFETCH) scan_dispatch_prefetch(td.dtype, tile, td.nbytes, lane, rec);
            else          scan_dispatch(td.dtype, tile, td.nbytes, lane, rec);
        }
        if (lane == 0) store_record(&a.recs[(uint64_t)r * a.tiles_per_replica + t], rec);
        item = dynamic ? n_warps + __shfl_sync(0xFFFFFFFFu, next, 0) : item + n_warps;
    }
}

using SignKernel = void (*)(const SignArgs);
// The direct-scan kernel for a front end (0 direct, 1 register prefetch) and a launch
// whose tiles all have dtype `uniform` (specialised for fp32 and bf16), or mixed (-1).
SignKernel direct_kernel(int prefetch, int uniform) {
    if (prefetch) {
        if (uniform == SCOUT_DT_F32) return sign_tiles_direct<1, SCOUT_DT_F32>;
        if (uniform == SCOUT_DT_BF16) return sign_tiles_direct<1, SCOUT_DT_BF16>;
        return sign_tiles_direct<1, -1>;
    }
    if (uniform == SCOUT_DT_F32) return sign_tiles_direct<0, SCOUT_DT_F32>;
    if (uniform == SCOUT_DT_BF16) return sign_tiles_direct<0, SCOUT_DT_BF16>;
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

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
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
    const uint64_t n_warps = (uint64_t)gridDim.x * (SIGN_THREADS / 32);
    const uint64_t n_items = a.n_tiles * a.n_replicas;
    // the same work distribution as the scan (see sign_tiles_direct)
    unsigned long long *work = a.work ? a.work + a.work_parity : nullptr;
    if (work && warp == 0 && lane == 0) a.work[a.work_parity ^ 1u] = 0ull;
    const bool dynamic = work != nullptr && n_items > n_warps;
    uint64_t item = warp;
    while (item < n_items) {
        unsigned long long next = 0;
        if (dynamic) {
            if (lane == 0) next = atomicAdd(work, 1ull);
        }
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
        item = dynamic ? n_warps + __shfl_sync(0xFFFFFFFFu, next, 0) : item + n_warps;
    }
}

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


__global__ void __launch_bounds__(FIN_THREADS) finalize_chunks(const ChunkDesc *chunks, uint64_t C,
                                                               uint32_t R, const TileRec *recs,
                                                               uint64_t tiles_per_replica,
                                                               uint32_t tile_rows, uint64_t p_stride,
                                                               scout_sig_t *sigs, CertifyOut *zero_out) {
    pdl_launch_dependents();
    pdl_wait();
    if (zero_out && blockIdx.x == 0 && threadIdx.x < sizeof(CertifyOut) / sizeof(uint64_t))
        reinterpret_cast<uint64_t *>(zero_out)[threadIdx.x] = 0ull;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (FIN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (FIN_THREADS / 32);
    for (uint64_t item = warp; item < C * R; item += n_warps) {
        const uint64_t c = item / R;
        const uint32_t r = (uint32_t)(item - c * R);
        const ChunkDesc cd = chunks[c];
        const scout_sig_t o = combine_tiles(recs + (uint64_t)r * tiles_per_replica + cd.tile0, cd.ntiles,
                                            cd.nbytes, cd.k, cd.dtype, cd.meta, p_stride,
                                            combine_weight(cd.ntiles, cd.nbytes, tile_rows, lane), lane);
        if (lane == 0) {
            sigs[c * R + r] = o;
        }
    }
}


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
        if constexpr (DTSEL >= 0) scan_tile<DTSEL>(tile, td.nbytes, lane, rec);
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
            if constexpr (DTSEL >= 0) scan_tile<DTSEL>(base + off, nbytes, lane, rec);
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

namespace {
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
                    uint64_t tiles_per_replica, uint32_t tile_rows, scout_sig_t *d_sigs,
                    CertifyOut *zero_out, cudaStream_t stream) {
    if (C == 0) return SCOUT_OK;
    const uint64_t items = C * R;
    uint64_t blocks = (items + FIN_THREADS / 32 - 1) / (FIN_THREADS / 32);
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    static_assert(sizeof(CertifyOut) / sizeof(uint64_t) <= FIN_THREADS, "one thread per word clears it");
    SCOUT_CUDA(launch_dependent(finalize_chunks, dim3((unsigned)blocks), dim3(FIN_THREADS), stream, chunks, C,
                                R, recs, tiles_per_replica, tile_rows, pow_p(32ull * tile_rows), d_sigs,
                                zero_out));
    return SCOUT_OK;
}

}  // namespace scout

// ---- signing without any allocation ------------------------------------------
// scout_sign_chunks_noalloc serves callers that must not allocate device memory
// while they run: a health check placed in the middle of a training step, where
// the framework's caching allocator already holds almost all of HBM (a
// cudaMalloc there can fail, and it also stalls the device), or a handler that
// runs right after an out-of-memory error.  It takes no plan: the replicas are R
// contiguous buffers holding one tensor each, and the per-tile partial records
// go to a fixed array that lives in the library's device image.
namespace scout {
namespace {

constexpr uint32_t NOALLOC_MAX_RECORDS = 65536;  // 2 MiB of scratch, held by every GPU that loads the library
constexpr uint32_t NOALLOC_MAX_DEVICES = 64;

// The scratch itself.  In host code this name is only a stand-in for the
// symbol, not an address a kernel can use; the host obtains the device address
// with cudaGetSymbolAddress (below) and passes that to the kernels.
// Eight records (256 bytes) of guard band on either side: they are filled with a pattern at
// set-up and scout_noalloc_guards_ok() checks that no kernel has written to them.
constexpr uint32_t NOALLOC_GUARD_RECORDS = 8;
constexpr int NOALLOC_GUARD_PATTERN = 0xC3;
static __device__ __align__(256) TileRec g_noalloc_scratch[NOALLOC_GUARD_RECORDS + NOALLOC_MAX_RECORDS +
                                                           NOALLOC_GUARD_RECORDS];

struct NoallocArgs {
    const uint8_t *replica[64];
    uint64_t nbytes, chunk_bytes, meta;
    uint64_t n_tiles;          // tiles per replica
    uint32_t tiles_per_chunk;  // tiles of a full chunk
    uint32_t tile_bytes;
    uint32_t R, dtype;
    TileRec *recs;             // device address of g_noalloc_scratch
    scout_sig_t *sigs;
};

// Same scan as sign_tiles_direct, with the tile geometry computed from the tile
// index instead of read from a table (there is no table: nothing was allocated).
__global__ void __launch_bounds__(SIGN_THREADS) sign_tiles_noalloc(const __grid_constant__ NoallocArgs a) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (SIGN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (SIGN_THREADS / 32);
    const uint64_t n_items = a.n_tiles * a.R;
    for (uint64_t item = warp; item < n_items; item += n_warps) {
        const uint32_t r = (uint32_t)(item / a.n_tiles);
        const uint64_t t = item - (uint64_t)r * a.n_tiles;
        const uint64_t c = t / a.tiles_per_chunk;
        const uint64_t j = t - c * a.tiles_per_chunk;
        const uint64_t chunk_off = c * a.chunk_bytes;
        const uint64_t chunk_n = min(a.chunk_bytes, a.nbytes - chunk_off);
        const uint64_t in_chunk = j * a.tile_bytes;
        const uint32_t n = (uint32_t)min((uint64_t)a.tile_bytes, chunk_n - in_chunk);
        TileRec rec;
        scan_dispatch(a.dtype, a.replica[r] + chunk_off + in_chunk, n, lane, rec);
        if (lane == 0) a.recs[(uint64_t)r * a.n_tiles + t] = rec;
    }
}

// The combine of finalize_chunks for a single tensor whose chunk geometry is arithmetic.
__global__ void __launch_bounds__(FIN_THREADS) finalize_noalloc(const __grid_constant__ NoallocArgs a,
                                                                uint64_t C, uint64_t p_stride) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (FIN_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (FIN_THREADS / 32);
    const uint32_t tile_rows = a.tile_bytes / ROW_BYTES;
    for (uint64_t item = warp; item < C * a.R; item += n_warps) {
        const uint64_t c = item / a.R;
        const uint32_t r = (uint32_t)(item - c * a.R);
        const uint64_t chunk_n = min(a.chunk_bytes, a.nbytes - c * a.chunk_bytes);
        const uint32_t nt = (uint32_t)((chunk_n + a.tile_bytes - 1) / a.tile_bytes);
        const scout_sig_t o = combine_tiles(a.recs + (uint64_t)r * a.n_tiles + c * a.tiles_per_chunk, nt,
                                            chunk_n, c, a.dtype, a.meta, p_stride,
                                            combine_weight(nt, chunk_n, tile_rows, lane), lane);
        if (lane == 0) {
            a.sigs[c * a.R + r] = o;
        }
    }
}

// Device address of the scratch array and SM count, looked up once per device.
// The table is filled under a mutex, so that host threads making their first call
// at the same time do not race on it.
struct NoallocDevice {
    TileRec *scratch;
    int sms;
    bool ready;
};
static NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
static std::mutex g_noalloc_mutex;

int noalloc_setup(int device, NoallocDevice *out) {
    if (device < 0 || device >= (int)NOALLOC_MAX_DEVICES) return SCOUT_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(g_noalloc_mutex);
    NoallocDevice &d = g_noalloc_dev[device];
    if (!d.ready) {
        // `device` is the current device here, so the address is this GPU's copy
        void *ptr = nullptr;
        SCOUT_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        int sms = 0;
        SCOUT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        TileRec *base = static_cast<TileRec *>(ptr);
        SCOUT_CUDA(cudaMemset(base, NOALLOC_GUARD_PATTERN, NOALLOC_GUARD_RECORDS * sizeof(TileRec)));
        SCOUT_CUDA(cudaMemset(base + NOALLOC_GUARD_RECORDS + NOALLOC_MAX_RECORDS, NOALLOC_GUARD_PATTERN,
                              NOALLOC_GUARD_RECORDS * sizeof(TileRec)));
        d.scratch = base + NOALLOC_GUARD_RECORDS;
        d.sms = sms;
        d.ready = true;
    }
    *out = d;
    return SCOUT_OK;
}

}  // namespace
}  // namespace scout

extern "C" int scout_noalloc_guards_ok(int *ok) {
    using namespace scout;
    if (!ok) return SCOUT_ERR_INVALID;
    int device = 0;
    SCOUT_CUDA(cudaGetDevice(&device));
    NoallocDevice dev;
    int rc = noalloc_setup(device, &dev);
    if (rc) return rc;
    SCOUT_CUDA(cudaDeviceSynchronize());
    uint8_t host[2 * NOALLOC_GUARD_RECORDS * sizeof(TileRec)];
    const size_t band = NOALLOC_GUARD_RECORDS * sizeof(TileRec);
    SCOUT_CUDA(cudaMemcpy(host, dev.scratch - NOALLOC_GUARD_RECORDS, band, cudaMemcpyDeviceToHost));
    SCOUT_CUDA(cudaMemcpy(host + band, dev.scratch + NOALLOC_MAX_RECORDS, band, cudaMemcpyDeviceToHost));
    *ok = 1;
    for (uint8_t b : host)
        if (b != (uint8_t)NOALLOC_GUARD_PATTERN) *ok = 0;
    return SCOUT_OK;
}

extern "C" int scout_sign_chunks_noalloc(uint32_t R, const void *const *replica_ptrs, uint64_t nbytes,
                                         uint32_t dtype, uint64_t meta_tag, uint64_t chunk_bytes,
                                         scout_sig_t *d_sigs, void *stream) {
    using namespace scout;
    if (R < 2 || !replica_ptrs || !d_sigs || nbytes == 0) return SCOUT_ERR_INVALID;
    if (R > 64) return SCOUT_ERR_UNSUPPORTED;
    if (chunk_bytes == 0 || chunk_bytes % ROW_BYTES != 0 || chunk_bytes > (1ull << 30))
        return SCOUT_ERR_INVALID;
    static const uint32_t elem[7] = {1, 4, 2, 8, 2, 8, 4};
    if (dtype > SCOUT_DT_I32 || nbytes % elem[dtype] != 0) return SCOUT_ERR_INVALID;
    for (uint32_t r = 0; r < R; ++r) {
        if (!replica_ptrs[r]) return SCOUT_ERR_INVALID;
        if ((uintptr_t)replica_ptrs[r] & 15u) return SCOUT_ERR_ALIGN;
    }
    // smallest tile (power of two, 2 KiB .. 64 KiB) whose records fit the fixed scratch
    const uint64_t C = (nbytes + chunk_bytes - 1) / chunk_bytes;
    const uint64_t last_n = nbytes - (C - 1) * chunk_bytes;
    uint32_t tile = 2048;
    uint64_t tpc = 0, n_tiles = 0;
    for (;; tile *= 2) {
        tpc = (chunk_bytes + tile - 1) / tile;
        n_tiles = (C - 1) * tpc + (last_n + tile - 1) / tile;
        if (n_tiles * R <= NOALLOC_MAX_RECORDS) break;
        if (tile == 65536) return SCOUT_ERR_UNSUPPORTED;  // more data than the fixed scratch covers
    }
    int device = 0;
    SCOUT_CUDA(cudaGetDevice(&device));
    NoallocDevice dev_info;
    int rc = noalloc_setup(device, &dev_info);
    if (rc) return rc;
    const NoallocDevice *dev = &dev_info;

    NoallocArgs a;
    for (uint32_t r = 0; r < 64; ++r) a.replica[r] = r < R ? (const uint8_t *)replica_ptrs[r] : nullptr;
    a.nbytes = nbytes;
    a.chunk_bytes = chunk_bytes;
    a.meta = meta_tag;
    a.n_tiles = n_tiles;
    a.tiles_per_chunk = (uint32_t)tpc;
    a.tile_bytes = tile;
    a.R = R;
    a.dtype = dtype;
    a.recs = dev->scratch;
    a.sigs = d_sigs;
    cudaStream_t s = (cudaStream_t)stream;
    const uint64_t items = n_tiles * R;
    uint64_t grid = (items + SIGN_THREADS / 32 - 1) / (SIGN_THREADS / 32);
    if (grid > (uint64_t)dev->sms * 4) grid = (uint64_t)dev->sms * 4;
    sign_tiles_noalloc<<<(unsigned)grid, SIGN_THREADS, 0, s>>>(a);
    SCOUT_CUDA(cudaGetLastError());
    uint64_t fgrid = (C * R + FIN_THREADS / 32 - 1) / (FIN_THREADS / 32);
    if (fgrid > (uint64_t)dev->sms * 8) fgrid = (uint64_t)dev->sms * 8;
    finalize_noalloc<<<(unsigned)fgrid, FIN_THREADS, 0, s>>>(a, C, pow_p(32ull * (tile / ROW_BYTES)));
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}
