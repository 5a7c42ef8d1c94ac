// Comparable evidence (Sec. 5.2): the row routine of the bulk fold, i.e. what one warp
// does with one tile of replica bytes.  Included by every translation unit that has a
// scan kernel (the staged scan, the one-launch kernels, the no-allocation entry point).
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
#pragma once

#include <cuda_fp16.h>

#include <cstddef>
#include <type_traits>

#include "scout_internal.h"

namespace scout {
namespace {

constexpr int SIGN_THREADS = 256;
// Compile-time settings (the defaults are the measured optimum on B200; build.py
// can compile a copy with others, selected at run time by the SCOUT_LIB variable):
//   SCOUT_UNROLL         rows (16 B per lane each) a warp has in flight, direct scan
//   SCOUT_MINBLOCKS      CTAs per SM the direct scan is compiled for (caps registers)
//   SCOUT_MINBLOCKS_PF   the same for the register-prefetch front end
//   SCOUT_PF_ROWS        rows the register-prefetch front end keeps in flight
//   SCOUT_PF_BITROUTE    bf16 elements per word quad it widens by bit placement
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
// instead of the conversion pipe (see stats_fast), in every front end but the register
// pipeline (which has its own setting, PF_BITROUTE).  Default 0: where a warp also sits out
// its own load latency every instruction costs about 1.6 issue cycles whatever its pipe, so
// the route with the fewest instructions wins even though it keeps the conversion pipe
// busiest (measured on 125 GB of bf16: 6,361 GB/s with 0, 6,282 with 1, 6,223 with 2, 6,016 with 3).
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
template <int DT, int BITROUTE = BF16_BITROUTE>
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
            if (i < BITROUTE) {
                const uint32_t uh = (uint32_t)((int)w[i] >> 3) & 0x8FFFE000u;
                const double u = __hiloint2double((int)uh, 0);
                const double x2 = __hiloint2double((int)(uh | 0x70000000u), 0);
                a.s1 += u;
                a.q1 = fma(u, x2, a.q1);
            } else {
                double hi;
                asm("cvt.f64.bf16 %0, %1;" : "=d"(hi) : "h"(h16));
                if (BITROUTE > 0) {
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

template <int DT, int BITROUTE = BF16_BITROUTE>
__device__ __forceinline__ bool may_hold_nonfinite(const Acc &a) {
    if constexpr (DT == SCOUT_DT_BF16) {
        // non-finite element, or a subnormal one on the bit-placement route
        return !(a.q0 + a.q1 < 1.157920892373162e77) ||                    // 2^256
               (BITROUTE > 0 && a.q1 > 0.0 && a.q1 < 6.525304467998525e-55);  // 2^-180
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
// h * P lets every product be a 32x32+64 multiply-add.  Two spellings of the same
// arithmetic.  From the C++ expression the compiler makes 11 instructions per row; from
// the PTX chain the 7 it needs (one wide multiply and two 32-bit multiply-adds for h * P,
// four wide multiply-adds).  Which one is faster depends on what surrounds it (measured
// in one session, 3 GB to 125 GB per step).  In the kernels compiled for a single element
// type the PTX chain wins (front end 0: fp32 6,905-6,918 -> 7,027-7,034 GB/s, bf16
// 6,352-6,381 -> 6,470-6,490).  In the kernel that reads the type from the tile table it
// depends on the front end: with batches of rows (front end 0) the C++ form wins (int64
// 7,198 against 7,009, uint8 7,194 / 6,990, int32 7,175 / 6,799, fp64 6,883 / 6,803), with
// the register pipeline (front end 1) the PTX chain does (10,000 mixed tensors 7,124 ->
// 7,167-7,178, int32 6,921 -> 6,955, the others equal).  Each kernel uses what measured
// faster for it.
template <bool PTX_CHAIN>
__device__ __forceinline__ void fold_row(uint64_t &h, const uint4 &v, const uint32_t (&m)[4]) {
    if constexpr (PTX_CHAIN) {
        const uint32_t lo = (uint32_t)h, hi = (uint32_t)(h >> 32);
        constexpr uint32_t P_LO = (uint32_t)HASH_P, P_HI = (uint32_t)(HASH_P >> 32);
        uint64_t t;
        uint32_t th;
        asm("mul.wide.u32 %0, %1, %2;" : "=l"(t) : "r"(lo), "r"(P_LO));
        asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(th) : "r"(lo), "r"(P_HI), "r"((uint32_t)(t >> 32)));
        asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(th) : "r"(hi), "r"(P_LO), "r"(th));
        t = ((uint64_t)th << 32) | (uint32_t)t;
        asm("mad.wide.u32 %0, %1, %2, %0;" : "+l"(t) : "r"(m[0]), "r"(v.x));
        asm("mad.wide.u32 %0, %1, %2, %0;" : "+l"(t) : "r"(m[1]), "r"(v.y));
        asm("mad.wide.u32 %0, %1, %2, %0;" : "+l"(t) : "r"(m[2]), "r"(v.z));
        asm("mad.wide.u32 %0, %1, %2, %0;" : "+l"(t) : "r"(m[3]), "r"(v.w));
        h = t;
    } else {
        uint64_t t = h * HASH_P;
        t += (uint64_t)m[0] * v.x;
        t += (uint64_t)m[1] * v.y;
        t += (uint64_t)m[2] * v.z;
        t += (uint64_t)m[3] * v.w;
        h = t;
    }
}

// Per-lane state of one tile's scan: the lane's four slot multipliers, its share
// of the hash recurrence, and its fp64 accumulators.  Rows may be fed from
// registers (direct loads) or from shared memory (bulk-async ring); the
// arithmetic is the same.
template <int DT, bool PTX_CHAIN = false, int BITROUTE = BF16_BITROUTE>
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
    __device__ __forceinline__ void row_hash(const uint4 &v) { fold_row<PTX_CHAIN>(h, v, m); }
    __device__ __forceinline__ void row_stats(const uint4 &v) { stats_fast<DT, BITROUTE>(v, a); }
    __device__ __forceinline__ void row(const uint4 &v) {
        fold_row<PTX_CHAIN>(h, v, m);
        stats_fast<DT, BITROUTE>(v, a);
    }
    // Warp reduction of what the lanes hold: hash share, sums, and whether any lane
    // suspects a non-finite (or, for bf16, subnormal) element.
    __device__ __forceinline__ void reduce(uint64_t &h_out, double &s, double &q, bool &suspect) const {
        q = a.q0 + a.q1;
        if constexpr (DT == SCOUT_DT_BF16 && BITROUTE > 0)
            s = fma(a.s1, 0x1p896, a.s0);  // s1 holds x * 2^-896: exact power-of-two rescale
        else
            s = a.s0 + a.s1;
        suspect = __any_sync(0xFFFFFFFFu, may_hold_nonfinite<DT, BITROUTE>(a));
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
template <int DT, bool PTX_CHAIN = false>
__device__ __forceinline__ void scan_tile(const uint8_t *tile, uint32_t nbytes, uint32_t lane,
                                          TileRec &out) {
    TileScan<DT, PTX_CHAIN> st;
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

// Front end 1 (the default of the staged scan): rotating register pipeline.  PF_ROWS rows
// are always in flight: as soon as a row has been folded its registers are reloaded with
// the row PF_ROWS ahead, so a warp's loads overlap its own arithmetic.  80 registers, three
// CTAs per SM.  Measured against front end 0 in one session (GB/s, whole step): 36 GB of
// fp32 7,039-7,063 -> 7,226-7,236 (the scan kernel at 0.99 of the read probe), 125 GB of bf16
// 6,511-6,521 -> 6,554-6,577, 71 GB of mixed tensors 7,010 -> 7,120-7,143; depths 6, 10, 12
// and 16 rows and 64 or 128 registers were equal or slower.
#ifndef SCOUT_PF_ROWS
#define SCOUT_PF_ROWS 8
#endif
constexpr int PF_ROWS = SCOUT_PF_ROWS;
// spelling of the hash fold in the mixed-type kernel of this front end (see fold_row)
constexpr bool MIXED_PTX_CHAIN = true;
// bf16 elements per word quad that this front end widens by bit placement (see stats_fast).
// With the loads overlapped the conversion pipe is the busiest unit of the bf16 scan (75 %),
// and unloading a quarter of its work for six more instructions per row pays: 125 GB of bf16
// 6,558 (none) / 6,548 (one) / 6,654-6,681 (two) / 6,645 (three).  Front end 0, whose warps
// also have their own load latency to sit out, is fastest with none (6,361 / 6,282 / 6,223 / 6,016).
#ifndef SCOUT_PF_BITROUTE
#define SCOUT_PF_BITROUTE 2
#endif
constexpr int PF_BITROUTE = SCOUT_PF_BITROUTE;
// ... and in the mixed-type kernel of this front end, where none is faster (10,000 mixed
// tensors: 7,172-7,176 with none, 7,118-7,137 with two)
constexpr int MIXED_PF_BITROUTE = 0;

template <int DT, bool PTX_CHAIN = false, int BITROUTE = PF_BITROUTE>
__device__ __forceinline__ void scan_tile_prefetch(const uint8_t *tile, uint32_t nbytes, uint32_t lane,
                                                   TileRec &out) {
    TileScan<DT, PTX_CHAIN, BITROUTE> st;
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
    uint32_t work_streams; // counters the items are dealt from (>= 1)
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
        case SCOUT_DT_F32:  scan_tile_prefetch<SCOUT_DT_F32, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_BF16: scan_tile_prefetch<SCOUT_DT_BF16, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_I64:  scan_tile_prefetch<SCOUT_DT_I64, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_F16:  scan_tile_prefetch<SCOUT_DT_F16, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_F64:  scan_tile_prefetch<SCOUT_DT_F64, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
        case SCOUT_DT_I32:  scan_tile_prefetch<SCOUT_DT_I32, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
        default:            scan_tile_prefetch<SCOUT_DT_U8, MIXED_PTX_CHAIN, MIXED_PF_BITROUTE>(tile, nbytes, lane, rec); break;
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

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

}  // namespace
}  // namespace scout
