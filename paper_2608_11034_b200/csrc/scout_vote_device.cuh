// Exact consensus on one chunk by one warp (Sec. 5.3; Algorithm 1, Exact branch),
// shared by the stand-alone vote kernel and by the one-launch certify kernel.
#pragma once

#include "scout_internal.h"

namespace scout {

// Lane j holds e_j in e0 and e_{j+32} in e1 (R <= 64).  cnt_j = #{i : e_i = e_j};
// c* = max cnt.  2 c* <= R: Inconclusive, bitmap 0.  Otherwise e* is the unique
// value with count c* and bit j = 1{e_j != e*}.  Writes the chunk's status, bitmap
// and majority hash, appends its outlier pairs (one atomic per warp) or its id to
// the undecided list, and returns the status; every lane returns the same values.
__device__ __forceinline__ uint32_t vote_chunk(uint32_t R, uint64_t c, uint64_t e0, uint64_t e1,
                                               uint32_t lane, const VoteSinks &o, uint64_t &bitmap,
                                               uint64_t &majority) {
    const bool have0 = lane < R, have1 = lane + 32u < R;
    uint32_t cnt0 = 0, cnt1 = 0;
    for (uint32_t i = 0; i < R; ++i) {
        const uint64_t lo = __shfl_sync(0xFFFFFFFFu, e0, i & 31u);
        const uint64_t hi = __shfl_sync(0xFFFFFFFFu, e1, i & 31u);
        const uint64_t ei = i < 32u ? lo : hi;
        cnt0 += (ei == e0);
        cnt1 += (ei == e1);
    }
    if (!have0) cnt0 = 0;
    if (!have1) cnt1 = 0;
    const uint32_t mine = cnt0 > cnt1 ? cnt0 : cnt1;
    const uint32_t best = __reduce_max_sync(0xFFFFFFFFu, mine);

    bitmap = 0;
    majority = 0;
    uint32_t st;
    if (2u * best <= R) {
        st = SCOUT_INCONCLUSIVE;
    } else {
        // the lanes holding e* (count == best) agree on one value
        const uint32_t holders = __ballot_sync(0xFFFFFFFFu, cnt0 == best);
        const uint32_t holders_hi = __ballot_sync(0xFFFFFFFFu, cnt1 == best);
        if (holders) majority = __shfl_sync(0xFFFFFFFFu, e0, __ffs(holders) - 1);
        else         majority = __shfl_sync(0xFFFFFFFFu, e1, __ffs(holders_hi) - 1);
        const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, have0 && e0 != majority);
        const uint32_t b1 = __ballot_sync(0xFFFFFFFFu, have1 && e1 != majority);
        bitmap = ((uint64_t)b1 << 32) | b0;
        st = bitmap ? SCOUT_ATTRIBUTED : SCOUT_AGREE;
    }
    if (lane == 0) {
        if (o.status) o.status[c] = (uint8_t)st;
        if (o.bitmap) o.bitmap[c] = bitmap;
        if (o.majority) o.majority[c] = majority;
    }
    if (bitmap) {  // warp-aggregated append of (chunk, replica) pairs
        const uint32_t n = __popcll(bitmap);
        unsigned long long base = 0;
        if (lane == 0) base = atomicAdd((unsigned long long *)&o.counts[4], (unsigned long long)n);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        const uint32_t b0 = (uint32_t)bitmap, b1 = (uint32_t)(bitmap >> 32);
        const uint32_t below = (1u << lane) - 1u;
        if ((b0 >> lane) & 1u) {
            const uint64_t pos = base + __popc(b0 & below);
            if (pos < o.outlier_cap) o.outliers[pos] = scout_outlier_t{c, lane, 0u};
        }
        if ((b1 >> lane) & 1u) {
            const uint64_t pos = base + __popc(b0) + __popc(b1 & below);
            if (pos < o.outlier_cap) o.outliers[pos] = scout_outlier_t{c, lane + 32u, 0u};
        }
        if (o.cert && lane == 0) {
            uint64_t b = bitmap;
            while (b) {
                const int j = __ffsll((long long)b) - 1;
                atomicAdd((unsigned long long *)&o.cert->replica_bad[j], 1ull);
                b &= b - 1;
            }
        }
    }
    if (st == SCOUT_INCONCLUSIVE && lane == 0) {
        const unsigned long long pos = atomicAdd((unsigned long long *)&o.counts[5], 1ull);
        if (pos < o.undecided_cap) o.undecided[pos] = c;
    }
    return st;
}

}  // namespace scout
