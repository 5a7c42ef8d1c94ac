/*
 * scout_timing.h - statistical consensus of C3 (Sec. 5.4; Algorithm 1,
 * Statistical branch) for timing evidence, on the device.
 *
 * For every peer group g with timings tau_0..tau_{N-1}: m = median, d =
 * RobustScale; d = 0 (all timings identical) gives Agree with a zero bitmap;
 * otherwise bit j = 1{|tau_j - m| > kappa * d} and the status is Attributed if
 * any bit is set, else Agree (this branch never returns Inconclusive).
 *
 * The paper fixes the structure of RobustScale (median absolute deviation, then
 * the interquartile range, then a scaled observed range whenever the previous
 * estimate is zero) but not its constants.  This library's reading:
 *   median   even N: (x[N/2-1] + x[N/2]) * 0.5 of the sorted values
 *   MAD      median_i |tau_i - m|, unscaled
 *   IQR      Q(0.75) - Q(0.25), Q(p) = x[k] + (h - k) * (x[k+1] - x[k]) with
 *            h = (N-1) p, k = floor(h) (linear interpolation of order statistics)
 *   range    (max - min) / N
 * All arithmetic is IEEE fp64 without fused multiply-add, in exactly this order,
 * so results are bit-identical to a plain fp64 evaluation of the same formulas.
 * Timings must be finite.
 */
#ifndef SCOUT_TIMING_H
#define SCOUT_TIMING_H

#include "scout.h"

#ifdef __cplusplus
extern "C" {
#endif

/*   N         peers per group, 2..64
 *   G         number of groups
 *   d_times   device [G][N] doubles
 *   kappa     sensitivity multiplier, > 0 (how many units of dispersion a timing
 *             may deviate from the median)
 *   d_status  device [G] (SCOUT_AGREE or SCOUT_ATTRIBUTED); d_bitmap device [G];
 *   d_median, d_scale  device [G], either may be NULL
 * Asynchronous on `stream`. */
SCOUT_API int scout_consensus_timing(uint32_t N, uint64_t G, const double *d_times, double kappa,
                                     uint8_t *d_status, uint64_t *d_bitmap, double *d_median,
                                     double *d_scale, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SCOUT_TIMING_H */
