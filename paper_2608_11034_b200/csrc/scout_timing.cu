// Statistical consensus (Sec. 5.4; Algorithm 1, Statistical branch): one warp per
// peer group, lane j holds tau_j and tau_{j+32}.  Order statistics come from
// ranks (rank_j = number of values before tau_j in the stable sorted order),
// computed with N shuffles; no sorting network, no shared memory.
#include <math_constants.h>

#include "scout_internal.h"
#include "scout_timing.h"

namespace scout {
namespace {

constexpr int TIMING_THREADS = 128;

struct Ranked {
    double v0, v1;     // the lane's two values (+inf in unused slots)
    uint32_t r0, r1;   // their ranks in the stable ascending order
};

// rank of (v, idx): values strictly smaller, or equal with a smaller index
__device__ __forceinline__ void rank_all(Ranked &x, uint32_t N, uint32_t lane) {
    uint32_t r0 = 0, r1 = 0;
    for (uint32_t i = 0; i < N; ++i) {
        const double a = __shfl_sync(0xFFFFFFFFu, x.v0, i & 31u);
        const double b = __shfl_sync(0xFFFFFFFFu, x.v1, i & 31u);
        const double xi = i < 32u ? a : b;
        r0 += (xi < x.v0) || (xi == x.v0 && i < lane);
        r1 += (xi < x.v1) || (xi == x.v1 && i < lane + 32u);
    }
    x.r0 = r0;
    x.r1 = r1;
}

// k-th order statistic (k < N): the one value whose rank is k
__device__ __forceinline__ double select(const Ranked &x, uint32_t k, uint32_t N, uint32_t lane) {
    const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, lane < N && x.r0 == k);
    const uint32_t b1 = __ballot_sync(0xFFFFFFFFu, lane + 32u < N && x.r1 == k);
    const double a = __shfl_sync(0xFFFFFFFFu, x.v0, b0 ? __ffs(b0) - 1 : 0);
    const double b = __shfl_sync(0xFFFFFFFFu, x.v1, b1 ? __ffs(b1) - 1 : 0);
    return b0 ? a : b;
}

__device__ __forceinline__ double median_of(const Ranked &x, uint32_t N, uint32_t lane) {
    const double hi = select(x, N / 2, N, lane);
    if (N & 1u) return hi;
    const double lo = select(x, N / 2 - 1, N, lane);
    return __dmul_rn(__dadd_rn(lo, hi), 0.5);
}

// Q(p) with h = (N-1) p: x[k] + (h - k) (x[k+1] - x[k]); no fused multiply-add
__device__ __forceinline__ double quantile_of(const Ranked &x, double p, uint32_t N, uint32_t lane) {
    const double h = __dmul_rn((double)(N - 1), p);
    const uint32_t k = (uint32_t)floor(h);
    const double xk = select(x, k, N, lane);
    if (k + 1 >= N) return xk;
    const double xk1 = select(x, k + 1, N, lane);
    return __dadd_rn(xk, __dmul_rn(__dsub_rn(h, (double)k), __dsub_rn(xk1, xk)));
}

__global__ void __launch_bounds__(TIMING_THREADS) timing_consensus(uint32_t N, uint64_t G,
                                                                   const double *__restrict__ times,
                                                                   double kappa, uint8_t *status,
                                                                   uint64_t *bitmap, double *median_out,
                                                                   double *scale_out) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warp = (uint64_t)blockIdx.x * (TIMING_THREADS / 32) + (threadIdx.x >> 5);
    const uint64_t n_warps = (uint64_t)gridDim.x * (TIMING_THREADS / 32);
    for (uint64_t g = warp; g < G; g += n_warps) {
        const double *t = times + g * N;
        Ranked x;
        x.v0 = lane < N ? t[lane] : CUDART_INF;
        x.v1 = lane + 32u < N ? t[lane + 32u] : CUDART_INF;
        rank_all(x, N, lane);
        const double m = median_of(x, N, lane);

        // RobustScale: MAD, then the interquartile range, then the scaled range
        Ranked dev;
        dev.v0 = lane < N ? fabs(__dsub_rn(x.v0, m)) : CUDART_INF;
        dev.v1 = lane + 32u < N ? fabs(__dsub_rn(x.v1, m)) : CUDART_INF;
        rank_all(dev, N, lane);
        double d = median_of(dev, N, lane);
        if (d == 0.0) d = __dsub_rn(quantile_of(x, 0.75, N, lane), quantile_of(x, 0.25, N, lane));
        if (d == 0.0)
            d = __ddiv_rn(__dsub_rn(select(x, N - 1, N, lane), select(x, 0, N, lane)), (double)N);

        uint64_t B = 0;
        if (d != 0.0) {
            const double limit = __dmul_rn(kappa, d);
            const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, lane < N && dev.v0 > limit);
            const uint32_t b1 = __ballot_sync(0xFFFFFFFFu, lane + 32u < N && dev.v1 > limit);
            B = ((uint64_t)b1 << 32) | b0;
        }
        if (lane == 0) {
            status[g] = B ? SCOUT_ATTRIBUTED : SCOUT_AGREE;
            bitmap[g] = B;
            if (median_out) median_out[g] = m;
            if (scale_out) scale_out[g] = d;
        }
    }
}

}  // namespace
}  // namespace scout

extern "C" int scout_consensus_timing(uint32_t N, uint64_t G, const double *d_times, double kappa,
                                      uint8_t *d_status, uint64_t *d_bitmap, double *d_median,
                                      double *d_scale, void *stream) {
    using namespace scout;
    if (N < 2) return SCOUT_ERR_INVALID;
    if (N > 64) return SCOUT_ERR_UNSUPPORTED;
    if (!(kappa > 0.0) || !d_status || !d_bitmap || (G && !d_times)) return SCOUT_ERR_INVALID;
    if (G == 0) return SCOUT_OK;
    uint64_t blocks = (G + TIMING_THREADS / 32 - 1) / (TIMING_THREADS / 32);
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    timing_consensus<<<(unsigned)blocks, TIMING_THREADS, 0, (cudaStream_t)stream>>>(
        N, G, d_times, kappa, d_status, d_bitmap, d_median, d_scale);
    SCOUT_CUDA(cudaGetLastError());
    return SCOUT_OK;
}
