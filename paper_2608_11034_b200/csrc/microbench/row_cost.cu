// Compute-only cost of the scan's row routine (TileScan of scout_scan.cuh): the rows
// come from shared memory (one 16-byte load per lane per row, as from global memory in the
// real kernel), so no DRAM traffic is involved, and the kernel runs in the scan's launch
// configuration: 256 threads per CTA, 1, 2 or 4 CTAs per SM (2, 4, 8 warps per scheduler).
// Reported: SM cycles per 512-byte row per scheduler (CUDA-event time at the clock given on
// the command line, default 1965 MHz) and the scan rate that cost would allow if nothing else
// limited it.  Modes: the whole routine, the hash fold alone, the statistics alone.
//
// This is the bound the scan is compared with when it is not limited by HBM: the bf16
// routine needs about 80 cycles per row, which at the 1.65-1.75 GHz the board sustains in
// long launches is 6.3-6.7 TB/s.
#include <cstdio>
#include <cstdlib>

#include "../scout_scan.cuh"
using namespace scout;

static __device__ __forceinline__ uint4 lds16(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

template <int DT, int MODE, bool PTX_CHAIN, int BITROUTE = 0>
__global__ void __launch_bounds__(256, 4) rows(const uint4 *in, TileRec *out, int iters) {
    extern __shared__ __align__(16) uint8_t sm[];
    const uint32_t lane = threadIdx.x & 31u, wib = threadIdx.x >> 5;
    uint4 *mine = reinterpret_cast<uint4 *>(sm) + wib * 256;
    for (int u = 0; u < 8; ++u) mine[u * 32 + lane] = in[(blockIdx.x * 8 + wib) % 64 * 256 + u * 32 + lane];
    __syncthreads();
    const uint32_t base = smem_u32(mine) + 16u * lane;
    TileScan<DT, PTX_CHAIN, BITROUTE> st;
    st.begin(lane);
#pragma unroll 1
    for (int it = 0; it < iters; ++it) {
        uint4 v[8];
        // the address changes with the iteration, so that neither the loads nor anything computed
        // from the loaded words alone can be moved out of the loop
        const uint32_t b = base ^ ((uint32_t)(it & 1) << 4);
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = lds16(b + u * 512);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (MODE == 0) st.row(v[u]);
            if (MODE == 1) st.row_hash(v[u]);
            if (MODE == 2) st.row_stats(v[u]);
        }
    }
    TileRec rec;
    st.finish(reinterpret_cast<const uint8_t *>(in), 0, lane, rec);
    if (lane == 0) out[blockIdx.x * 8 + wib] = rec;
}

static double g_mhz = 1965.0;
static int g_sms = 148;

template <int DT, int MODE, bool PTX_CHAIN, int BITROUTE = 0>
void run(const char *dtype, const uint4 *in, TileRec *out) {
    static const char *mode[3] = {"hash + statistics", "hash only", "statistics only"};
    const int iters = 2000;
    cudaFuncSetAttribute(rows<DT, MODE, PTX_CHAIN, BITROUTE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768);
    for (int per_sm = 1; per_sm <= 4; per_sm *= 2) {
        rows<DT, MODE, PTX_CHAIN, BITROUTE><<<g_sms * per_sm, 256, 32768>>>(in, out, iters);
        cudaDeviceSynchronize();
        cudaEvent_t e0, e1;
        cudaEventCreate(&e0); cudaEventCreate(&e1);
        cudaEventRecord(e0);
        rows<DT, MODE, PTX_CHAIN, BITROUTE><<<g_sms * per_sm, 256, 32768>>>(in, out, iters);
        cudaEventRecord(e1);
        cudaDeviceSynchronize();
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double rows_per_sched = 2.0 * per_sm * iters * 8.0;
        const double cyc = ms * 1e-3 * g_mhz * 1e6 / rows_per_sched;
        printf("%-20s %-18s %d warps/scheduler: %6.2f cycles per row per scheduler -> %6.0f GB/s at %.0f MHz\n", dtype,
               mode[MODE], 2 * per_sm, cyc, 512.0 * 4 * g_sms * g_mhz * 1e6 / cyc / 1e9, g_mhz);
        cudaEventDestroy(e0); cudaEventDestroy(e1);
    }
}

int main(int argc, char **argv) {
    if (argc > 1) g_mhz = atof(argv[1]);
    cudaDeviceGetAttribute(&g_sms, cudaDevAttrMultiProcessorCount, 0);
    uint4 *in;
    TileRec *out;
    if (cudaMalloc(&in, 64 * 4096) != cudaSuccess) { printf("no device\n"); return 1; }
    cudaMalloc(&out, (size_t)g_sms * 4 * 8 * 32);
    // finite bf16 / fp32 patterns with exponents near those of N(0, 0.02) samples
    uint32_t *h = (uint32_t *)malloc(64 * 4096);
    uint32_t x = 12345;
    for (int i = 0; i < 64 * 1024; ++i) {
        x = x * 1664525u + 1013904223u;
        const uint32_t hi = 0x3C000000u | (x & 0x807F0000u) | ((x >> 3) & 0x01800000u);
        const uint32_t lo = 0x3C00u | ((x >> 8) & 0x807Fu) | ((x >> 20) & 0x0180u);
        h[i] = hi | lo;
    }
    cudaMemcpy(in, h, 64 * 4096, cudaMemcpyHostToDevice);
    // the kernels compiled for one element type (fp32, bf16, fp16) use the PTX spelling of the hash
    // fold, the kernel that reads the type from the tile table the C++ one: see fold_row
    // bf16 as the default kernel runs it: two of eight elements widened by bit placement
    run<SCOUT_DT_BF16, 0, true, PF_BITROUTE>("bf16 (2 of 8 placed)", in, out);
    run<SCOUT_DT_BF16, 2, true, PF_BITROUTE>("bf16 (2 of 8 placed)", in, out);
    run<SCOUT_DT_BF16, 0, true>("bf16", in, out); run<SCOUT_DT_BF16, 1, true>("bf16", in, out);
    run<SCOUT_DT_BF16, 2, true>("bf16", in, out);
    run<SCOUT_DT_F32, 0, true>("f32", in, out);   run<SCOUT_DT_F32, 2, true>("f32", in, out);
    run<SCOUT_DT_BF16, 0, false>("bf16 (C++ fold)", in, out); run<SCOUT_DT_F32, 0, false>("f32 (C++ fold)", in, out);
    run<SCOUT_DT_F16, 0, true>("f16", in, out);
    run<SCOUT_DT_I64, 0, false>("i64", in, out);
    run<SCOUT_DT_U8, 0, false>("u8", in, out);
    const cudaError_t e = cudaGetLastError();
    printf("status: %s\n", cudaGetErrorString(e));
    return e != cudaSuccess;
}
