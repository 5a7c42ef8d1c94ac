// Instruction issue rates of one B200 SM sub-partition, measured the way the scan kernel
// runs: 4 CTAs of 256 threads per SM (8 warps per scheduler), every SM busy.
//
// Each test repeats a group of independent instructions (one of each selected kind, four
// independent chains per kind) and reports the device time per group per scheduler in SM
// cycles at the clock given on the command line (default 1965 MHz, the maximum of this part).
// The time comes from CUDA events around the kernel; a clock64() read in one warp would
// measure that warp only, and the scheduler favours the oldest warp.
//
// What the numbers say (B200, 1965 MHz): a warp instruction on the integer, fp64 or
// integer-multiply pipe takes 2.04 cycles of its pipe; two different pipes do not overlap
// fully (lop3 + dadd 3.5 instead of 2.04 per pair); a conversion to fp64 takes about 8.5.
// The scan's row routine is made of exactly these instructions, which is why its cost per
// 512-byte row is close to 1.6 cycles times its instruction count (see row_cost.cu).
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <cuda_runtime.h>

constexpr int ITER = 4000, GROUPS = 32;
enum : int { LOP3 = 1, DADD = 2, IMAD = 4, CVT = 8, FFMA = 16, MADWIDE = 32, SHF = 64, DFMA = 128, MUL64 = 256 };

template <int MASK>
__global__ void __launch_bounds__(256, 4) mix(uint32_t *out, uint32_t seed) {
    uint32_t a[4], b[4], c[4], e[4];
    double d[4], g[4], x[4];
    uint64_t q[4], h[4];
    float f[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        a[i] = seed * (threadIdx.x + 1) + i; b[i] = a[i] * 3; c[i] = a[i] * 5; e[i] = a[i] * 7;
        d[i] = 1.0 + i; g[i] = 2.0 + i; x[i] = 0.5; q[i] = a[i]; h[i] = b[i]; f[i] = 1.0f + i;
    }
#pragma unroll 1
    for (int it = 0; it < ITER; ++it) {
#pragma unroll
        for (int jj = 0; jj < GROUPS; ++jj) {
            const int i = jj & 3;
            if (MASK & LOP3) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a[i]) : "r"(a[(i + 1) & 3]), "r"(a[(i + 2) & 3]));
            if (MASK & DADD) asm volatile("add.f64 %0, %0, %1;" : "+d"(d[i]) : "d"(d[(i + 1) & 3]));
            if (MASK & IMAD) asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(b[i]) : "r"(b[(i + 1) & 3]), "r"(b[(i + 2) & 3]));
            if (MASK & CVT) {  // the converted value feeds an fp64 add, as in the scan
                double t;
                c[i] += 0x10001u;
                asm volatile("cvt.f64.bf16 %0, %1;" : "=d"(t) : "h"((uint16_t)c[i]));
                asm volatile("add.f64 %0, %0, %1;" : "+d"(x[i]) : "d"(t));
            }
            if (MASK & FFMA) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[i]) : "f"(f[(i + 1) & 3]), "f"(f[(i + 2) & 3]));
            if (MASK & MADWIDE) { e[i] += 0x9E3779B9u; asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(q[i]) : "r"(e[i]), "r"(e[(i + 1) & 3])); }
            if (MASK & SHF) asm volatile("shf.r.clamp.b32 %0, %0, %1, 3;" : "+r"(c[i]) : "r"(c[(i + 1) & 3]));
            if (MASK & DFMA) asm volatile("fma.rn.f64 %0, %1, %1, %0;" : "+d"(g[i]) : "d"(g[(i + 1) & 3]));
            if (MASK & MUL64) h[i] = h[i] * 0x9E3779B97F4A7C15ull + q[(i + 1) & 3];
        }
    }
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        r ^= a[i] ^ b[i] ^ c[i] ^ e[i] ^ (uint32_t)__double2hiint(d[i]) ^ (uint32_t)__double2hiint(g[i]) ^
             (uint32_t)__double2hiint(x[i]) ^ (uint32_t)q[i] ^ (uint32_t)(h[i] >> 32) ^ __float_as_uint(f[i]);
    out[blockIdx.x * blockDim.x + threadIdx.x] = r;
}

static double g_mhz = 1965.0;
static int g_sms = 148;

template <int MASK>
void run(const char *name, int n_instr, uint32_t *out) {
    mix<MASK><<<g_sms * 4, 256>>>(out, 7);
    cudaDeviceSynchronize();
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    cudaEventRecord(e0);
    mix<MASK><<<g_sms * 4, 256>>>(out, 7);
    cudaEventRecord(e1);
    cudaDeviceSynchronize();
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    const double per_group = ms * 1e-3 * g_mhz * 1e6 / (ITER * (double)GROUPS * 8.0);
    printf("%-40s %6.2f cycles per group per scheduler = %5.2f per instruction (%d in the group)\n", name, per_group,
           per_group / n_instr, n_instr);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
}

int main(int argc, char **argv) {
    if (argc > 1) g_mhz = atof(argv[1]);
    cudaDeviceGetAttribute(&g_sms, cudaDevAttrMultiProcessorCount, 0);
    uint32_t *out;
    if (cudaMalloc(&out, (size_t)g_sms * 4 * 256 * 4) != cudaSuccess) { printf("no device\n"); return 1; }
    printf("SMs %d, assumed SM clock %.0f MHz\n", g_sms, g_mhz);
    run<LOP3>("lop3", 1, out);
    run<SHF>("shf", 1, out);
    run<IMAD>("mad.lo.u32", 1, out);
    run<MADWIDE>("add.u32 + mad.wide.u32 (64-bit acc.)", 2, out);
    run<MUL64>("u64 * const + u64", 1, out);
    run<FFMA>("fma.f32", 1, out);
    run<DADD>("add.f64", 1, out);
    run<DFMA>("fma.f64", 1, out);
    run<CVT>("add.u32 + cvt.f64.bf16 + add.f64", 3, out);
    run<LOP3 | SHF>("lop3 + shf (same pipe)", 2, out);
    run<DADD | DFMA>("add.f64 + fma.f64 (same pipe)", 2, out);
    run<LOP3 | DADD>("lop3 + add.f64", 2, out);
    run<LOP3 | IMAD>("lop3 + mad.lo", 2, out);
    run<DADD | IMAD>("add.f64 + mad.lo", 2, out);
    run<FFMA | LOP3>("fma.f32 + lop3", 2, out);
    run<FFMA | DADD>("fma.f32 + add.f64", 2, out);
    run<LOP3 | DADD | IMAD>("lop3 + add.f64 + mad.lo", 3, out);
    run<LOP3 | DADD | IMAD | FFMA>("lop3 + add.f64 + mad.lo + fma.f32", 4, out);
    run<CVT | LOP3>("cvt group + lop3", 4, out);
    run<CVT | DFMA | MADWIDE>("cvt group + fma.f64 + mad.wide group", 6, out);
    const cudaError_t e = cudaGetLastError();
    printf("status: %s\n", cudaGetErrorString(e));
    return e != cudaSuccess;
}
