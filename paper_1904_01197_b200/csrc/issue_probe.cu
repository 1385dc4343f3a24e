// Issue-cost probe for sm_100a: how many scheduler cycles one warp instruction of each class costs, alone and in
// the mixes that the encode and decode kernels are made of (wide multiplies and three-input XORs of Philox,
// shifts and logic of the bit packing, fp32 adds and multiply-adds of the quantizer).
//
// One CTA per SM, 16 or 32 warps, every thread runs kChains independent dependency chains for kIters iterations
// of one instruction group; a group's cost is the elapsed SM clock divided by the groups a scheduler issued.
// Stand-alone program (no library code): prints one line per group.
#include <cstdint>
#include <cstdio>
#include <cuda_runtime.h>

namespace {

constexpr int kIters = 2048;
constexpr int kChains = 8;

enum Group : int {
    kWide, kMulHi, kMulLo, kMulHiLo, kLop3, kShf, kImad, kFfma, kFadd, kWide2Ffma, kWide4Ffma, kWide3Lop3,
    kLop3Ffma2, kPhiloxRound, kShfLop3Fadd, kShfFfma, kDecodeLike, kNumGroups
};

struct GroupInfo { const char* name; int instructions; };
const GroupInfo kInfo[kNumGroups] = {
    {"mul.wide.u32 + xor", 2}, {"mul.hi.u32 + xor", 2}, {"mul.lo.u32 + xor", 2}, {"mul.hi + mul.lo + xor", 3},
    {"lop3 (3-input xor)", 1}, {"shr", 1}, {"mad.lo.u32", 1}, {"fma.rn.f32", 1}, {"add.rn.f32", 1},
    {"wide + xor + 2 fma", 4}, {"wide + xor + 4 fma", 6}, {"wide + 3 lop3", 4}, {"lop3 + 2 fma", 3},
    {"Philox round: 2 wide + 2 lop3", 4}, {"shr + lop3 + add.f32", 3}, {"shr + fma (subnormal dither)", 2},
    {"wide + 2 lop3 + add.f32 + fma", 5},
};

__device__ __forceinline__ void wide(uint32_t a, uint32_t m, uint32_t& lo, uint32_t& hi)
{
    asm volatile("{.reg .u64 t; mul.wide.u32 t, %2, %3; mov.b64 {%0,%1}, t;}" : "=r"(lo), "=r"(hi) : "r"(a), "r"(m));
}
__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm volatile("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ float ffma(float a, float b, float c)
{
    float d;
    asm volatile("fma.rn.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float fadd(float a, float b)
{
    float d;
    asm volatile("add.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ uint32_t shr(uint32_t a, uint32_t s)
{
    uint32_t d;
    asm volatile("shr.u32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(s));
    return d;
}

template <int G>
__global__ void __launch_bounds__(1024) probe(uint32_t* sink, long long* cycles, uint32_t seed, float fs)
{
    uint32_t a[kChains], b[kChains];
    float f[kChains], g[kChains];
#pragma unroll
    for (int j = 0; j < kChains; ++j) {
        a[j] = seed + threadIdx.x * 7u + j;
        b[j] = seed ^ (j * 0x9E3779B9u);
        f[j] = fs + j;
        g[j] = fs * j;
    }
    const uint32_t m0 = 0xD2511F53u, m1 = 0xCD9E8D57u;
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int j = 0; j < kChains; ++j) {
            uint32_t lo, hi, lo1, hi1;
            if (G == kWide) { wide(a[j], m0, lo, hi); a[j] = hi ^ lo; }
            if (G == kMulHi) { asm volatile("mul.hi.u32 %0, %1, %2;" : "=r"(hi) : "r"(a[j]), "r"(m0)); a[j] = hi ^ b[j]; }
            if (G == kMulLo) { asm volatile("mul.lo.u32 %0, %1, %2;" : "=r"(lo) : "r"(a[j]), "r"(m0)); a[j] = lo ^ b[j]; }
            if (G == kMulHiLo) {
                asm volatile("mul.hi.u32 %0, %1, %2;" : "=r"(hi) : "r"(a[j]), "r"(m0));
                asm volatile("mul.lo.u32 %0, %1, %2;" : "=r"(lo) : "r"(a[j]), "r"(m0));
                a[j] = hi ^ lo;
            }
            if (G == kLop3) a[j] = xor3(a[j], b[j], m0);
            if (G == kShf) a[j] = shr(a[j], 1u) + 0u * b[j];
            if (G == kImad) asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(a[j]) : "r"(a[j]), "r"(m0), "r"(b[j]));
            if (G == kFfma) f[j] = ffma(f[j], fs, g[j]);
            if (G == kFadd) f[j] = fadd(f[j], g[j]);
            if (G == kWide2Ffma || G == kWide4Ffma) {
                wide(a[j], m0, lo, hi); a[j] = hi ^ lo;
                f[j] = ffma(f[j], fs, g[j]); g[j] = ffma(g[j], fs, f[j]);
                if (G == kWide4Ffma) { f[j] = ffma(f[j], fs, g[j]); g[j] = ffma(g[j], fs, f[j]); }
            }
            if (G == kWide3Lop3) {
                wide(a[j], m0, lo, hi);
                a[j] = xor3(hi, lo, m0); b[j] = xor3(b[j], lo, m1); b[j] = xor3(b[j], hi, m1);
            }
            if (G == kLop3Ffma2) { a[j] = xor3(a[j], b[j], m0); f[j] = ffma(f[j], fs, g[j]); g[j] = ffma(g[j], fs, f[j]); }
            if (G == kPhiloxRound) {
                wide(a[j], m0, lo, hi); wide(b[j], m1, lo1, hi1);
                a[j] = xor3(hi1, lo, m0); b[j] = xor3(hi, lo1, m1);
            }
            if (G == kShfLop3Fadd) {
                uint32_t t = shr(a[j], 9u);
                asm volatile("lop3.b32 %0, %1, %2, %3, 0xFE;" : "=r"(t) : "r"(t), "r"(0x3F800001u), "r"(0u));
                f[j] = fadd(f[j], __uint_as_float(t));
                a[j] = __float_as_uint(f[j]);
            }
            if (G == kShfFfma) {
                f[j] = ffma(__uint_as_float(shr(a[j], 10u)), 1.7014118346046923e38f, f[j]);
                a[j] = __float_as_uint(f[j]);
            }
            if (G == kDecodeLike) {
                wide(a[j], m0, lo, hi);
                a[j] = xor3(hi, lo, m0); b[j] = xor3(b[j], lo, m1);
                f[j] = fadd(f[j], g[j]); g[j] = ffma(g[j], fs, f[j]);
            }
        }
    }
    const long long t1 = clock64();
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < kChains; ++j) acc ^= a[j] ^ b[j] ^ __float_as_uint(f[j]) ^ __float_as_uint(g[j]);
    sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
    if (threadIdx.x == 0 && blockIdx.x == 0) *cycles = t1 - t0;
}

template <int G>
bool run_group(int threads, int sms, uint32_t* sink, long long* cycles)
{
    for (int rep = 0; rep < 2; ++rep) {                 // the first launch warms the instruction cache
        probe<G><<<sms, threads>>>(sink, cycles, 1234u, 1.0000001f);
        if (cudaDeviceSynchronize() != cudaSuccess) return false;
    }
    long long c = 0;
    if (cudaMemcpy(&c, cycles, sizeof(c), cudaMemcpyDeviceToHost) != cudaSuccess) return false;
    const int warps_per_scheduler = threads / 32 / 4;
    const double per_group = (double)c / ((double)kIters * kChains * warps_per_scheduler);
    printf("%-34s %2d warps/scheduler  %d instr  %6.2f cycles/group  %5.2f cycles/instr\n", kInfo[G].name,
           warps_per_scheduler, kInfo[G].instructions, per_group, per_group / kInfo[G].instructions);
    return true;
}

template <int G>
bool run_all(int threads, int sms, uint32_t* sink, long long* cycles)
{
    if (!run_group<G>(threads, sms, sink, cycles)) return false;
    if constexpr (G + 1 < kNumGroups) return run_all<G + 1>(threads, sms, sink, cycles);
    return true;
}

}  // namespace

int main()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        fprintf(stderr, "no CUDA device\n");
        return 1;
    }
    uint32_t* sink = nullptr;
    long long* cycles = nullptr;
    if (cudaMalloc(&sink, (size_t)sms * 1024 * sizeof(uint32_t)) != cudaSuccess ||
        cudaMalloc(&cycles, sizeof(long long)) != cudaSuccess) {
        fprintf(stderr, "allocation failed\n");
        return 1;
    }
    printf("issue cost per scheduler, %d SMs, %d chains per thread, %d iterations\n", sms, kChains, kIters);
    bool ok = true;
    for (int threads : {512, 1024}) ok = ok && run_all<0>(threads, sms, sink, cycles);
    cudaFree(sink);
    cudaFree(cycles);
    if (!ok) { fprintf(stderr, "CUDA error: %s\n", cudaGetErrorString(cudaGetLastError())); return 1; }
    return 0;
}
