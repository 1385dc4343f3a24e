// Issue-cost probe for sm_100a: how many scheduler cycles one warp instruction of each class costs, alone and in
// the mixes that the encode and decode kernels are made of (the 32x32->64 multiplies and three-input XORs of
// Philox, the shifts and logic of the bit packing, the fp32 adds and multiply-adds of the quantizer).
//
// One CTA per SM with 16 or 32 warps (4 or 8 per scheduler).  Every thread runs eight independent dependency
// chains; the loop body holds 64 instruction groups, so the loop's own counter, compare and branch are under 2 %
// of the instructions.  fp32 operands are (register, constant, constant), which cannot collide in the register
// file's banks.  A group's cost is the SM clock that the slowest warp of SM 0 needed, divided by the groups one
// scheduler issued.  Stand-alone program (no library code):
//     issue_probe                 every group, 4 and 8 warps per scheduler
//     issue_probe NAME [WARPS]    one group (for a profiler capture of a single kernel)
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cuda_runtime.h>

namespace {

constexpr int kIters = 256;
constexpr int kUnroll = 8;
constexpr int kChains = 8;

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
__device__ __forceinline__ float fmul(float a, float b)
{
    float d;
    asm volatile("mul.rn.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ uint32_t shf(uint32_t lo, uint32_t hi, uint32_t s)
{
    uint32_t d;
    asm volatile("shf.r.wrap.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(lo), "r"(hi), "r"(s));
    return d;
}
__device__ __forceinline__ uint32_t shr(uint32_t a, uint32_t n)
{
    uint32_t d;
    asm volatile("shr.u32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(n));
    return d;
}
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c)      // (a & b) | c
{
    uint32_t d;
    asm volatile("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t imad(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm volatile("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t mulhi(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm volatile("mul.hi.u32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm volatile("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ double dfma(double a, double b, double c)
{
    double d;
    asm volatile("fma.rn.f64 %0, %1, %2, %3;" : "=d"(d) : "d"(a), "d"(b), "d"(c));
    return d;
}

struct State {
    uint32_t a[kChains], b[kChains];
    float f[kChains], g[kChains];
    uint64_t p[kChains];
    double d[kChains];
    uint32_t m0, m1;
    float c;
    uint64_t pc;
    double dc;
};

enum Group : int {
    gFfma, gFadd, gFfma3, gLop3, gShf, gImad, gMulHi, gWide, gFfma2, gDfma,
    gLopF1, gLopF2, gLopF3, gLop2F1, gImadF1, gImadF2, gImadLop,
    gWideF1, gWideF2, gWideF4, gWideA2, gWideM2, gWideF2r, gWideFLF, gWideF2i, gWideL1, gWideL2, gWideL3, gWideL1F2, gWideDfma,
    gRound, gRoundF2, gRoundF4, gRoundF2x2, gRoundL2F4, gEncodeLike, gDecodeLike, gDecCoarse, gDecFine, gEncCoarse, gEncFine, gNumGroups
};

struct GroupInfo { const char* key; const char* name; int instructions; };
const GroupInfo kInfo[gNumGroups] = {
    {"ffma", "fma.rn.f32 (reg, const, const)", 1},
    {"fadd", "add.rn.f32", 1},
    {"ffma3", "fma.rn.f32 with three register sources", 1},
    {"lop3", "lop3 (3-input xor)", 1},
    {"shf", "shf.r (funnel shift)", 1},
    {"imad", "mad.lo.u32", 1},
    {"mulhi", "mul.hi.u32", 1},
    {"wide", "mul.wide.u32", 1},
    {"ffma2", "fma.rn.f32x2", 1},
    {"dfma", "fma.rn.f64", 1},
    {"lop3_f1", "lop3 + 1 ffma", 2},
    {"lop3_f2", "lop3 + 2 ffma", 3},
    {"lop3_f3", "lop3 + 3 ffma", 4},
    {"lop3x2_f1", "2 lop3 + 1 ffma", 3},
    {"imad_f1", "imad + 1 ffma", 2},
    {"imad_f2", "imad + 2 ffma", 3},
    {"imad_lop3", "imad + lop3", 2},
    {"wide_f1", "wide + 1 ffma", 2},
    {"wide_f2", "wide + 2 ffma", 3},
    {"wide_f4", "wide + 4 ffma", 5},
    {"wide_a2", "wide + 2 fadd", 3},
    {"wide_m2", "wide + 2 fmul", 3},
    {"wide_f2r", "wide + 2 ffma with register operands only", 3},
    {"wide_flf", "wide + ffma, lop3, ffma", 4},
    {"wide_f2i", "wide + 2 ffma with an immediate operand", 3},
    {"wide_l1", "wide + 1 lop3", 2},
    {"wide_l2", "wide + 2 lop3", 3},
    {"wide_l3", "wide + 3 lop3", 4},
    {"wide_l1_f2", "wide + 1 lop3 + 2 ffma", 4},
    {"wide_dfma", "wide + dfma", 2},
    {"round", "Philox round: 2 wide + 2 lop3", 4},
    {"round_f2", "round + 2 ffma", 6},
    {"round_f4", "round + 4 ffma", 8},
    {"round_f2x2", "round + 2 ffma2 (four fp32 results)", 6},
    {"round_l2_f4", "round + 2 lop3 + 4 ffma", 10},
    {"encode_like", "9 rounds + 4 x (shr, 2 ffma, fadd, shf): the NDQSG encoder's mix for 4 elements", 56},
    {"decode_like", "9 rounds + 4 x (shr, shf, lop3, 4 ffma, 5 fadd): the NDQSG decoder's mix for 4 elements", 84},
    {"dec_coarse", "decoder mix, 4 blocks in flight: 9 rounds, then the arithmetic of 16 elements", 336},
    {"dec_fine", "decoder mix, 4 blocks in flight: element arithmetic spread between the multiplies", 336},
    {"enc_coarse", "encoder mix, 4 blocks in flight: 9 rounds, then the arithmetic of 16 elements", 224},
    {"enc_fine", "encoder mix, 4 blocks in flight: element arithmetic spread between the multiplies", 224},
};

#define F1 s.f[j] = ffma(s.f[j], c, c)
#define F2 s.g[j] = ffma(s.g[j], c, c)
#define A1 s.f[j] = fadd(s.f[j], c)
#define L1 s.b[j] = xor3(s.b[j], s.m0, s.m0)
#define WIDE_HL wide(s.a[j], s.m0, lo, hi); s.a[j] = hi; s.b[j] = lo
#define WIDE_X wide(s.a[j], s.m0, lo, hi); s.a[j] = xor3(hi, lo, s.m1)
#define ROUND                                                                                                       \
    wide(s.a[j], s.m0, lo, hi); wide(s.b[j], s.m1, lo1, hi1);                                                       \
    s.a[j] = xor3(hi1, lo, s.m0); s.b[j] = xor3(hi, lo1, s.m1)

template <int G>
__device__ __forceinline__ void step(State& s, int j)
{
    uint32_t lo, hi, lo1, hi1;
    const float c = s.c;
    if (G == gFfma) { F1; }
    if (G == gFadd) { A1; }
    if (G == gFfma3) s.f[j] = ffma(s.f[j], c, s.g[j]);
    if (G == gLop3) { L1; }
    if (G == gShf) s.b[j] = shf(s.b[j], s.m0, 3u);
    if (G == gImad) s.b[j] = imad(s.b[j], s.m0, s.m0);
    if (G == gMulHi) s.b[j] = mulhi(s.b[j], s.m0);
    if (G == gWide) { WIDE_HL; }
    if (G == gFfma2) s.p[j] = ffma2(s.p[j], s.pc, s.pc);
    if (G == gDfma) s.d[j] = dfma(s.d[j], s.dc, s.dc);
    if (G == gLopF1) { L1; F1; }
    if (G == gLopF2) { L1; F1; F2; }
    if (G == gLopF3) { L1; F1; F2; F1; }
    if (G == gLop2F1) { L1; F1; s.a[j] = xor3(s.a[j], s.m1, s.m1); }
    if (G == gImadF1) { s.b[j] = imad(s.b[j], s.m0, s.m0); F1; }
    if (G == gImadF2) { s.b[j] = imad(s.b[j], s.m0, s.m0); F1; F2; }
    if (G == gImadLop) { s.b[j] = imad(s.b[j], s.m0, s.m0); s.a[j] = xor3(s.a[j], s.m1, s.m1); }
    if (G == gWideF1) { WIDE_HL; F1; }
    if (G == gWideF2) { WIDE_HL; F1; F2; }
    if (G == gWideF4) { WIDE_HL; F1; F2; F1; F2; }
    if (G == gWideA2) { WIDE_HL; s.f[j] = fadd(s.f[j], c); s.g[j] = fadd(s.g[j], c); }
    if (G == gWideM2) { WIDE_HL; s.f[j] = fmul(s.f[j], c); s.g[j] = fmul(s.g[j], c); }
    if (G == gWideF2r) { WIDE_HL; s.f[j] = ffma(s.f[j], s.g[j], s.g[j]); s.g[j] = ffma(s.g[j], s.f[j], s.f[j]); }
    if (G == gWideFLF) { wide(s.a[j], s.m0, lo, hi); s.a[j] = hi; F1; s.b[j] = xor3(s.b[j], lo, s.m0); F2; }
    if (G == gWideF2i) {
        WIDE_HL;
        asm volatile("fma.rn.f32 %0, %0, 0f3F800001, 0f33800000;" : "+f"(s.f[j]));
        asm volatile("fma.rn.f32 %0, %0, 0f3F800001, 0f33800000;" : "+f"(s.g[j]));
    }
    if (G == gWideL1) { WIDE_X; }
    if (G == gWideL2) { WIDE_X; L1; }
    if (G == gWideL3) { WIDE_X; L1; L1; }
    if (G == gWideL1F2) { WIDE_X; F1; F2; }
    if (G == gWideDfma) { WIDE_HL; s.d[j] = dfma(s.d[j], s.dc, s.dc); }
    if (G == gRound) { ROUND; }
    if (G == gRoundF2) { ROUND; F1; F2; }
    if (G == gRoundF4) { ROUND; F1; F2; F1; F2; }
    if (G == gRoundF2x2) { ROUND; s.p[j] = ffma2(s.p[j], s.pc, s.pc); s.p[j] = ffma2(s.p[j], s.pc, s.pc); }
    if (G == gRoundL2F4) { ROUND; F1; s.a[j] = xor3(s.a[j], s.m1, s.m1); F2; F1; s.b[j] = xor3(s.b[j], s.m1, s.m1); F2; }
    if (G == gEncodeLike || G == gDecodeLike) {
        // A Philox block is 18 wide multiplies (nine rounds' worth) and yields four dither values: nine rounds
        // interleaved with the arithmetic of four elements
#pragma unroll
        for (int r = 0; r < 9; ++r) {
            ROUND;
#pragma unroll
            for (int e = 0; e < ((r & 1) && r < 8 ? 1 : 0); ++e) {
                // dither: shift + multiply-add on the bit pattern
                s.g[j] = ffma(__uint_as_float(shr(s.b[j], 10u)), c, s.g[j]);
                if (G == gEncodeLike) {
                    F1; A1;
                    s.a[j] = shf(s.a[j], __float_as_uint(s.f[j]), 2u);
                } else {
                    const uint32_t u = and_or(shf(s.a[j], s.m1, 7u), 0x007FFFFFu, 0x3F800000u);
                    s.f[j] = fadd(s.f[j], __uint_as_float(u));
                    A1; F1; F2; A1; F1; A1; A1;
                }
            }
        }
    }
}

// One instruction of an element's arithmetic (position k in the per-element list), on chain j's fp32 registers.
// Decoder (12): shr, ffma (dither); shf, lop3, fadd (unpack); fadd, ffma, ffma, fadd, ffma, fadd, fadd.
// Encoder (5): shr, ffma (dither); ffma, fadd (quantize); shf (pack).
template <bool DEC>
__device__ __forceinline__ void elem_instr(State& s, int j, int k, uint32_t& t)
{
    const float c = s.c;
    if (DEC) {
        switch (k) {
            case 0: t = shr(s.b[j], 10u); break;
            case 1: s.g[j] = ffma(__uint_as_float(t), c, s.g[j]); break;
            case 2: t = shf(s.a[j], s.m1, 7u); break;
            case 3: t = and_or(t, 0x007FFFFFu, 0x3F800000u); break;
            case 4: s.f[j] = fadd(s.f[j], __uint_as_float(t)); break;
            case 5: case 8: case 10: case 11: s.f[j] = fadd(s.f[j], c); break;
            default: s.f[j] = ffma(s.f[j], c, c); break;
        }
    } else {
        switch (k) {
            case 0: t = shr(s.b[j], 10u); break;
            case 1: s.g[j] = ffma(__uint_as_float(t), c, s.g[j]); break;
            case 2: s.f[j] = ffma(s.f[j], c, c); break;
            case 3: s.f[j] = fadd(s.f[j], c); break;
            default: s.p[j] = shf((uint32_t)s.p[j], __float_as_uint(s.f[j]), 2u); break;
        }
    }
}

// Four Philox blocks in flight (chains 0..3), as in the kernels: nine rounds with the chains innermost, and the
// arithmetic of the 16 elements either after the rounds (FINE = false) or spread between the multiplies.
template <bool DEC, bool FINE>
__device__ __forceinline__ void kernel_like(State& s)
{
    constexpr int kPerElem = DEC ? 12 : 5;
    constexpr int kTotal = 4 * kPerElem;               // per chain: four elements
    uint32_t t[4] = {0u, 0u, 0u, 0u};
    int done[4] = {0, 0, 0, 0};
#pragma unroll
    for (int r = 0; r < 9; ++r) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t lo, hi, lo1, hi1;
            const int want = FINE ? (kTotal * (r + 1)) / 9 : 0;      // element instructions issued by the end of round r
            wide(s.a[j], s.m0, lo, hi);
            if (FINE) {
#pragma unroll
                for (int q = 0; q < 3; ++q)
                    if (done[j] < want - (want - (kTotal * r) / 9) / 2) { elem_instr<DEC>(s, j, done[j] % kPerElem, t[j]); ++done[j]; }
            }
            wide(s.b[j], s.m1, lo1, hi1);
            if (FINE) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (done[j] < want) { elem_instr<DEC>(s, j, done[j] % kPerElem, t[j]); ++done[j]; }
            }
            s.a[j] = xor3(hi1, lo, s.m0);
            s.b[j] = xor3(hi, lo1, s.m1);
        }
    }
    if (!FINE) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
#pragma unroll
            for (int k = 0; k < kPerElem; ++k) {
#pragma unroll
                for (int j = 0; j < 4; ++j) elem_instr<DEC>(s, j, k, t[j]);
            }
        }
    }
}

template <int G>
__global__ void __launch_bounds__(1024) probe(uint32_t* sink, long long* cycles, uint32_t seed, float fs)
{
    State s;
#pragma unroll
    for (int j = 0; j < kChains; ++j) {
        s.a[j] = seed + threadIdx.x * 7u + j;
        s.b[j] = seed ^ (j * 0x9E3779B9u);
        s.f[j] = fs + j;
        s.g[j] = fs * j;
        s.p[j] = ((uint64_t)__float_as_uint(fs + j) << 32) | __float_as_uint(fs * j);
        s.d[j] = (double)fs + j;
    }
    s.m0 = 0xD2511F53u ^ (seed >> 31);
    s.m1 = 0xCD9E8D57u ^ (seed >> 31);
    s.c = fs;
    s.pc = ((uint64_t)__float_as_uint(fs) << 32) | __float_as_uint(fs);
    s.dc = (double)fs;
    __shared__ unsigned long long slowest;
    if (threadIdx.x == 0) slowest = 0ull;
    __syncthreads();
    constexpr bool kWhole = (G >= gDecCoarse);        // one group works on all its chains itself
    constexpr int kBody = (G == gEncodeLike || G == gDecodeLike || kWhole) ? 1 : kUnroll;
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int u = 0; u < kBody; ++u) {
            if (kWhole) {
                if (G == gDecCoarse) kernel_like<true, false>(s);
                if (G == gDecFine) kernel_like<true, true>(s);
                if (G == gEncCoarse) kernel_like<false, false>(s);
                if (G == gEncFine) kernel_like<false, true>(s);
            } else {
#pragma unroll
                for (int j = 0; j < kChains; ++j) step<G>(s, j);
            }
        }
    }
    const long long t1 = clock64();
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < kChains; ++j)
        acc ^= s.a[j] ^ s.b[j] ^ __float_as_uint(s.f[j]) ^ __float_as_uint(s.g[j]) ^ (uint32_t)s.p[j] ^
               (uint32_t)(s.p[j] >> 32) ^ (uint32_t)__double_as_longlong(s.d[j]);
    sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
    if ((threadIdx.x & 31) == 0) atomicMax(&slowest, (unsigned long long)(t1 - t0));
    __syncthreads();
    if (threadIdx.x == 0 && blockIdx.x == 0) *cycles = (long long)slowest;
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
    const int body = (G == gEncodeLike || G == gDecodeLike || G >= gDecCoarse) ? 1 : kUnroll;
    const int chains = (G >= gDecCoarse) ? 1 : kChains;
    const double per_group = (double)c / ((double)kIters * body * chains * warps_per_scheduler);
    printf("%-12s %-86s %d warps/scheduler %3d instr %7.2f cycles/group %5.2f cycles/instr\n", kInfo[G].key,
           kInfo[G].name, warps_per_scheduler, kInfo[G].instructions, per_group, per_group / kInfo[G].instructions);
    fflush(stdout);
    return true;
}

template <int G>
bool run_matching(const char* key, int threads, int sms, uint32_t* sink, long long* cycles)
{
    bool ok = true;
    if (key == nullptr || strcmp(key, kInfo[G].key) == 0) ok = run_group<G>(threads, sms, sink, cycles);
    if constexpr (G + 1 < gNumGroups) return ok && run_matching<G + 1>(key, threads, sms, sink, cycles);
    return ok;
}

}  // namespace

int main(int argc, char** argv)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        fprintf(stderr, "no CUDA device\n");
        return 1;
    }
    const char* key = (argc > 1) ? argv[1] : nullptr;
    const int only_warps = (argc > 2) ? atoi(argv[2]) : 0;
    uint32_t* sink = nullptr;
    long long* cycles = nullptr;
    if (cudaMalloc(&sink, (size_t)sms * 1024 * sizeof(uint32_t)) != cudaSuccess ||
        cudaMalloc(&cycles, sizeof(long long)) != cudaSuccess) {
        fprintf(stderr, "allocation failed\n");
        return 1;
    }
    bool ok = true;
    for (int threads : {512, 1024}) {
        if (only_warps != 0 && threads != only_warps * 128) continue;
        ok = ok && run_matching<0>(key, threads, sms, sink, cycles);
    }
    cudaFree(sink);
    cudaFree(cycles);
    if (!ok) { fprintf(stderr, "CUDA error: %s\n", cudaGetErrorString(cudaGetLastError())); return 1; }
    return 0;
}
