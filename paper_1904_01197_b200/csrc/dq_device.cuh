// Device-side building blocks shared by the encode and decode kernels: the Philox4x32-10 dither stream,
// the bit-pattern tricks that replace int<->float conversions, and the asynchronous tile copy (TMA)
// wrappers.  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dq {

// ---------------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  The ten round keys (key + r * Weyl constant) are computed on the
// host and travel as kernel parameters, so the logic ops read them straight from the constant bank.
// ---------------------------------------------------------------------------------------------------
constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

struct PhiloxStream {
    uint32_t rk[10][2];   // round keys
    uint32_t c1, c2, c3;  // counter words 1..3: worker, lo32(step), hi32(step)
    // Only counter word 0 differs between blocks, so parts of rounds 0..2 are the same for every block of a
    // (seed, worker, step) stream; the host folds them into four words:
    uint32_t v0;          // c3 ^ rk[0][1]
    uint32_t v1;          // lo(M1*c2) ^ rk[1][0]
    uint32_t v2;          // hi(M0*u0) ^ rk[1][1],  u0 = hi(M1*c2) ^ c1 ^ rk[0][0]
    uint32_t v3;          // lo(M0*u0) ^ rk[2][1]
};

// M0 * j for j = 0..7: the blocks of a row have consecutive counters base + j, and M0 * (base + j) is
// M0 * base + M0 * j without a carry out of 64 bits, so the first multiply of block j takes its counter's offset
// as the 64-bit addend of the multiply-add (an operand from constant memory) instead of an integer add of its own.
static __constant__ uint64_t c_philox_m0j[8] = {
    0ull * kPhiloxM0, 1ull * kPhiloxM0, 2ull * kPhiloxM0, 3ull * kPhiloxM0,
    4ull * kPhiloxM0, 5ull * kPhiloxM0, 6ull * kPhiloxM0, 7ull * kPhiloxM0};

// N blocks at once, rounds outermost, so N independent dependency chains are in flight.
// Counter word 0 of block j is c0[j] = index of its 4-element chunk (element index / 4).
template <int N>
__device__ __forceinline__ void philox4x32_10_xN(const uint32_t (&c0in)[N], const PhiloxStream& ps,
                                                 uint32_t (&out)[N][4])
{
    uint32_t c0[N], c1[N], c2[N], c3[N];
    // round 0: only M0*c0 depends on the block
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * (uint64_t)c0in[j];
        c2[j] = (uint32_t)(p0 >> 32) ^ ps.v0;
        c3[j] = (uint32_t)p0;
    }
    // round 1: c0, c1 are still block-independent
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const uint64_t p1 = (uint64_t)kPhiloxM1 * (uint64_t)c2[j];
        c0[j] = (uint32_t)(p1 >> 32) ^ ps.v1;
        c1[j] = (uint32_t)p1;
        c2[j] = c3[j] ^ ps.v2;
    }
    // round 2: c3 is block-independent (folded into v3)
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * (uint64_t)c0[j];
        const uint64_t p1 = (uint64_t)kPhiloxM1 * (uint64_t)c2[j];
        c0[j] = (uint32_t)(p1 >> 32) ^ c1[j] ^ ps.rk[2][0];
        c1[j] = (uint32_t)p1;
        c2[j] = (uint32_t)(p0 >> 32) ^ ps.v3;
        c3[j] = (uint32_t)p0;
    }
#pragma unroll
    for (int r = 3; r < 10; ++r) {
#pragma unroll
        for (int j = 0; j < N; ++j) {
            const uint64_t p0 = (uint64_t)kPhiloxM0 * (uint64_t)c0[j];
            const uint64_t p1 = (uint64_t)kPhiloxM1 * (uint64_t)c2[j];
            c0[j] = (uint32_t)(p1 >> 32) ^ c1[j] ^ ps.rk[r][0];
            c1[j] = (uint32_t)p1;
            c2[j] = (uint32_t)(p0 >> 32) ^ c3[j] ^ ps.rk[r][1];
            c3[j] = (uint32_t)p0;
        }
    }
#pragma unroll
    for (int j = 0; j < N; ++j) { out[j][0] = c0[j]; out[j][1] = c1[j]; out[j][2] = c2[j]; out[j][3] = c3[j]; }
}

// The same for the N consecutive blocks base + first, ..., base + first + N - 1 of a row (first + N <= 8 and
// base + 7 < 2^32): see c_philox_m0j.
template <int N>
__device__ __forceinline__ void philox4x32_10_row(uint32_t base, int first, const PhiloxStream& ps,
                                                  uint32_t (&out)[N][4])
{
    uint32_t c0[N], c1[N], c2[N], c3[N];
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * (uint64_t)base + c_philox_m0j[first + j];
        c2[j] = (uint32_t)(p0 >> 32) ^ ps.v0;
        c3[j] = (uint32_t)p0;
    }
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const uint64_t p1 = (uint64_t)kPhiloxM1 * (uint64_t)c2[j];
        c0[j] = (uint32_t)(p1 >> 32) ^ ps.v1;
        c1[j] = (uint32_t)p1;
        c2[j] = c3[j] ^ ps.v2;
    }
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * (uint64_t)c0[j];
        const uint64_t p1 = (uint64_t)kPhiloxM1 * (uint64_t)c2[j];
        c0[j] = (uint32_t)(p1 >> 32) ^ c1[j] ^ ps.rk[2][0];
        c1[j] = (uint32_t)p1;
        c2[j] = (uint32_t)(p0 >> 32) ^ ps.v3;
        c3[j] = (uint32_t)p0;
    }
#pragma unroll
    for (int r = 3; r < 10; ++r) {
#pragma unroll
        for (int j = 0; j < N; ++j) {
            const uint64_t p0 = (uint64_t)kPhiloxM0 * (uint64_t)c0[j];
            const uint64_t p1 = (uint64_t)kPhiloxM1 * (uint64_t)c2[j];
            c0[j] = (uint32_t)(p1 >> 32) ^ c1[j] ^ ps.rk[r][0];
            c1[j] = (uint32_t)p1;
            c2[j] = (uint32_t)(p0 >> 32) ^ c3[j] ^ ps.rk[r][1];
            c3[j] = (uint32_t)p0;
        }
    }
#pragma unroll
    for (int j = 0; j < N; ++j) { out[j][0] = c0[j]; out[j][1] = c1[j]; out[j][2] = c2[j]; out[j][3] = c3[j]; }
}

// One block (reference form, all ten rounds written out).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, const PhiloxStream& ps, uint32_t (&out)[4])
{
    const uint32_t in[1] = {c0};
    uint32_t o[1][4];
    philox4x32_10_xN<1>(in, ps, o);
    out[0] = o[0][0]; out[1] = o[0][1]; out[2] = o[0][2]; out[3] = o[0][3];
}

// Dither values without an integer-to-float conversion and with a single integer instruction: the 22 random
// bits j = x >> 10, read as a float, are the subnormal j * 2^-149; one multiply-add scales them by 2^127 and
// adds the offset, and since the result lies on the grid of step 2^-23 it is exact.  (Integer and logic
// instructions cost about twice the issue bandwidth of fp32 ones on this GPU.)
//   f     = 1 + (2j+1) 2^-23              in [1, 2): the dither in fine-step units is f - 1.5
//   delta = (2j+1) 2^-23 - 1/2            the dither itself
constexpr float kTwo127 = 1.7014118346046923e38f;      // 2^127
constexpr float kTwo125 = 4.2535295865117308e37f;      // 2^125

__device__ __forceinline__ float dither_f12(uint32_t x)
{
    return __fmaf_rn(__uint_as_float(x >> 10), kTwo127, 1.00000011920928955078125f);      // 1 + 2^-23
}

__device__ __forceinline__ float dither_delta(uint32_t x)
{
    return __fmaf_rn(__uint_as_float(x >> 10), kTwo127, -0.49999988079071044921875f);     // -(1/2 - 2^-23)
}

// 16-bit stream: half-word h -> f = 1 + (2h+1) 2^-17, delta = (2h+1) 2^-17 - 1/2.  One byte permutation puts
// h into bits 8..23 (the subnormal or small normal number h * 2^-141); the multiply-add scales by 2^125.
__device__ __forceinline__ float half_word_as_small_float(uint32_t word, int high)
{
    return __uint_as_float(__byte_perm(word, 0u, high ? 0x4324u : 0x4104u));
}

__device__ __forceinline__ float dither16_f12(uint32_t word, int high)
{
    return __fmaf_rn(half_word_as_small_float(word, high), kTwo125, 1.00000762939453125f);   // 1 + 2^-17
}

__device__ __forceinline__ float dither16_delta(uint32_t word, int high)
{
    return __fmaf_rn(half_word_as_small_float(word, high), kTwo125, -0.49999237060546875f);  // -(1/2 - 2^-17)
}

// f of element t (0 .. 4*EPB-1) of a group of four Philox blocks; EPB = elements per block (4 or 8).
template <int DITH>
__device__ __forceinline__ float dither_of(const uint32_t (&rnd)[4][4], int t)
{
    if (DITH == 0) return 1.5f;                      // no dither at the receiver (half-dithered decoding)
    if (DITH == 16) return dither16_f12(rnd[t >> 3][(t & 7) >> 1], t & 1);
    return dither_f12(rnd[t >> 2][t & 3]);
}

// The dither itself (encoder side).
template <int DITH>
__device__ __forceinline__ float dither_delta_of(const uint32_t (&rnd)[4][4], int t)
{
    if (DITH == 16) return dither16_delta(rnd[t >> 3][(t & 7) >> 1], t & 1);
    return dither_delta(rnd[t >> 2][t & 3]);
}

// Round-to-nearest-even of |w| < 2^22 by adding 1.5 * 2^23: the integer lands in the low mantissa bits.
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23
constexpr uint32_t kMagicBits = 0x4B400000u;   // bit pattern of kMagic

// ---------------------------------------------------------------------------------------------------
// Asynchronous tile copies (TMA) with an mbarrier, and a bounded wait.
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// Load a [rows x 32 floats] box whose first row is `row0` into shared memory (128-byte swizzle).
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap* tmap, uint32_t bar, int32_t row0)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"((uint64_t)tmap), "r"(bar), "r"(0), "r"(row0)
        : "memory");
}

// Contiguous bulk copy global -> shared memory (both addresses 16-byte aligned, size a multiple of 16 bytes).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Store a [32 rows x 32 floats] box from shared memory (128-byte swizzle) to rows row0.. of the mapped array; rows
// past the array's end are not written.  Completion is tracked by the issuing thread's bulk groups.
__device__ __forceinline__ void tma_store_rows(const CUtensorMap* tmap, uint32_t src, int32_t row0)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"((uint64_t)tmap), "r"(src), "r"(0), "r"(row0)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit_group()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Waits until at most N of this thread's bulk groups still have to read their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// Makes this thread's earlier shared-memory writes visible to the asynchronous copy engine.
__device__ __forceinline__ void fence_proxy_async_shared()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Upper bound, in nanoseconds, that one try may stay suspended in hardware before it reports "not yet".
constexpr uint32_t kWaitHintNs = 2000u;
// A copy that has not landed after this long (by the global nanosecond timer) is given up: a tile copy takes
// microseconds, so 20 ms means that it will never arrive.
constexpr uint64_t kWaitGiveUpNs = 20ull * 1000ull * 1000ull;

__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kWaitHintNs)
        : "memory");
    return ok != 0u;
}

// Waits for phase `parity` of the barrier, but not for ever: after kWaitGiveUpNs (or after a single try when
// `single_try` is set, which callers do once a wait has already run out) it returns false, so a copy that never
// lands cannot hang the kernel.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, bool single_try = false)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (single_try) return false;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > kWaitGiveUpNs) return false;
    }
}

// Named barrier over `threads` threads (a multiple of 32); id 1..15 (0 is __syncthreads).
__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ void prefetch_l1(const void* p)
{
    asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
}

__device__ __forceinline__ void prefetch_l2(const void* p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// Programmatic dependent launch: wait until the previous kernel of the stream has completed and its writes are
// visible (a no-op when the kernel was launched normally), and allow the next kernel to begin launching.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void grid_dependency_launch_next()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

}  // namespace dq
