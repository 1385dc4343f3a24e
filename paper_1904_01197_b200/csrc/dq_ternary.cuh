// Radix-3 container for three-level (ternary) DQSG messages: five codes per byte instead of four, 1.6 bits per
// element against the log2(3) = 1.585 of the paper's raw-bit count (Section 4, raw-bits table).  Two small
// transcoding kernels between the 2-bit stream the encode / decode kernels use and the container; they touch
// only the packed data (n/4 + n/5 bytes), not the gradient.
//
//   byte k = t_{5k} + 3 t_{5k+1} + 9 t_{5k+2} + 27 t_{5k+3} + 81 t_{5k+4},   codes past the end counting as 0.
//
// Work unit = 80 codes = five words of the 2-bit stream = sixteen container bytes, so both sides of a unit are
// whole words and no two threads share one.  One thread per unit.
#pragma once

#include "dq_device.cuh"

namespace dq {

constexpr int kTernaryThreads = 256;
constexpr uint32_t kWarnCodeRange = 0x4u;      // DQ_WARN_CODE_RANGE

// The ten bits (five 2-bit codes) that start at bit 10*b of a unit's 160-bit string.
__device__ __forceinline__ uint32_t ten_bits(const uint32_t (&w)[5], int b)
{
    const int bit = 10 * b, wi = bit >> 5, sh = bit & 31;
    uint32_t v = w[wi] >> sh;
    if (sh + 10 > 32) v |= w[wi + 1] << (32 - sh);
    return v & 0x3FFu;
}

__global__ void __launch_bounds__(kTernaryThreads)
ternary_pack_kernel(const uint32_t* __restrict__ packed, uint64_t n, uint8_t* __restrict__ out, uint32_t* status)
{
    grid_dependency_wait();
    grid_dependency_launch_next();
    const uint64_t unit = (uint64_t)blockIdx.x * kTernaryThreads + threadIdx.x;
    if (unit * 80u >= n) return;
    const uint64_t num_words = (n + 15u) >> 4;
    const uint64_t num_bytes = (n + 4u) / 5u;
    const uint64_t left = n - unit * 80u;                      // codes from the start of this unit to the end
    uint32_t w[5];
    uint32_t bad = 0u;
#pragma unroll
    for (int j = 0; j < 5; ++j) {
        const uint64_t wi = unit * 5u + j;
        uint32_t v = (wi < num_words) ? __ldg(packed + wi) : 0u;
        if (left < 16u * (j + 1)) {                            // codes past the end count as 0
            const uint32_t keep = (left > 16u * j) ? (uint32_t)(left - 16u * j) : 0u;
            v = keep ? (v & (0xFFFFFFFFu >> (32u - 2u * keep))) : 0u;
        }
        const uint32_t three = v & (v >> 1) & 0x55555555u;     // low bit of every code that is 3
        bad |= three;
        w[j] = v ^ three;                                      // a three-level message has no code 3: stored as 2
    }
    if (bad != 0u && status != nullptr) atomicOr(status, kWarnCodeRange);
    uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int b = 0; b < 16; ++b) {
        const uint32_t g = ten_bits(w, b);
        const uint32_t byte = (g & 3u) + 3u * ((g >> 2) & 3u) + 9u * ((g >> 4) & 3u) + 27u * ((g >> 6) & 3u) +
                              81u * (g >> 8);
        o[b >> 2] |= byte << (8 * (b & 3));
    }
    const uint64_t byte0 = unit * 16u;
    if (byte0 + 16u <= num_bytes) {
        reinterpret_cast<uint4*>(out)[unit] = make_uint4(o[0], o[1], o[2], o[3]);
    } else {
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (byte0 + b < num_bytes) out[byte0 + b] = (uint8_t)(o[b >> 2] >> (8 * (b & 3)));
    }
}

__global__ void __launch_bounds__(kTernaryThreads)
ternary_unpack_kernel(const uint8_t* __restrict__ data, uint64_t n, uint32_t* __restrict__ packed)
{
    grid_dependency_wait();
    grid_dependency_launch_next();
    const uint64_t unit = (uint64_t)blockIdx.x * kTernaryThreads + threadIdx.x;
    if (unit * 80u >= n) return;
    const uint64_t num_words = (n + 15u) >> 4;
    const uint64_t num_bytes = (n + 4u) / 5u;
    const uint64_t left = n - unit * 80u;
    const uint64_t byte0 = unit * 16u;
    uint32_t in[4] = {0u, 0u, 0u, 0u};
    if (byte0 + 16u <= num_bytes) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(data) + unit);
        in[0] = v.x; in[1] = v.y; in[2] = v.z; in[3] = v.w;
    } else {
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (byte0 + b < num_bytes) in[b >> 2] |= (uint32_t)__ldg(data + byte0 + b) << (8 * (b & 3));
    }
    uint32_t w[5] = {0u, 0u, 0u, 0u, 0u};
#pragma unroll
    for (int b = 0; b < 16; ++b) {
        uint32_t v = (in[b >> 2] >> (8 * (b & 3))) & 0xFFu;
        uint32_t g = 0u;
#pragma unroll
        for (int q = 0; q < 5; ++q) {                          // code q of the byte = digit q of v in base 3
            g |= (v % 3u) << (2 * q);
            v /= 3u;
        }
        const int bit = 10 * b, wi = bit >> 5, sh = bit & 31;
        w[wi] |= g << sh;
        if (sh + 10 > 32) w[wi + 1] |= g >> (32 - sh);
    }
#pragma unroll
    for (int j = 0; j < 5; ++j) {
        const uint64_t wi = unit * 5u + j;
        if (wi >= num_words) break;
        uint32_t v = w[j];
        if (left < 16u * (j + 1)) {                            // pad bits of the last word are written as 0
            const uint32_t keep = (uint32_t)(left - 16u * j);  // >= 1 because wi < num_words
            v &= 0xFFFFFFFFu >> (32u - 2u * keep);
        }
        packed[wi] = v;
    }
}

}  // namespace dq
