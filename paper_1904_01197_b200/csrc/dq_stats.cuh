// Histogram of the codes of a packed message: the input of the paper's rate accounting (entropy of the index
// stream, Section 4, tables of raw and entropy-coded bits).  Not on the hot path; one pass over the packed words.
#pragma once

#include "dq_device.cuh"

namespace dq {

constexpr int kHistThreads = 256;

// Each warp counts into its own 256-bin histogram in shared memory (no contention between warps); the CTA's
// histograms are added to the global one at the end.  A thread handles one row (32 codes, `bits` words) at a time.
__global__ void __launch_bounds__(kHistThreads)
code_histogram_kernel(const uint32_t* __restrict__ packed, uint64_t n, uint32_t bits, unsigned long long* hist)
{
    __shared__ uint32_t bins[kHistThreads / 32][256];
    grid_dependency_wait();
    grid_dependency_launch_next();
    const uint32_t warp = threadIdx.x >> 5;
    for (uint32_t i = threadIdx.x; i < (kHistThreads / 32) * 256u; i += kHistThreads) (&bins[0][0])[i] = 0u;
    __syncthreads();

    const uint64_t rows = (n + 31u) >> 5;
    const uint64_t num_words = (n * bits + 31u) >> 5;
    const uint32_t mask = (1u << bits) - 1u;
    for (uint64_t row = (uint64_t)blockIdx.x * kHistThreads + threadIdx.x; row < rows;
         row += (uint64_t)gridDim.x * kHistThreads) {
        const uint32_t valid = (row * 32u + 32u <= n) ? 32u : (uint32_t)(n - row * 32u);
        const uint64_t w0 = row * bits;
        uint32_t lo = __ldg(packed + w0);
        uint32_t next_word = 1u;
        uint32_t have = 32u;                                     // unread bits left in `lo`
        for (uint32_t e = 0; e < valid; ++e) {
            uint32_t code = lo;
            if (have < bits) {                                   // the code straddles into the next word
                const uint32_t hi = (w0 + next_word < num_words) ? __ldg(packed + w0 + next_word) : 0u;
                ++next_word;
                code |= hi << have;
                lo = hi >> (bits - have);
                have += 32u - bits;
            } else {
                lo = (bits < 32u) ? (lo >> bits) : 0u;
                have -= bits;
            }
            atomicAdd(&bins[warp][code & mask], 1u);
        }
    }
    __syncthreads();
    for (uint32_t b = threadIdx.x; b <= mask; b += kHistThreads) {
        unsigned long long s = 0ull;
#pragma unroll
        for (int w = 0; w < kHistThreads / 32; ++w) s += bins[w][b];
        if (s) atomicAdd(hist + b, s);
    }
}

}  // namespace dq
