// Fused decode-and-average kernel (Algorithm 1, server steps; nested decoder equation and Algorithm 2,
// server loop with the side information given as a vector or taken as the running mean).
//
// One lane owns one row = 32 consecutive elements: 32 fp32 accumulators in registers, and per worker
// exactly `bits` packed words.  For every worker (in array order) the lane reloads that worker's words and
// bucket scale, regenerates the 32 dithers (Philox blocks four at a time, so four dependency chains are in
// flight), reconstructs and accumulates; the mean is written at the end.  The packed streams, the side
// information and the output are each touched once in HBM (the side information of a CTA's 128 rows is staged
// in swizzled shared memory and re-read from there per worker, which keeps it out of the register file).
//
// The path is bound by instruction issue, not by HBM: each (element, worker) pair needs a quarter of a
// Philox block (9.25 integer instructions) before any reconstruction arithmetic.
#pragma once

#include "dq_device.cuh"

namespace dq {

enum DecKind : uint32_t { kDecDqsg = 0, kDecNdqsgPow2 = 1, kDecNdqsgPow2Shrink = 2, kDecNdqsgAnyK = 3 };

struct DecWorker {
    const uint32_t* packed;
    const float* scale;
    PhiloxStream ps;
    uint32_t kind;        // DecKind
    uint32_t bits;
    float s;              // DQSG (L-1)/2
    float cconst;         // DQSG: 4194304 + s - 1.5 ; NDQSG: 4194304 - 1.5   (see unpack_half_biased)
    float A;              // NDQSG alpha * M1
    float M1;
    float alpha;
    float one_m_alpha2;   // 1 - alpha*alpha
    float Kf;             // (float)K
    float invK;           // 1/K (exact when K is a power of two)
    float rcp_count;      // running-mean mode: 1 / (number of workers before this one)
};

struct DecodeArgs {
    const float* side;
    float* out;
    uint32_t* status;
    // A call may cover the elements [first, n) of a longer gradient (first a multiple of the bucket size, 0 for a
    // whole gradient).  Rows, elements and buckets are then numbered as in the whole gradient -- which is what the
    // dither counters need -- and every pointer below is the buffer's address minus the range's offset, so that
    // "pointer + global index" lands in the caller's buffer.
    uint64_t n;               // end of the range (element index)
    uint64_t rows;            // ceil(n / 32): end of the range (row index)
    uint64_t first_row;       // first / 32
    uint32_t prefetch_blocks; // distance, in 128-row blocks, of the L2 prefetch (0 = none)
    uint32_t W;
    uint32_t rows_per_bucket; // B / 32
    uint32_t half_bias_bits;  // 0x4A800000 (bit pattern of 2^22), passed in so that it lives in a register
    float Wf;
    float invW;               // 1/W when W is a power of two, else 0
    DecWorker w[64];
};

// Code of element `idx` of a row, returned as the float 2^22 + code/1 ... precisely: the bit pattern of
// 2^22 with the code in mantissa bits 1.., i.e. the value 2^22 + code (floats in [2^22, 2^23) step by 1/2).
// Subtracting a constant then gives code - c exactly.
template <int BITS>
__device__ __forceinline__ float unpack_half_biased(const uint32_t (&words)[BITS], int idx, uint32_t bias_bits)
{
    const int bit = idx * BITS;
    const int wi = bit >> 5;
    const int sh = bit & 31;
    constexpr uint32_t mask2 = ((1u << BITS) - 1u) << 1;
    uint32_t v;
    if (sh + BITS <= 32) {
        v = (sh == 0) ? (words[wi] << 1) : (words[wi] >> (sh - 1));
    } else {
        v = __funnelshift_r(words[wi], words[(wi + 1) % BITS], sh - 1);
    }
    return __uint_as_float((v & mask2) | bias_bits);          // one logic op: (v & immediate) | register
}

// A worker's packed words of one row (bits words, at most 8) and its bucket scale.
__device__ __forceinline__ void load_worker_row(const DecWorker& wk, uint64_t row, uint64_t bucket,
                                                uint32_t (&words)[8], float& kappa)
{
    const uint32_t* src = wk.packed + row * wk.bits;
#pragma unroll
    for (uint32_t j = 0; j < 8; ++j)
        if (j < wk.bits) words[j] = __ldg(src + j);
    kappa = __ldg(wk.scale + bucket);
}

// One worker's contribution to the 32 accumulators of a row.
//   DQSG:  g~ = (kappa/s) ((k - s) - delta); (k - s + 1.5) - f rounds once to the same value.
//   NDQSG: r = (m - delta) - y a;  jj = rint(r / K);  q1^ = m - K jj;  g~ = beta (q1^ - delta) [+ (1-alpha^2) y]
template <int BITS, uint32_t KIND, int DITH, bool RUN>
__device__ __forceinline__ void decode_row(const DecWorker& wk, uint64_t row, const uint32_t (&cur)[8],
                                           float kappa, const float* side_row, float (&acc)[32],
                                           uint32_t* status, uint32_t bias_bits)
{
    uint32_t words[BITS];
#pragma unroll
    for (int j = 0; j < BITS; ++j) words[j] = cur[j];

    if (status != nullptr && !(fabsf(kappa) <= 3.402823466e38f)) atomicOr(status, 0x1u);

    float c, a = 0.0f;
    if (KIND == kDecDqsg) {
        c = __fdiv_rn(kappa, wk.s);
    } else {
        a = (kappa >= 0x1p-100f) ? __fdiv_rn(wk.A, kappa) : 0.0f;
        c = __fdiv_rn(__fmul_rn(wk.alpha, kappa), wk.M1);                 // beta
    }
    constexpr int EPB = (DITH == 16) ? 8 : 4;       // elements per Philox block
    constexpr int PASS = 4 * EPB;                   // elements per group of four blocks
#pragma unroll
    for (int h = 0; h < 32 / PASS; ++h) {
        uint32_t rnd[4][4];
        if (DITH != 0) philox4x32_10_row<4>((uint32_t)row * (32u / EPB), 4 * h, wk.ps, rnd);
#pragma unroll
        for (int q = 0; q < PASS / 4; ++q) {        // four elements at a time (one 16-byte piece of y)
            float y[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (KIND != kDecDqsg && !RUN) {
                // the row's side information sits in shared memory, 16-byte pieces swizzled by (row & 7)
                const uint32_t piece = (uint32_t)((PASS / 4) * h + q) ^ (threadIdx.x & 7u);
                const float4 v = *reinterpret_cast<const float4*>(side_row + 4u * piece);
                y[0] = v.x; y[1] = v.y; y[2] = v.z; y[3] = v.w;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int t = 4 * q + e;
                const int idx = PASS * h + t;
                const float f = dither_of<DITH>(rnd, t);
                const float X = __fadd_rn(unpack_half_biased<BITS>(words, idx, bias_bits), -wk.cconst);
                float gt;
                if (KIND == kDecDqsg) {
                    const float d = __fadd_rn(X, -f);                      // (k - s) - delta
                    gt = __fmul_rn(c, d);
                } else {
                    // side information: the given vector, or (Algorithm 2 as written) the mean of the
                    // reconstructions accumulated so far
                    const float yy = RUN ? __fmul_rn(acc[idx], wk.rcp_count) : y[e];
                    const float r1 = __fadd_rn(X, -f);                     // m - delta
                    const float r = __fmaf_rn(-yy, a, r1);
                    float jj;
                    if (KIND == kDecNdqsgAnyK) {
                        jj = __fadd_rn(__fadd_rn(__fdiv_rn(r, wk.Kf), kMagic), -kMagic);
                    } else {
                        // K is a power of two: r * (1/K) is exact, so one rounding gives rint(r / K)
                        jj = __fadd_rn(__fmaf_rn(r, wk.invK, kMagic), -kMagic);
                    }
                    const float Y = __fmaf_rn(-wk.Kf, jj, X);              // q1^ + 1.5, exact
                    const float d = __fadd_rn(Y, -f);                      // q1^ - delta
                    if (KIND == kDecNdqsgPow2) gt = __fmul_rn(c, d);                          // alpha == 1
                    else if (KIND == kDecNdqsgPow2Shrink) gt = __fmaf_rn(c, d, __fmul_rn(wk.one_m_alpha2, yy));
                    else if (wk.alpha == 1.0f) gt = __fmul_rn(c, d);
                    else gt = __fmaf_rn(c, d, __fmul_rn(wk.one_m_alpha2, yy));
                }
                acc[idx] = __fadd_rn(acc[idx], gt);
            }
        }
    }
}

template <uint32_t KIND, int DITH, bool RUN>
__device__ __forceinline__ void decode_row_bits(const DecWorker& wk, uint64_t row, const uint32_t (&cur)[8],
                                                float kappa, const float* side_row, float (&acc)[32],
                                                uint32_t* status, uint32_t bias_bits)
{
    switch (wk.bits) {
        case 1: decode_row<1, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        case 2: decode_row<2, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        case 3: decode_row<3, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        case 4: decode_row<4, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        case 5: decode_row<5, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        case 6: decode_row<6, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        case 7: decode_row<7, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
        default: decode_row<8, KIND, DITH, RUN>(wk, row, cur, kappa, side_row, acc, status, bias_bits); break;
    }
}

// The last row of a gradient whose length is not a multiple of 32: one element at a time, everything at run
// time.  Same arithmetic, in the same order, as decode_row.
template <int DITH, bool RUN>
__device__ __noinline__ void decode_partial_row(const DecodeArgs& args, uint64_t row, uint64_t bucket, uint32_t nvalid)
{
    for (uint32_t e = 0; e < nvalid; ++e) {
        const uint64_t i = row * 32u + e;
        const float yside = (!RUN && args.side) ? __ldg(args.side + i) : 0.0f;
        float acc = 0.0f;
        for (uint32_t w = 0; w < args.W; ++w) {
            const DecWorker& wk = args.w[w];
            const uint32_t bits = wk.bits;
            const uint64_t bit = i * bits;
            const uint64_t num_words = (args.n * bits + 31u) >> 5;
            uint32_t lo = __ldg(wk.packed + (bit >> 5));
            const uint32_t sh = (uint32_t)(bit & 31u);
            uint32_t code = lo >> sh;
            if (sh + bits > 32u && (bit >> 5) + 1u < num_words) code |= __ldg(wk.packed + (bit >> 5) + 1u) << (32u - sh);
            code &= (1u << bits) - 1u;
            uint32_t ctr[1], rnd[1][4];
            float f;
            if (DITH == 0) {
                f = 1.5f;
            } else if (DITH == 16) {
                ctr[0] = (uint32_t)(i >> 3);
                philox4x32_10_xN<1>(ctr, wk.ps, rnd);
                f = dither16_f12(rnd[0][(i & 7u) >> 1], (int)(i & 1u));
            } else {
                ctr[0] = (uint32_t)(i >> 2);
                philox4x32_10_xN<1>(ctr, wk.ps, rnd);
                f = dither_f12(rnd[0][i & 3u]);
            }
            const float kappa = __ldg(wk.scale + bucket);
            if (args.status != nullptr && !(fabsf(kappa) <= 3.402823466e38f)) atomicOr(args.status, 0x1u);
            const float X = __fadd_rn(__uint_as_float((code << 1) | 0x4A800000u), -wk.cconst);
            float gt;
            if (wk.kind == kDecDqsg) {
                gt = __fmul_rn(__fdiv_rn(kappa, wk.s), __fadd_rn(X, -f));
            } else {
                const float yy = RUN ? __fmul_rn(acc, wk.rcp_count) : yside;
                const float a = (kappa >= 0x1p-100f) ? __fdiv_rn(wk.A, kappa) : 0.0f;
                const float c = __fdiv_rn(__fmul_rn(wk.alpha, kappa), wk.M1);
                const float r = __fmaf_rn(-yy, a, __fadd_rn(X, -f));
                const float t = (wk.kind == kDecNdqsgAnyK) ? __fdiv_rn(r, wk.Kf) : __fmul_rn(r, wk.invK);
                const float jj = __fadd_rn(__fadd_rn(t, kMagic), -kMagic);
                const float d = __fadd_rn(__fmaf_rn(-wk.Kf, jj, X), -f);
                gt = (wk.alpha == 1.0f) ? __fmul_rn(c, d) : __fmaf_rn(c, d, __fmul_rn(wk.one_m_alpha2, yy));
            }
            acc = __fadd_rn(acc, gt);
        }
        args.out[i] = (args.invW != 0.0f) ? __fmul_rn(acc, args.invW) : __fdiv_rn(acc, args.Wf);
    }
}

constexpr int kDecThreads = 128;
#ifndef DQ_DEC_MINBLOCKS
#define DQ_DEC_MINBLOCKS 4
#endif
constexpr int kDecMinBlocks = DQ_DEC_MINBLOCKS;

template <int DITH, bool RUN>
__global__ void __launch_bounds__(kDecThreads, kDecMinBlocks)
decode_aggregate_kernel(const __grid_constant__ DecodeArgs args)
{
    // Side information of the CTA's 128 rows -> shared memory (coalesced loads, 16-byte pieces swizzled so
    // that "lane r reads row r" is free of bank conflicts); every worker then re-reads it from there.
    __shared__ __align__(16) float side_tile[RUN ? 4 : kDecThreads * 32];
    grid_dependency_wait();
    grid_dependency_launch_next();
    const uint64_t row0 = args.first_row + (uint64_t)blockIdx.x * blockDim.x;
    {
        // Ask the L2 for what the CTA that runs `prefetch_blocks` blocks later (one block per SM ahead) will load
        // first: its side information and every message's words, so that those loads find their lines
        // in the L2 instead of waiting for HBM.
        const uint64_t frow0 = row0 + (uint64_t)args.prefetch_blocks * kDecThreads;
        if (frow0 + threadIdx.x < args.rows) {
            if (!RUN && args.side != nullptr) prefetch_l2(args.side + (frow0 + threadIdx.x) * 32u);
        }
        const uint32_t lane = threadIdx.x & 31u;
        for (uint32_t w = threadIdx.x >> 5; w < args.W; w += (uint32_t)kDecThreads / 32u) {
            const uint64_t first_word = frow0 * args.w[w].bits + 32u * lane;          // lines of 32 words
            if (lane < 4u * args.w[w].bits && first_word < args.rows * args.w[w].bits)
                prefetch_l2(args.w[w].packed + first_word);
        }
    }
    if (!RUN && args.side != nullptr) {
        // kDecThreads rows x 8 pieces = 8 pieces per thread
#pragma unroll
        for (uint32_t k = 0; k < 8u; ++k) {
            const uint32_t q = threadIdx.x + (uint32_t)kDecThreads * k;       // 16-byte piece inside the CTA's block
            const uint64_t piece = row0 * 8u + q;
            if (piece * 4u + 4u <= args.n) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(args.side) + piece);
                const uint32_t r = q >> 3, c = q & 7u;
                *reinterpret_cast<float4*>(side_tile + r * 32u + ((c ^ (r & 7u)) << 2)) = v;
            }
        }
        __syncthreads();
    }

    const uint64_t row = row0 + threadIdx.x;
    if (row >= args.rows) return;
    const uint64_t base = row * 32u;
    const uint64_t bucket = row / args.rows_per_bucket;
    if (base + 32u > args.n) {
        decode_partial_row<DITH, RUN>(args, row, bucket, (uint32_t)(args.n - base));
        return;
    }
    const float* side_row = side_tile + (RUN ? 0u : threadIdx.x * 32u);

    float acc[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) acc[e] = 0.0f;

    for (uint32_t w = 0; w < args.W; ++w) {
        const DecWorker& wk = args.w[w];
        uint32_t cur[8];
        float kappa;
        load_worker_row(wk, row, bucket, cur, kappa);
        switch (wk.kind) {
            case kDecDqsg: decode_row_bits<kDecDqsg, DITH, RUN>(wk, row, cur, kappa, side_row, acc, args.status, args.half_bias_bits); break;
            case kDecNdqsgPow2: decode_row_bits<kDecNdqsgPow2, DITH, RUN>(wk, row, cur, kappa, side_row, acc, args.status, args.half_bias_bits); break;
            case kDecNdqsgPow2Shrink: decode_row_bits<kDecNdqsgPow2Shrink, DITH, RUN>(wk, row, cur, kappa, side_row, acc, args.status, args.half_bias_bits); break;
            default: decode_row_bits<kDecNdqsgAnyK, DITH, RUN>(wk, row, cur, kappa, side_row, acc, args.status, args.half_bias_bits); break;
        }
    }

#pragma unroll
    for (int e = 0; e < 32; ++e)
        acc[e] = (args.invW != 0.0f) ? __fmul_rn(acc[e], args.invW) : __fdiv_rn(acc[e], args.Wf);

#pragma unroll
    for (int c = 0; c < 8; ++c)
        reinterpret_cast<float4*>(args.out + base)[c] =
            make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
}

}  // namespace dq
