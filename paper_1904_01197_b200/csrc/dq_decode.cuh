// Fused decode-and-average kernel (Algorithm 1, server steps; nested decoder equation and Algorithm 2,
// server loop with the side information given as a vector).
//
// One lane owns one row = 32 consecutive elements: 32 fp32 accumulators in registers, and per worker
// exactly `bits` packed words.  For every worker (in array order) the lane reloads that worker's words and
// bucket scale, regenerates the 32 dithers with eight Philox blocks, reconstructs and accumulates; the mean
// is written at the end.  The packed streams, the side information and the output are each touched once.
#pragma once

#include "dq_device.cuh"

namespace dq {

struct DecWorker {
    const uint32_t* packed;
    const float* scale;
    PhiloxStream ps;
    uint32_t kind;        // 0 DQSG, 1 NDQSG
    uint32_t bits;
    uint32_t K;           // NDQSG coarse ratio
    uint32_t K_is_pow2;
    float s;              // DQSG (L-1)/2
    float cconst;         // DQSG: 4194304 + s - 1.5 ; NDQSG: 4194304 - 1.5   (see unpack_half_biased)
    float A;              // NDQSG alpha * M1
    float M1;
    float alpha;
    float one_m_alpha2;   // 1 - alpha*alpha
    float Kf;             // (float)K
    float invK;           // 1/K (exact when K is a power of two)
};

struct DecodeArgs {
    const float* side;
    float* out;
    uint32_t* status;
    uint64_t n;
    uint64_t rows;            // ceil(n / 32)
    uint32_t W;
    uint32_t rows_per_bucket; // B / 32
    float Wf;
    float invW;               // 1/W when W is a power of two, else 0
    DecWorker w[64];
};

// Code of element `idx` of a row, returned as the bit pattern of the float 2^22 + code (code in mantissa
// bits 1.., since floats in [2^22, 2^23) step by 1/2).  Subtracting a constant then gives code - c exactly.
template <int BITS>
__device__ __forceinline__ float unpack_half_biased(const uint32_t (&words)[BITS], int idx)
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
    return __uint_as_float((v & mask2) | 0x4A800000u);
}

template <int BITS>
__device__ __forceinline__ void decode_row(const DecWorker& wk, uint64_t row, uint64_t bucket, bool full_row,
                                           uint64_t n, const float (&y)[32], float (&acc)[32],
                                           uint32_t* status)
{
    // this worker's words for the row
    uint32_t words[BITS];
    const uint32_t* src = wk.packed + row * BITS;
    if (full_row) {
        if constexpr (BITS % 4 == 0) {
#pragma unroll
            for (int j = 0; j < BITS; j += 4) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(src) + (j >> 2));
                words[j] = v.x; words[j + 1] = v.y; words[j + 2] = v.z; words[j + 3] = v.w;
            }
        } else if constexpr (BITS % 2 == 0) {
#pragma unroll
            for (int j = 0; j < BITS; j += 2) {
                const uint2 v = __ldg(reinterpret_cast<const uint2*>(src) + (j >> 1));
                words[j] = v.x; words[j + 1] = v.y;
            }
        } else {
#pragma unroll
            for (int j = 0; j < BITS; ++j) words[j] = __ldg(src + j);
        }
    } else {
        const uint64_t num_words = (n * BITS + 31u) >> 5;
#pragma unroll
        for (int j = 0; j < BITS; ++j) words[j] = (row * BITS + j < num_words) ? __ldg(src + j) : 0u;
    }

    const float kappa = __ldg(wk.scale + bucket);
    if (status != nullptr && !(fabsf(kappa) <= 3.402823466e38f)) atomicOr(status, 0x1u);

    const uint32_t chunk0 = (uint32_t)(row * 8u);
    if (wk.kind == 0u) {
        // g~ = (kappa/s) ((k - s) - delta), with (k - s + 1.5) - f == (k - s) - delta after one rounding
        const float c = __fdiv_rn(kappa, wk.s);
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
            uint32_t rnd[4];
            philox4x32_10(chunk0 + (uint32_t)ch, wk.ps, rnd);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int idx = 4 * ch + e;
                const float X = __fadd_rn(unpack_half_biased<BITS>(words, idx), -wk.cconst);   // k - s + 1.5
                const float d = __fadd_rn(X, -dither_f12(rnd[e]));
                acc[idx] = __fadd_rn(acc[idx], __fmul_rn(c, d));
            }
        }
    } else {
        const float a = (kappa >= 0x1p-100f) ? __fdiv_rn(wk.A, kappa) : 0.0f;
        const float beta = __fdiv_rn(__fmul_rn(wk.alpha, kappa), wk.M1);
        const bool shrink = (wk.alpha != 1.0f);
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
            uint32_t rnd[4];
            philox4x32_10(chunk0 + (uint32_t)ch, wk.ps, rnd);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int idx = 4 * ch + e;
                const float f = dither_f12(rnd[e]);
                const float X1 = __fadd_rn(unpack_half_biased<BITS>(words, idx), -wk.cconst);  // m + 1.5
                const float r1 = __fadd_rn(X1, -f);                                            // m - delta
                const float r = __fmaf_rn(-y[idx], a, r1);
                const float t = wk.K_is_pow2 ? __fmul_rn(r, wk.invK) : __fdiv_rn(r, wk.Kf);
                const float jj = __fadd_rn(__fadd_rn(t, kMagic), -kMagic);                     // rint(r / K)
                const float Y = __fmaf_rn(-wk.Kf, jj, X1);                                     // q1^ + 1.5, exact
                const float d = __fadd_rn(Y, -f);                                              // q1^ - delta
                float gt;
                if (shrink) gt = __fmaf_rn(beta, d, __fmul_rn(wk.one_m_alpha2, y[idx]));
                else gt = __fmul_rn(beta, d);
                acc[idx] = __fadd_rn(acc[idx], gt);
            }
        }
    }
}

template <bool HAS_SIDE>
__global__ void __launch_bounds__(128)
decode_aggregate_kernel(const __grid_constant__ DecodeArgs args)
{
    const uint64_t row = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= args.rows) return;
    const uint64_t base = row * 32u;
    const bool full_row = (base + 32u <= args.n);
    const uint32_t nvalid = full_row ? 32u : (uint32_t)(args.n - base);
    const uint64_t bucket = row / args.rows_per_bucket;

    float y[32];
    float acc[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) { acc[e] = 0.0f; y[e] = 0.0f; }
    if (HAS_SIDE) {
        if (full_row) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(args.side + base) + c);
                y[4 * c] = v.x; y[4 * c + 1] = v.y; y[4 * c + 2] = v.z; y[4 * c + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) y[e] = ((uint32_t)e < nvalid) ? __ldg(args.side + base + e) : 0.0f;
        }
    }

    for (uint32_t w = 0; w < args.W; ++w) {
        const DecWorker& wk = args.w[w];
        switch (wk.bits) {
            case 1: decode_row<1>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            case 2: decode_row<2>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            case 3: decode_row<3>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            case 4: decode_row<4>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            case 5: decode_row<5>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            case 6: decode_row<6>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            case 7: decode_row<7>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
            default: decode_row<8>(wk, row, bucket, full_row, args.n, y, acc, args.status); break;
        }
    }

#pragma unroll
    for (int e = 0; e < 32; ++e)
        acc[e] = (args.invW != 0.0f) ? __fmul_rn(acc[e], args.invW) : __fdiv_rn(acc[e], args.Wf);

    if (full_row) {
#pragma unroll
        for (int c = 0; c < 8; ++c)
            reinterpret_cast<float4*>(args.out + base)[c] =
                make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
    } else {
#pragma unroll
        for (int e = 0; e < 32; ++e)
            if ((uint32_t)e < nvalid) args.out[base + e] = acc[e];
    }
}

}  // namespace dq
