// Encode kernels: per-bucket scale, dither, quantize, (coset), pack -- all in one pass over the gradient
// (Eq. (DQSG) and Algorithm 1, worker steps; nested encoder equation and Algorithm 2, workers in P2).
//
// Work decomposition: a "row" is 32 consecutive elements = one 128-byte line of the gradient and exactly
// `bits` 32-bit words of the bit stream.  One lane quantizes and packs whole rows, so no lane ever shares a
// packed word with another lane.
//   * encode_tiles_kernel: power-of-two buckets.  A warp owns a tile of max(B, 1024) elements; the tile is
//     brought into shared memory by one asynchronous 2-D tile copy with the 128-byte swizzle, which makes
//     "lane r reads row r" free of bank conflicts.  Pass 1 reduces max|g| per bucket with warp shuffles,
//     pass 2 re-reads the tile from shared memory, so the gradient is read from HBM exactly once.
//   * encode_buckets_kernel: any bucket size, the ragged tail, and everything the tile kernel leaves over;
//     plain loads, one warp per bucket.
#pragma once

#include "dq_device.cuh"

namespace dq {

enum EncMode : int { kEncDqsg = 0, kEncNdqsgPow2 = 1, kEncNdqsgAnyK = 2 };

struct EncodeArgs {
    const float* grad;       // only used by encode_buckets_kernel
    uint32_t* packed;
    float* scale;
    uint64_t n;              // elements in the gradient
    uint64_t first_bucket;   // encode_buckets_kernel: first bucket to handle
    uint64_t num_buckets;    // total buckets of the gradient
    uint64_t num_words;      // total packed words of the gradient
    uint32_t num_tiles;      // encode_tiles_kernel: full tiles
    uint32_t bucket;         // B
    uint32_t rows_per_tile;  // T / 32
    uint32_t lanes_per_bucket;  // B / 32 when B < 1024, else 32
    float gain_num;          // DQSG: s = (L-1)/2;  NDQSG: A = alpha * M1
    float shift;             // DQSG: s;  NDQSG: unused
    float kmax;              // DQSG: L - 1
    uint32_t K;              // NDQSG: coarse ratio
    uint32_t K_offset;       // NDQSG any K: multiple of K that is >= 2^22
    PhiloxStream ps;
};

__device__ unsigned int g_dq_error_flags = 0u;

// Quantize and pack one row.  x: the 32 elements; chunk0: index of the row's first 4-element chunk in the
// whole gradient (= row index * 8); a: the bucket's gain.  out: the row's BITS words.
template <int BITS, int MODE>
__device__ __forceinline__ void encode_row(const float (&x)[32], uint32_t chunk0, float a,
                                           const EncodeArgs& args, uint32_t (&out)[BITS])
{
#pragma unroll
    for (int j = 0; j < BITS; ++j) out[j] = 0u;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t rnd[4];
        philox4x32_10(chunk0 + (uint32_t)c, args.ps, rnd);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = 4 * c + e;
            const float delta = __fadd_rn(dither_f12(rnd[e]), -1.5f);     // exact
            const float v = __fmaf_rn(x[idx], a, delta);
            uint32_t code;
            if (MODE == kEncDqsg) {
                float w = __fadd_rn(v, args.shift);
                w = fminf(fmaxf(w, 0.0f), args.kmax);                      // clamp, then round: same integer
                code = __float_as_uint(__fadd_rn(w, kMagic)) & 0xFFu;
            } else {
                const uint32_t tb = __float_as_uint(__fadd_rn(v, kMagic)); // kMagicBits + q1 (two's complement)
                if (MODE == kEncNdqsgPow2) {
                    code = tb & (args.K - 1u);
                } else {
                    const uint32_t q_off = tb - kMagicBits + args.K_offset; // q1 + multiple of K, positive
                    code = q_off % args.K;
                }
            }
            const int bit = idx * BITS;
            const int wi = bit >> 5;
            const int sh = bit & 31;
            out[wi] |= code << sh;
            if (sh + BITS > 32) out[wi + 1] |= code >> (32 - sh);
        }
    }
}

template <int BITS>
__device__ __forceinline__ void store_row_words(uint32_t* dst, const uint32_t (&out)[BITS])
{
    if constexpr (BITS % 4 == 0) {
#pragma unroll
        for (int j = 0; j < BITS; j += 4)
            reinterpret_cast<uint4*>(dst)[j >> 2] = make_uint4(out[j], out[j + 1], out[j + 2], out[j + 3]);
    } else if constexpr (BITS % 2 == 0) {
#pragma unroll
        for (int j = 0; j < BITS; j += 2)
            reinterpret_cast<uint2*>(dst)[j >> 1] = make_uint2(out[j], out[j + 1]);
    } else {
#pragma unroll
        for (int j = 0; j < BITS; ++j) dst[j] = out[j];
    }
}

__device__ __forceinline__ float bucket_gain(float num, float kappa)
{
    return (kappa >= 0x1p-100f) ? __fdiv_rn(num, kappa) : 0.0f;
}

// ---------------------------------------------------------------------------------------------------
// Power-of-two buckets, full tiles.  blockDim.x = 32 * warps; dynamic shared memory =
// warps * rows_per_tile * 128 + 1024 bytes.
// ---------------------------------------------------------------------------------------------------
constexpr int kEncMaxWarps = 8;

template <int BITS, int MODE>
__global__ void __launch_bounds__(32 * kEncMaxWarps)
encode_tiles_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ EncodeArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kEncMaxWarps];

    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t tile = blockIdx.x * warps + warp;
    if (tile >= args.num_tiles) return;

    const uint32_t tile_bytes = args.rows_per_tile * 128u;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t tile_smem = smem_base + warp * tile_bytes;
    const uint32_t bar = smem_u32(&bars[warp]);
    const uint32_t row0 = tile * args.rows_per_tile;        // first row of the tile in the gradient

    if (lane == 0) {
        mbar_init(bar, 1u);
        fence_mbar_init();
    }
    __syncwarp();
    if (lane == 0) {
        mbar_expect_tx(bar, tile_bytes);
        tma_load_rows(tile_smem, &tmap, bar, (int32_t)row0);
    }
    if (!mbar_wait_bounded(bar, 0u)) {
        if (lane == 0) atomicOr(&g_dq_error_flags, 0x2u);
        return;
    }

    const uint32_t rows_per_lane = args.rows_per_tile >> 5;
    const uint32_t swz = lane & 7u;                         // (row & 7) is the same for all of a lane's rows

    // pass 1: max |g| over the lane's rows, then over the lanes of the bucket
    float mx = 0.0f;
    for (uint32_t k = 0; k < rows_per_lane; ++k) {
        const uint32_t row_addr = tile_smem + (lane + 32u * k) * 128u;
#pragma unroll
        for (uint32_t c = 0; c < 8; ++c) {
            float4 v;
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                         : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                         : "r"(row_addr + ((c ^ swz) << 4)));
            mx = fmaxf(mx, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        }
    }
    for (uint32_t off = args.lanes_per_bucket >> 1; off > 0; off >>= 1)
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));

    if (args.bucket >= 1024u) {
        if (lane == 0) args.scale[tile] = mx;
    } else if ((lane & (args.lanes_per_bucket - 1u)) == 0u) {
        const uint32_t buckets_per_tile = 32u / args.lanes_per_bucket;
        args.scale[(uint64_t)tile * buckets_per_tile + lane / args.lanes_per_bucket] = mx;
    }
    const float a = bucket_gain(args.gain_num, mx);

    // pass 2: quantize and pack, one row at a time
    for (uint32_t k = 0; k < rows_per_lane; ++k) {
        const uint32_t r = lane + 32u * k;
        const uint32_t row_addr = tile_smem + r * 128u;
        float x[32];
#pragma unroll
        for (uint32_t c = 0; c < 8; ++c) {
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                         : "=f"(x[4 * c]), "=f"(x[4 * c + 1]), "=f"(x[4 * c + 2]), "=f"(x[4 * c + 3])
                         : "r"(row_addr + ((c ^ swz) << 4)));
        }
        uint32_t out[BITS];
        const uint32_t grow = row0 + r;
        encode_row<BITS, MODE>(x, grow * 8u, a, args, out);
        store_row_words<BITS>(args.packed + (uint64_t)grow * BITS, out);
    }
}

// ---------------------------------------------------------------------------------------------------
// Any bucket size / ragged tail: one warp per bucket, plain loads.
// ---------------------------------------------------------------------------------------------------
template <int BITS, int MODE>
__global__ void __launch_bounds__(128)
encode_buckets_kernel(const __grid_constant__ EncodeArgs args)
{
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t bucket = args.first_bucket + (uint64_t)blockIdx.x * (blockDim.x >> 5) + warp;
    if (bucket >= args.num_buckets) return;

    const uint64_t lo = bucket * args.bucket;
    const uint32_t len = (uint32_t)((args.n - lo < args.bucket) ? (args.n - lo) : args.bucket);
    const float* g = args.grad + lo;

    float mx = 0.0f;
    for (uint32_t i = lane; i < len; i += 32u) mx = fmaxf(mx, fabsf(g[i]));
#pragma unroll
    for (uint32_t off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
    if (lane == 0) args.scale[bucket] = mx;
    const float a = bucket_gain(args.gain_num, mx);

    const uint32_t rows = (len + 31u) >> 5;
    for (uint32_t r = lane; r < rows; r += 32u) {
        const uint32_t base = r * 32u;
        const uint32_t nvalid = (len - base < 32u) ? (len - base) : 32u;
        float x[32];
        if (nvalid == 32u) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 v = reinterpret_cast<const float4*>(g + base)[c];
                x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) x[e] = ((uint32_t)e < nvalid) ? g[base + e] : 0.0f;
        }
        uint32_t out[BITS];
        const uint64_t grow = (lo >> 5) + r;
        encode_row<BITS, MODE>(x, (uint32_t)(grow * 8u), a, args, out);
        uint32_t* dst = args.packed + grow * BITS;
        if (nvalid == 32u) {
            store_row_words<BITS>(dst, out);
        } else {
            // last row of the gradient: clear the codes of elements past the end, write only existing words
            const uint32_t valid_bits = nvalid * BITS;
#pragma unroll
            for (int j = 0; j < BITS; ++j) {
                const int32_t keep = (int32_t)valid_bits - 32 * j;
                if (keep <= 0) continue;
                const uint32_t m = (keep >= 32) ? 0xFFFFFFFFu : ((1u << keep) - 1u);
                if (grow * BITS + j < args.num_words) dst[j] = out[j] & m;
            }
        }
    }
}

}  // namespace dq
