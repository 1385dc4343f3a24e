// Encode kernel: per-bucket scale, dither, quantize, (coset), pack -- one pass over the gradient
// (Eq. (DQSG) and Algorithm 1, worker steps; nested encoder equation and Algorithm 2, workers in P2).
//
// Work decomposition: a "row" is 32 consecutive elements = one 128-byte line of the gradient and exactly
// `bits` 32-bit words of the bit stream.  One lane quantizes and packs a whole row, so no lane ever shares a
// packed word with another lane and no shuffles are needed for packing.
//
// Power-of-two buckets up to 8192 take the tile path: persistent CTAs of eight warps, every warp with its own
// two-stage shared-memory pipeline of 4 KB tiles (32 rows) filled by asynchronous 2-D tile copies (128-byte
// swizzle, which makes "lane r reads row r" free of bank conflicts).
//   B <= 1024: a work unit is 1024 elements; a warp takes a stage into registers, re-arms the stage with the
//     copy for the unit after next, reduces max|g| over each bucket with shuffles and quantizes from registers.
//   B = 2048, 4096, 8192: a work unit is a bucket and a warp takes 2048 elements of it as two halves in time,
//     one per stage: when both have landed it reads the maximum of the second half from shared memory, takes the
//     first half into registers, and quantizes one half after the other, re-arming each stage as soon as it is
//     in registers.  For B = 2048 no other warp is involved; for 4096 and 8192 the two or four warps of a bucket
//     meet once per bucket in a named barrier to exchange their maxima.
// The units are dealt out round-robin over the warp groups of all CTAs.  The gradient is read from HBM exactly once.
//
// Everything else -- other bucket sizes, the part of the vector past the last whole tile, the ragged end --
// is handled by plain-load code in extra CTAs of the same launch: buckets of at most 32 rows in warp windows of
// whole buckets (one row per lane, segmented maximum over the lanes), buckets of up to 4096 elements one per warp,
// larger ones one per CTA (a sweep for the maximum, then a second, cached sweep that quantizes).
#pragma once

#include "dq_device.cuh"

namespace dq {

// kEncNdqsgPow2: K = 2^BITS, the coset is the low BITS bits of the fine index; kEncNdqsgPow2Mask: a smaller power
// of two; kEncNdqsgAnyK: any K (a true modulo).
enum EncMode : int { kEncDqsg = 0, kEncNdqsgPow2 = 1, kEncNdqsgAnyK = 2, kEncNdqsgPow2Mask = 3 };

constexpr int kTileRows = 256;                     // rows a CTA holds per pipeline stage (8 warps x 32 rows, 32 KB)
constexpr int kTileBytes = kTileRows * 128;
constexpr int kConsumerWarps = kTileRows / 32;     // one row per lane
constexpr int kWarpTileBytes = 32 * 128;           // the 32 rows of a tile that one warp owns
constexpr int kEncThreads = 32 * kConsumerWarps;
#ifndef DQ_ENC_STAGES
#define DQ_ENC_STAGES 2
#endif
#ifndef DQ_ENC_CTAS_PER_SM
#define DQ_ENC_CTAS_PER_SM 3
#endif
constexpr int kEncStages = DQ_ENC_STAGES;
constexpr int kEncCtasPerSm = DQ_ENC_CTAS_PER_SM;
constexpr size_t kEncSmemBytes = (size_t)kEncStages * kTileBytes + 1024;
// Time HBM needs to deliver one warp's pipeline stages (8 KB) to each of the 148 SMs: 148 x 8 KB / 6.5 TB/s.
constexpr uint32_t kFirstRequestSpacingNs = 190u;
// Plain-load part: buckets up to 1024 elements are taken in warp windows, up to this size by one warp, above by a CTA.
constexpr uint32_t kPlainWarpBucketMax = 4096u;

struct EncodeArgs {
    const float* grad;
    uint32_t* packed;
    float* scale;
    uint64_t n;              // elements in the gradient
    uint64_t first_bucket;   // first bucket of the plain-load part
    uint64_t num_buckets;    // total buckets of the gradient
    uint64_t num_words;      // total packed words of the gradient
    uint32_t num_units;      // work units of the tile path: max(B, 1024) elements each (see encode_kernel)
    uint32_t plain_ctas;     // the first plain_ctas CTAs run the plain-load part, the rest walk over the tiles
    uint64_t plain_windows;  // B <= 1024: windows of whole buckets (at most 32 rows) in the plain-load part
    uint32_t bucket;         // B
    uint32_t bucket_log2;    // log2(B) on the tile path
    uint32_t lanes_per_bucket;  // B / 32 when B < 1024, else 32
    uint32_t warps_per_bucket;  // B / 2048 when B >= 2048, else 1
    uint32_t pair_in_time;      // B = 2048, 4096, 8192: a warp handles 2048 elements of a bucket as two halves in
                                // time; warps_per_bucket = B / 2048 warps share a bucket (units are buckets)
    float gain_num;          // DQSG: s = (L-1)/2;  NDQSG: A = alpha * M1
    float shift;             // DQSG: s
    float kmax;              // DQSG: L - 1
    uint32_t K;              // NDQSG: coarse ratio
    uint32_t K_offset;       // NDQSG any K: multiple of K that is >= 2^22
    uint32_t row_offset;     // index of grad[0]'s row in the whole gradient (0 unless a bucket range is encoded):
                             // only the dither counters see it
    uint32_t sm_count;       // SMs of the device            } spacing of the first tile requests,
    uint32_t request_spacing_ns;   // see encode_kernel      } 0 when the grid does not fill the device
    uint32_t early_read;     // the caller guarantees that grad was complete before the previous kernel of the stream
                             // began: the tile path requests (and quantizes) its first tiles while that kernel
                             // drains, and only its stores wait for it
    uint32_t early_store;    // ... and that the previous kernel neither reads nor writes this call's outputs: nothing
                             // waits for that kernel except the end of this one (see encode_kernel)
    uint32_t test_drop_copy; // test hook: warp 0 of the first tile CTA arms the barrier for its last unit without
                             // issuing the copy, so that the bounded wait for it runs out (see DQ_FLAG_TEST_DROP_COPY)
    unsigned int* error_flags;     // the library's per-device error word
    PhiloxStream ps;
};

// max(m, |a|, |b|) in one instruction (three-input max, sm_100).
__device__ __forceinline__ float max3_abs(float m, float a, float b)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(m), "f"(fabsf(a)), "f"(fabsf(b)));
    return d;
}

// Appends the low BITS bits of `tb` to the row's bit stream.  `sr` is a 32-bit shift register whose top bits are
// the most recent part of the stream: one funnel shift moves the older codes down and drops the bits of `tb` above
// the code, so no masking and no shift of the code itself is needed.  `idx` (the element's position in the row) is
// a compile-time constant after unrolling; a second funnel shift is only needed where a code straddles two words.
template <int BITS>
__device__ __forceinline__ void push_code(uint32_t& sr, uint32_t tb, int idx, uint32_t (&out)[BITS])
{
    const int end = (idx + 1) * BITS;                       // stream position after this code
    const int over = end & 31;                              // bits of this code that belong to the next word
    const bool completes = (end >> 5) != ((idx * BITS) >> 5);
    if (completes && over != 0) out[(end >> 5) - 1] = __funnelshift_r(sr, tb, BITS - over);
    sr = __funnelshift_r(sr, tb, BITS);
    if (completes && over == 0) out[(end >> 5) - 1] = sr;
}

// DQSG: bit pattern kMagicBits + k of one element, k the rounded, clamped index (0 .. L-1).
//   v = fma(g, a, delta);  w = v + s;  k = clamp(rint(w), 0, L-1)   (clamping before rounding gives the same k)
__device__ __forceinline__ uint32_t dqsg_index_bits(float x, float a, float delta, const EncodeArgs& args)
{
    const float v = __fmaf_rn(x, a, delta);
    float w = __fadd_rn(v, args.shift);
    w = fminf(fmaxf(w, 0.0f), args.kmax);
    return __float_as_uint(__fadd_rn(w, kMagic));                         // rint for 0 <= w < 2^22
}

// NDQSG: bit pattern kMagicBits + q1 (two's complement in the low bits) of one element.
__device__ __forceinline__ uint32_t ndqsg_index_bits(float x, float a, float delta)
{
    const float v = __fmaf_rn(x, a, delta);
    return __float_as_uint(__fadd_rn(v, kMagic));
}

// Quantize and pack one row.  x: the 32 elements; row: index of the row in the whole gradient (the Philox
// counters follow from it; it differs from the row's position in this call's buffers when a bucket range is
// encoded); a: the bucket's gain.  out: the row's BITS words.  DITH: 32 or 16 random bits per dither value.
//
// Adding 1.5 * 2^23 leaves the rounded index in the low mantissa bits of a float, so a code costs one fp32 add and
// one funnel shift (push_code); only a coarse ratio below 2^BITS needs an extra mask or modulo.
template <int BITS, int MODE, int DITH>
__device__ __forceinline__ void encode_row(const float (&x)[32], uint32_t row, float a,
                                           const EncodeArgs& args, uint32_t (&out)[BITS])
{
    constexpr int EPB = (DITH == 16) ? 8 : 4;       // elements per Philox block
    constexpr int PASS = 4 * EPB;                   // elements per group of four blocks
    uint32_t sr = 0u;
#pragma unroll
    for (int h = 0; h < 32 / PASS; ++h) {           // four Philox blocks in flight at a time
        uint32_t rnd[4][4];
        philox4x32_10_row<4>(row * (32u / EPB), 4 * h, args.ps, rnd);
#pragma unroll
        for (int t = 0; t < PASS; ++t) {
            const int idx = PASS * h + t;
            const float delta = dither_delta_of<DITH>(rnd, t);
            uint32_t tb;
            if (MODE == kEncDqsg) {
                tb = dqsg_index_bits(x[idx], a, delta, args);
            } else {
                tb = ndqsg_index_bits(x[idx], a, delta);
                if (MODE == kEncNdqsgPow2Mask) tb &= args.K - 1u;
                if (MODE == kEncNdqsgAnyK) tb = (tb - kMagicBits + args.K_offset) % args.K;   // q1 + positive multiple of K
            }
            push_code<BITS>(sr, tb, idx, out);
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
// Plain-load part: any bucket size, the part of the vector past the last whole tile, the ragged end.
// ---------------------------------------------------------------------------------------------------

// The `nvalid` (1..32) elements of row `grow` of the gradient, zero-filled.
__device__ __forceinline__ void load_row_plain(const EncodeArgs& args, uint64_t grow, uint32_t nvalid, float (&x)[32])
{
    const float* g = args.grad + grow * 32u;
    if (nvalid == 32u) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float4 v = reinterpret_cast<const float4*>(g)[c];
            x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) x[e] = ((uint32_t)e < nvalid) ? g[e] : 0.0f;
    }
}

// Quantizes and stores row `grow` (already in registers) with the bucket's gain `a`.
template <int BITS, int MODE, int DITH>
__device__ __forceinline__ void encode_store_row_plain(const EncodeArgs& args, const float (&x)[32], uint64_t grow,
                                                       uint32_t nvalid, float a)
{
    uint32_t out[BITS];
    encode_row<BITS, MODE, DITH>(x, (uint32_t)grow + args.row_offset, a, args, out);
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

// Buckets of at most 32 rows: a warp takes a window of as many whole buckets as fit into 32 rows, one row per
// lane; the maximum of a bucket is a segmented reduction over the lanes that hold its rows.
template <int BITS, int MODE, int DITH>
__device__ __forceinline__ void encode_window_plain(const EncodeArgs& args, uint64_t window, uint32_t lane)
{
    const uint32_t rpb = args.bucket >> 5;                     // rows per bucket (<= 32)
    const uint32_t rows_per_window = (32u / rpb) * rpb;
    const uint64_t total_rows = (args.n + 31u) >> 5;
    const uint64_t grow = (args.first_bucket * rpb) + window * rows_per_window + lane;
    const bool active = lane < rows_per_window && grow < total_rows;
    const uint32_t nvalid = !active ? 0u : (args.n - grow * 32u < 32u) ? (uint32_t)(args.n - grow * 32u) : 32u;
    float x[32];
    float mx = 0.0f;
    if (active) {
        load_row_plain(args, grow, nvalid, x);
#pragma unroll
        for (int e = 0; e < 32; e += 2) mx = max3_abs(mx, x[e], x[e + 1]);
    }
    // lanes of one bucket are adjacent: take the neighbour's maximum while it belongs to the same bucket
    const uint32_t seg = lane / rpb;
#pragma unroll
    for (uint32_t off = 1; off < 32u; off <<= 1) {
        const float up = __shfl_up_sync(0xFFFFFFFFu, mx, off);
        const float down = __shfl_down_sync(0xFFFFFFFFu, mx, off);
        if (lane >= off && (lane - off) / rpb == seg) mx = fmaxf(mx, up);
        if (lane + off < 32u && (lane + off) / rpb == seg) mx = fmaxf(mx, down);
    }
    if (!active) return;
    if (lane % rpb == 0u) args.scale[grow / rpb] = mx;
    encode_store_row_plain<BITS, MODE, DITH>(args, x, grow, nvalid, bucket_gain(args.gain_num, mx));
}

// Buckets of 33 to 128 rows: one warp per bucket (a first sweep for the maximum, then one row per lane at a time).
template <int BITS, int MODE, int DITH>
__device__ __forceinline__ void encode_bucket_warp_plain(const EncodeArgs& args, uint64_t bucket, uint32_t lane)
{
    const uint64_t lo = bucket * args.bucket;
    const uint32_t len = (uint32_t)((args.n - lo < args.bucket) ? (args.n - lo) : args.bucket);
    const float* g = args.grad + lo;
    float mx = 0.0f;
    const uint32_t quads = len >> 2;
    for (uint32_t q = lane; q < quads; q += 32u) {
        const float4 v = reinterpret_cast<const float4*>(g)[q];
        mx = max3_abs(max3_abs(mx, v.x, v.y), v.z, v.w);
    }
    for (uint32_t i = (quads << 2) + lane; i < len; i += 32u) mx = fmaxf(mx, fabsf(g[i]));
#pragma unroll
    for (uint32_t off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
    if (lane == 0) args.scale[bucket] = mx;
    const float a = bucket_gain(args.gain_num, mx);
    const uint32_t rows = (len + 31u) >> 5;
    for (uint32_t r = lane; r < rows; r += 32u) {
        const uint32_t nvalid = (len - r * 32u < 32u) ? (len - r * 32u) : 32u;
        const uint64_t grow = (lo >> 5) + r;
        float x[32];
        load_row_plain(args, grow, nvalid, x);
        encode_store_row_plain<BITS, MODE, DITH>(args, x, grow, nvalid, a);
    }
}

// Buckets of more than 128 rows: the whole CTA takes one bucket; a first sweep finds the maximum, a second one
// (served by the caches) quantizes one row per lane at a time.
template <int BITS, int MODE, int DITH>
__device__ __forceinline__ void encode_bucket_cta_plain(const EncodeArgs& args, uint64_t bucket, float* cta_max)
{
    const uint64_t lo = bucket * args.bucket;
    const uint32_t len = (uint32_t)((args.n - lo < args.bucket) ? (args.n - lo) : args.bucket);
    const float* g = args.grad + lo;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;

    float mx = 0.0f;
    const uint32_t quads = len >> 2;
    for (uint32_t q = threadIdx.x; q < quads; q += (uint32_t)kEncThreads) {
        const float4 v = reinterpret_cast<const float4*>(g)[q];
        mx = max3_abs(max3_abs(mx, v.x, v.y), v.z, v.w);
    }
    for (uint32_t i = (quads << 2) + threadIdx.x; i < len; i += (uint32_t)kEncThreads) mx = fmaxf(mx, fabsf(g[i]));
#pragma unroll
    for (uint32_t off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
    __syncthreads();                                           // the previous bucket's maxima have been read
    if (lane == 0) cta_max[warp] = mx;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) mx = fmaxf(mx, cta_max[w]);
    if (threadIdx.x == 0) args.scale[bucket] = mx;
    const float a = bucket_gain(args.gain_num, mx);

    const uint32_t rows = (len + 31u) >> 5;
    for (uint32_t r = threadIdx.x; r < rows; r += (uint32_t)kEncThreads) {
        const uint32_t nvalid = (len - r * 32u < 32u) ? (len - r * 32u) : 32u;
        const uint64_t grow = (lo >> 5) + r;
        float x[32];
        load_row_plain(args, grow, nvalid, x);
        encode_store_row_plain<BITS, MODE, DITH>(args, x, grow, nvalid, a);
    }
}

// ---------------------------------------------------------------------------------------------------
// The encode kernel.  Grid = CTAs for the plain-load part (scheduled first) + persistent tile CTAs.
// Block = 8 warps.  Dynamic shared memory = kEncSmemBytes.
//
// Tile path: lane 0 of every warp issues the 4 KB tile copy for its next unit as soon as the warp has taken the
// current rows into registers, so a copy is always in flight while the warp quantizes, and no warp ever waits
// for another one except the warps that share a bucket of 4096 or 8192 elements (named barrier, once per bucket).
// ---------------------------------------------------------------------------------------------------
template <int BITS, int MODE, int DITH>
__global__ void __launch_bounds__(kEncThreads, kEncCtasPerSm)
encode_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ EncodeArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kConsumerWarps][kEncStages];
    __shared__ float warp_max[2][kConsumerWarps];

    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31u;

    grid_dependency_launch_next();

    if (blockIdx.x < args.plain_ctas) {
        grid_dependency_wait();
        if (args.bucket <= 1024u) {
            // windows of whole buckets (at most 32 rows), one per warp, round-robin over these CTAs
            for (uint64_t w = (uint64_t)blockIdx.x * kConsumerWarps + warp; w < args.plain_windows;
                 w += (uint64_t)args.plain_ctas * kConsumerWarps)
                encode_window_plain<BITS, MODE, DITH>(args, w, lane);
        } else if (args.bucket <= kPlainWarpBucketMax) {
            // one bucket per warp at a time
            for (uint64_t b = args.first_bucket + (uint64_t)blockIdx.x * kConsumerWarps + warp;
                 b < args.num_buckets; b += (uint64_t)args.plain_ctas * kConsumerWarps)
                encode_bucket_warp_plain<BITS, MODE, DITH>(args, b, lane);
        } else {
            // one bucket per CTA at a time
            for (uint64_t b = args.first_bucket + blockIdx.x; b < args.num_buckets; b += args.plain_ctas)
                encode_bucket_cta_plain<BITS, MODE, DITH>(args, b, &warp_max[0][0]);
        }
        return;
    }

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t my_smem = smem_base + warp * (uint32_t)(kEncStages * kWarpTileBytes);
    const uint32_t my_bar = smem_u32(&bar_full[warp][0]);
    // Work unit = one bucket (B >= 2048: B / 2048 warps work on it together) or 1024 elements (smaller buckets:
    // one warp).  The groups of all tile CTAs take units round-robin, which spreads the work over the SMs to
    // within one unit.
    const uint32_t wpb = args.warps_per_bucket;      // warps sharing a bucket (1, 2, 4)
    const uint32_t group = warp / wpb;               // group of this warp inside the CTA
    const uint32_t groups_per_cta = (uint32_t)kConsumerWarps / wpb;
    const uint32_t stride = (gridDim.x - args.plain_ctas) * groups_per_cta;
    const uint32_t first_tile = (blockIdx.x - args.plain_ctas) * groups_per_cta + group;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kEncStages; ++s) mbar_init(my_bar + 8u * s, 1u);
        fence_mbar_init();
        asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&tmap) : "memory");
    }
    // Nothing above touches memory that an earlier kernel of the stream may still be writing.  When the caller
    // has declared the gradient complete (early_read), the tile copies and the arithmetic below only read memory
    // that the previous kernel does not write, and the wait moves in front of this warp's first store; when the
    // outputs are declared free as well (early_store), it moves to the end of the warp's work, where it only keeps
    // this grid from completing before its predecessor (a later kernel that waits for this one may rely on both).
    bool waited = (args.early_read == 0u);
    const bool wait_before_store = (args.early_store == 0u);
    if (waited) grid_dependency_wait();
    if (lane == 0) {
        // All resident warps would request their first tiles (the whole shared memory of every SM, a quarter of a
        // ResNet-50-sized gradient) at the same instant; served interleaved, every warp would then get its data
        // late and the ALUs would idle for 3-6 us.  Spacing the requests of an SM's warps at the rate at which
        // HBM can serve them lets the first warps start after about 1 us while the memory system stays busy.
        // (CTAs are assumed to be placed round-robin over the SMs; any other placement only changes the order.)
        // The CTAs with the lowest indices go first; they are also the ones whose warps take one unit more when
        // the units do not divide evenly, so the longest-running warps start earliest.
        const uint32_t rank = ((blockIdx.x - args.plain_ctas) / args.sm_count) * (uint32_t)kConsumerWarps + warp;
        const uint64_t until = global_timer_ns() + (uint64_t)rank * args.request_spacing_ns;
        for (uint32_t it = 0; it < 4096u && args.request_spacing_ns != 0u && global_timer_ns() < until; ++it) { }
#pragma unroll
        for (int s = 0; s < kEncStages; ++s) {
            // first copies: the next two units of this warp, or (pair mode) the two halves of its first bucket
            const uint64_t tile = args.pair_in_time ? (uint64_t)first_tile : (uint64_t)first_tile + (uint64_t)s * stride;
            const uint64_t row0 = args.pair_in_time ? (tile * wpb + warp % wpb) * 64u + (uint64_t)s * 32u : tile * 32u;
            if (tile < args.num_units) {
                mbar_expect_tx(my_bar + 8u * s, (uint32_t)kWarpTileBytes);
                tma_load_rows(my_smem + s * kWarpTileBytes, &tmap, my_bar + 8u * s, (int32_t)row0);
            }
        }
    }
    __syncwarp();

    // 128-byte swizzle: the 16-byte piece c of row r sits at piece c ^ (r & 7).  A lane's row starts at a multiple
    // of 128 bytes, so "row address + ((c ^ swz) << 4)" is "(row address | swz << 4) ^ (c << 4)": one XOR with
    // an immediate per load.
    const uint32_t swz16 = (lane & 7u) << 4;         // (row & 7) << 4: the warp's rows start at a multiple of 32
    bool gave_up = false;
    uint32_t k = 0;

    if (args.pair_in_time) {
        // B = 2048: one warp handles the whole bucket as two consecutive 1024-element halves, one per stage, so
        // no other warp is involved.  The second half only has to have landed (it was requested a whole unit
        // earlier) for its maximum to be read from shared memory before the first half is quantized.
        // B = 4096, 8192: the same, with two or four warps taking 2048 elements each and meeting once per bucket
        // to exchange their maxima.
        const uint32_t sub = warp % wpb;                 // this warp's 2048-element part of the bucket
        // (unit indices stay far below 2^32 - stride: a unit is at least 2048 elements and n < 2^34)
        for (uint32_t pair = first_tile; pair < args.num_units; pair += stride, ++k) {
            const uint32_t par = k & 1u;
            const uint32_t part = pair * wpb + sub;      // index of this warp's 2048 elements in the gradient
            float x[32];
            float mx = 0.0f;
#pragma unroll 1
            for (uint32_t half = 0; half < 2u; ++half) {
                const uint32_t stage_addr = (my_smem + half * kWarpTileBytes + lane * 128u) | swz16;
                if (half == 0u) {
                    if (!mbar_wait_bounded(my_bar, par, gave_up) ||
                        !mbar_wait_bounded(my_bar + 8u, par, gave_up)) {
                        gave_up = true;
                        if (lane == 0) atomicOr(args.error_flags, 0x2u);
                    }
                    // maximum of the second half, straight from shared memory
                    const uint32_t other = (my_smem + kWarpTileBytes + lane * 128u) | swz16;
#pragma unroll
                    for (uint32_t c = 0; c < 8; ++c) {
                        float4 v;
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                                     : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                     : "r"(other ^ (c << 4))
                                     : "memory");
                        mx = max3_abs(max3_abs(mx, v.x, v.y), v.z, v.w);
                    }
                }
#pragma unroll
                for (uint32_t c = 0; c < 8; ++c) {
                    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                                 : "=f"(x[4 * c]), "=f"(x[4 * c + 1]), "=f"(x[4 * c + 2]), "=f"(x[4 * c + 3])
                                 : "r"(stage_addr ^ (c << 4))
                                 : "memory");
                }
                if (half == 0u) {
#pragma unroll
                    for (int e = 0; e < 32; e += 2) mx = max3_abs(mx, x[e], x[e + 1]);
#pragma unroll
                    for (uint32_t off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
                    if (wpb > 1u) {
                        if (lane == 0) warp_max[par][warp] = mx;
                        named_bar_sync(1u + group, wpb * 32u);
#pragma unroll
                        for (uint32_t i = 0; i < (uint32_t)kConsumerWarps; ++i) {
                            const float o = warp_max[par][i];
                            if (i / wpb == group) mx = fmaxf(mx, o);
                        }
                    }
                } else {
                    uint32_t sink = 0u;                 // all loads of this half have completed after this
#pragma unroll
                    for (int c = 0; c < 8; ++c) sink ^= __float_as_uint(x[4 * c]);
                    asm volatile("" ::"r"(sink));
                }
                __syncwarp();
                if (lane == 0) {
                    const uint32_t next = pair + stride;
                    if (next < args.num_units) {
                        mbar_expect_tx(my_bar + 8u * half, (uint32_t)kWarpTileBytes);
                        const bool drop = args.test_drop_copy != 0u && blockIdx.x == args.plain_ctas && warp == 0u &&
                                          half == 0u && next + stride >= args.num_units;
                        if (!drop)
                            tma_load_rows(my_smem + half * kWarpTileBytes, &tmap, my_bar + 8u * half,
                                          (int32_t)((next * wpb + sub) * 64u + half * 32u));
                    }
                }
                const float a = bucket_gain(args.gain_num, mx);
                const uint32_t row = part * 64u + half * 32u + lane;
                uint32_t out[BITS];
                encode_row<BITS, MODE, DITH>(x, row + args.row_offset, a, args, out);
                if (!waited && wait_before_store) { grid_dependency_wait(); waited = true; }
                if (half == 0u && lane == 0 && sub == 0u) args.scale[pair] = mx;
                store_row_words<BITS>(args.packed + (uint64_t)row * BITS, out);
            }
        }
        if (!waited) grid_dependency_wait();
        return;
    }

    // buckets of 1024 elements or fewer: a unit is 1024 elements, one warp, one row per lane
    for (uint64_t tile = first_tile; tile < args.num_units; tile += stride, ++k) {
        const uint32_t s = k % kEncStages;
        const uint32_t use = k / kEncStages;
        if (!mbar_wait_bounded(my_bar + 8u * s, use & 1u, gave_up)) {
            gave_up = true;
            if (lane == 0) atomicOr(args.error_flags, 0x2u);
        }
        // the lane's row -> registers
        float x[32];
        const uint32_t row_addr = (my_smem + s * kWarpTileBytes + lane * 128u) | swz16;
#pragma unroll
        for (uint32_t c = 0; c < 8; ++c) {
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                         : "=f"(x[4 * c]), "=f"(x[4 * c + 1]), "=f"(x[4 * c + 2]), "=f"(x[4 * c + 3])
                         : "r"(row_addr ^ (c << 4))
                         : "memory");
        }
        // max |g| over the bucket.  Every lane has used all of its loaded values once it reaches the
        // __syncwarp below, so after it the stage can be overwritten by the next copy.
        float mx = 0.0f;
#pragma unroll
        for (int e = 0; e < 32; e += 2) mx = max3_abs(mx, x[e], x[e + 1]);
#pragma unroll
        for (uint32_t off = 16; off > 0; off >>= 1) {
            const float o = __shfl_xor_sync(0xFFFFFFFFu, mx, off);
            if (off < args.lanes_per_bucket) mx = fmaxf(mx, o);
        }
        __syncwarp();
        if (lane == 0) {
            const uint64_t next = tile + (uint64_t)kEncStages * stride;
            if (next < args.num_units) {
                mbar_expect_tx(my_bar + 8u * s, (uint32_t)kWarpTileBytes);
                const bool drop = args.test_drop_copy != 0u && blockIdx.x == args.plain_ctas && warp == 0u &&
                                  next + stride >= args.num_units;
                if (!drop)
                    tma_load_rows(my_smem + s * kWarpTileBytes, &tmap, my_bar + 8u * s, (int32_t)(next * 32u));
            }
        }
        const uint32_t row = (uint32_t)tile * 32u + lane;   // row index in the gradient (< 2^29)
        const float a = bucket_gain(args.gain_num, mx);

        uint32_t out[BITS];
        encode_row<BITS, MODE, DITH>(x, row + args.row_offset, a, args, out);
        if (!waited && wait_before_store) { grid_dependency_wait(); waited = true; }
        if ((lane & (args.lanes_per_bucket - 1u)) == 0u) args.scale[row >> (args.bucket_log2 - 5u)] = mx;
        store_row_words<BITS>(args.packed + (uint64_t)row * BITS, out);
    }
    if (!waited) grid_dependency_wait();
}

}  // namespace dq
