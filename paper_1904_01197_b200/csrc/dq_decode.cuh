// Fused decode-and-average kernel (Algorithm 1, server steps; nested decoder equation and Algorithm 2,
// server loop with the side information given as a vector, taken as the running mean, or taken as the
// reconstruction of message 0).
//
// One lane owns one row = 32 consecutive elements: 32 fp32 accumulators in registers, and per worker exactly
// `bits` packed words.  A warp owns a unit of 32 rows.  One persistent CTA of sixteen warps runs per SM; its
// warps form teams of four that take four adjacent units at a time from the CTA's share of the gradient.  The
// share is fixed (CTA c owns every gridDim.x-th group of four units), the order inside it is not: teams draw the
// next group from a counter in shared memory, because the warp schedulers favour some warps by a fifth and a
// fixed split would leave the favoured ones idle at the end.
//   * The side information of a unit arrives in the warp's shared memory by one 2-D tile copy (32 rows x 128
//     bytes, 128-byte swizzle, so that "lane r reads row r" is free of bank conflicts), issued one unit ahead.
//   * Every worker's packed words of the next unit are requested into the L2 one unit ahead (one prefetch
//     instruction per unit: lane w asks for worker w's lines); each lane then loads exactly its `bits` words with
//     the widest vector loads their alignment allows, and the Philox work that follows hides the L2 latency.
//   * For every worker (in array order) the lane regenerates the 32 dithers (Philox blocks four at a time),
//     reconstructs and accumulates; the bucket scale is loaded one step ahead.
//   * The mean goes back through the tile buffer and leaves with one tile store per unit: full 128-byte lines,
//     issued by one lane.
// The packed streams, the side information and the output are each touched once in HBM.
//
// The path is bound by instruction issue, not by HBM: each (element, worker) pair needs a quarter of a
// Philox block (4.5 wide multiplies, which occupy the multiplier pipe for four cycles each) before any
// reconstruction arithmetic.
#pragma once

#include "dq_device.cuh"

namespace dq {

// Where the side information of the nested messages comes from: a vector given by the caller (or none at all: only
// DQSG messages), the running mean of the messages decoded so far, or the reconstruction of message 0.
enum DecSide : int { kSideGiven = 0, kSideRunning = 1, kSideFirst = 2 };

enum DecKind : uint32_t { kDecDqsg = 0, kDecNdqsgPow2 = 1, kDecNdqsgPow2Shrink = 2, kDecNdqsgAnyK = 3 };

struct DecWorker {
    const uint32_t* packed;   // } addresses of the (virtual) whole-gradient buffers, see DecodeArgs
    const float* scale;       // }
    uint32_t unit_lines;      // 128-byte lines of one unit's packed words (= bits)
    uint32_t group_end;       // index after the last worker of the run of equal variants that this worker belongs to
    PhiloxStream ps;
    uint32_t variant;     // DecKind * 8 + bits - 1: one jump selects the routine
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
    float step_mul;       // DQSG: 1/s, NDQSG: 1/M1, when that divisor is a power of two (the division is then an
                          // exact multiplication); 0 otherwise
};

struct DecodeArgs {
    const float* side;
    float* out;
    uint32_t* status;
    // A call may cover the elements [first, n) of a longer gradient (first a multiple of the bucket size, 0 for a
    // whole gradient).  Rows, elements and buckets are then numbered as in the whole gradient -- which is what the
    // dither counters need -- and every pointer above and in w[] is the buffer's address minus the range's offset,
    // so that "pointer + global index" lands in the caller's buffer.  The tile maps cover the caller's buffers
    // themselves (row 0 of a map = row first_row of the gradient) and only whole rows.
    uint64_t n;               // end of the range (element index)
    uint32_t rows;            // ceil(n / 32): end of the range (row index); below 2^29
    uint32_t first_row;       // first / 32
    uint32_t full_rows;       // floor(n / 32): rows below this index have 32 elements
    uint32_t num_units;       // ceil((rows - first_row) / 32): units of 32 rows
    uint32_t W;
    uint32_t rows_per_bucket; // B / 32
    uint32_t rpb_shift;       // log2(rows_per_bucket) when that is a power of two, else 0xFFFFFFFF
    uint32_t has_side;        // the side information vector is read (some message is NDQSG, not running-mean mode)
    uint32_t use_tiles;       // the range holds at least one whole row: the tile maps are valid
    uint32_t half_bias_bits;  // 0x4A800000 (bit pattern of 2^22), passed in so that it lives in a register
    float Wf;
    float invW;               // 1/W when W is a power of two, else 0
    unsigned int* error_flags;    // the library's per-device error word
    DecWorker w[64];
};

#ifndef DQ_DEC_THREADS
#define DQ_DEC_THREADS 512
#endif
constexpr int kDecThreads = DQ_DEC_THREADS;
constexpr int kDecWarps = kDecThreads / 32;
#ifndef DQ_DEC_MINBLOCKS
#define DQ_DEC_MINBLOCKS (512 / DQ_DEC_THREADS)
#endif
constexpr int kDecMinBlocks = DQ_DEC_MINBLOCKS;     // resident CTAs per SM the register budget is set for
#ifndef DQ_DEC_TEAM
#define DQ_DEC_TEAM 4
#endif
constexpr int kDecTeamWarps = DQ_DEC_TEAM;          // warps that take adjacent units and meet before each
constexpr int kDecTeams = kDecWarps / kDecTeamWarps;
static_assert(kDecWarps % kDecTeamWarps == 0 && kDecTeams >= 1 && (kDecTeamWarps == 1 || kDecTeams <= 15),
              "teams of several warps use named barriers 1..15");
constexpr int kDecTileBytes = 32 * 128;         // one unit of side information or output
constexpr int kDecTileBuffers = 3;              // per warp: side in flight / side in use, then output leaving
// Dynamic shared memory of a CTA: the warps' tile buffers (plus room to align to 1024 bytes).
constexpr uint32_t kDecSmemBytes = (uint32_t)(kDecWarps * kDecTileBuffers * kDecTileBytes) + 1024u;

// Code of element `idx` of a row as the float 2^22 + code: the bit pattern of 2^22 with the code in mantissa
// bits 1.. (floats in [2^22, 2^23) step by 1/2).  Subtracting a constant then gives code - c exactly.
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

// The lane's BITS words (p = address of the first one; a row of BITS words starts at a multiple of 4 * BITS
// bytes), with the widest loads that alignment allows.
template <int BITS>
__device__ __forceinline__ void load_words(const uint32_t* p, uint32_t (&w)[BITS])
{
    if constexpr (BITS % 4 == 0) {
#pragma unroll
        for (int j = 0; j < BITS; j += 4) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + j));
            w[j] = v.x; w[j + 1] = v.y; w[j + 2] = v.z; w[j + 3] = v.w;
        }
    } else if constexpr (BITS % 2 == 0) {
#pragma unroll
        for (int j = 0; j < BITS; j += 2) {
            const uint2 v = __ldg(reinterpret_cast<const uint2*>(p + j));
            w[j] = v.x; w[j + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int j = 0; j < BITS; ++j) w[j] = __ldg(p + j);
    }
}

// One worker's contribution to the 32 accumulators of a row.
//   DQSG:  g~ = (kappa/s) ((k - s) - delta); (k - s + 1.5) - f rounds once to the same value.
//   NDQSG: r = (m - delta) - y a;  jj = rint(r / K);  q1^ = m - K jj;  g~ = beta (q1^ - delta) [+ (1-alpha^2) y]
// load_row: the row whose words the lane loads (its own row, or the last whole row for lanes past the end, whose
// results are never stored); side_addr: shared-memory address of
// the lane's row of side information with the swizzle term already OR-ed in (piece p is at side_addr ^ (p << 4)).
template <int BITS, uint32_t KIND, int DITH, bool RUN>
__device__ __forceinline__ void decode_row(const DecWorker& wk, uint32_t row, uint32_t load_row, float kappa,
                                           uint32_t side_addr, float (&acc)[32], uint32_t bias_bits)
{
    uint32_t words[BITS];
    load_words<BITS>(wk.packed + (uint64_t)load_row * (uint32_t)BITS, words);

    // kappa / s and alpha kappa / M1: a division by a power of two is an exact multiplication
    float c, a = 0.0f;
    if (KIND == kDecDqsg) {
        c = (wk.step_mul != 0.0f) ? __fmul_rn(kappa, wk.step_mul) : __fdiv_rn(kappa, wk.s);
    } else {
        a = (kappa >= 0x1p-100f) ? __fdiv_rn(wk.A, kappa) : 0.0f;
        const float ak = __fmul_rn(wk.alpha, kappa);
        c = (wk.step_mul != 0.0f) ? __fmul_rn(ak, wk.step_mul) : __fdiv_rn(ak, wk.M1);            // beta
    }
    constexpr int EPB = (DITH == 16) ? 8 : 4;       // elements per Philox block
    constexpr int PASS = 4 * EPB;                   // elements per group of four blocks
#pragma unroll
    for (int h = 0; h < 32 / PASS; ++h) {
        uint32_t rnd[4][4];
        if (DITH != 0) philox4x32_10_row<4>(row * (32u / EPB), 4 * h, wk.ps, rnd);
#pragma unroll
        for (int q = 0; q < PASS / 4; ++q) {        // four elements at a time (one 16-byte piece of y)
            float y[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (KIND != kDecDqsg && !RUN) {
                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                             : "=f"(y[0]), "=f"(y[1]), "=f"(y[2]), "=f"(y[3])
                             : "r"(side_addr ^ (uint32_t)(((PASS / 4) * h + q) << 4))
                             : "memory");
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

// State of a lane while it walks over the workers of a unit.
struct DecLane {
    uint32_t row, load_row, bucket, bucket_next, row_addr, kappa_bits_max;
    float kappa_next;
};

// The workers [w, w_end) of one run of equal variants: the same routine for each, so the jump on the variant is taken
// once per run and not once per worker (Algorithm 2's groups P1 and P2 are two runs).
template <int BITS, uint32_t KIND, int DITH, int SIDE>
__device__ __forceinline__ void decode_run(const DecodeArgs& args, uint32_t w, uint32_t w_end, DecLane& ln, float (&acc)[32])
{
#pragma unroll 1
    for (; w < w_end; ++w) {
        const float kappa = ln.kappa_next;
        // the next step's scale: the next worker's for this bucket, or the first worker's for the next unit
        ln.kappa_next = (w + 1u < args.W) ? __ldg(args.w[w + 1u].scale + ln.bucket)
                                          : __ldg(args.w[0].scale + ln.bucket_next);
        decode_row<BITS, KIND, DITH, SIDE == kSideRunning>(args.w[w], ln.row, ln.load_row, kappa, ln.row_addr, acc,
                                                            args.half_bias_bits);
        if (SIDE == kSideFirst && w == 0u) {
            // the accumulators are now the reconstruction of message 0: it is the side information of the nested
            // messages that follow, which read it from the lane's row of the tile buffer
#pragma unroll
            for (int c = 0; c < 8; ++c)
                asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};"
                             ::"r"(ln.row_addr ^ (uint32_t)(c << 4)), "f"(acc[4 * c]), "f"(acc[4 * c + 1]),
                               "f"(acc[4 * c + 2]), "f"(acc[4 * c + 3])
                             : "memory");
        }
        const uint32_t kb = __float_as_uint(kappa) & 0x7FFFFFFFu;
        ln.kappa_bits_max = (kb > ln.kappa_bits_max) ? kb : ln.kappa_bits_max;
    }
}

// All W workers of a unit, run by run; dispatch on (kind, bits) with one jump per run.
template <int DITH, int SIDE>
__device__ __forceinline__ void decode_workers(const DecodeArgs& args, DecLane& ln, float (&acc)[32])
{
#define DQ_DEC_CASE(KIND, BITS)                                                                                    \
    case (KIND) * 8u + (BITS) - 1u: decode_run<BITS, KIND, DITH, SIDE>(args, w, w_end, ln, acc); break;
#define DQ_DEC_KIND(KIND)                                                                                          \
    DQ_DEC_CASE(KIND, 1) DQ_DEC_CASE(KIND, 2) DQ_DEC_CASE(KIND, 3) DQ_DEC_CASE(KIND, 4)                            \
    DQ_DEC_CASE(KIND, 5) DQ_DEC_CASE(KIND, 6) DQ_DEC_CASE(KIND, 7) DQ_DEC_CASE(KIND, 8)
#pragma unroll 1
    for (uint32_t w = 0; w < args.W;) {
        const uint32_t w_end = args.w[w].group_end;
        switch (args.w[w].variant) {
            DQ_DEC_KIND(kDecDqsg)
            DQ_DEC_KIND(kDecNdqsgPow2)
            DQ_DEC_KIND(kDecNdqsgPow2Shrink)
            DQ_DEC_KIND(kDecNdqsgAnyK)
            default: break;
        }
        w = w_end;
    }
#undef DQ_DEC_KIND
#undef DQ_DEC_CASE
}

// The last row of a gradient whose length is not a multiple of 32: one element per lane (`e` = the lane, of a
// whole warp), everything at run time, straight from and to global memory.  Same arithmetic, in the same order,
// as decode_row.  Each element is a chain of dependent loads and divisions, about a microsecond per worker.
template <int DITH, int SIDE>
__device__ __noinline__ void decode_partial_row(const DecodeArgs& args, uint32_t row, uint32_t bucket, uint32_t nvalid,
                                                uint32_t e)
{
    constexpr bool RUN = (SIDE == kSideRunning);
    if (e < nvalid) {
        const uint64_t i = (uint64_t)row * 32u + e;
        float yside = (!RUN && args.has_side) ? __ldg(args.side + i) : 0.0f;
        float acc = 0.0f;
        for (uint32_t w = 0; w < args.W; ++w) {
            if (SIDE == kSideFirst && w == 1u) yside = acc;      // the reconstruction of message 0
            const DecWorker& wk = args.w[w];
            const uint32_t kind = wk.variant >> 3;
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
            if (kind == kDecDqsg) {
                gt = __fmul_rn(__fdiv_rn(kappa, wk.s), __fadd_rn(X, -f));
            } else {
                const float yy = RUN ? __fmul_rn(acc, wk.rcp_count) : yside;
                const float a = (kappa >= 0x1p-100f) ? __fdiv_rn(wk.A, kappa) : 0.0f;
                const float c = __fdiv_rn(__fmul_rn(wk.alpha, kappa), wk.M1);
                const float r = __fmaf_rn(-yy, a, __fadd_rn(X, -f));
                const float t = (kind == kDecNdqsgAnyK) ? __fdiv_rn(r, wk.Kf) : __fmul_rn(r, wk.invK);
                const float jj = __fadd_rn(__fadd_rn(t, kMagic), -kMagic);
                const float d = __fadd_rn(__fmaf_rn(-wk.Kf, jj, X), -f);
                gt = (wk.alpha == 1.0f) ? __fmul_rn(c, d) : __fmaf_rn(c, d, __fmul_rn(wk.one_m_alpha2, yy));
            }
            acc = __fadd_rn(acc, gt);
        }
        args.out[i] = (args.invW != 0.0f) ? __fmul_rn(acc, args.invW) : __fdiv_rn(acc, args.Wf);
    }
}

// ---------------------------------------------------------------------------------------------------
// The decode kernel.  Grid = persistent CTAs (one per SM) of teams of four warps; dynamic shared memory =
// kDecSmemBytes.
// side_map / out_map: [whole rows x 32 floats] views of the caller's side information and output (valid when
// args.use_tiles; side_map only when args.has_side).
// ---------------------------------------------------------------------------------------------------
template <int DITH, int SIDE>
__global__ void __launch_bounds__(kDecThreads, kDecMinBlocks)
decode_aggregate_kernel(const __grid_constant__ CUtensorMap side_map, const __grid_constant__ CUtensorMap out_map,
                        const __grid_constant__ DecodeArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_side_mem[kDecWarps][kDecTileBuffers];

    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31u;
    grid_dependency_launch_next();

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t tiles = smem_base + warp * (uint32_t)(kDecTileBuffers * kDecTileBytes);
    const uint32_t bar_side = smem_u32(&bar_side_mem[warp][0]);
    const bool side_tiles = SIDE == kSideGiven && args.has_side != 0u && args.use_tiles != 0u;

    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kDecTileBuffers; ++i) mbar_init(bar_side + 8u * i, 1u);
        fence_mbar_init();
        if (args.use_tiles) asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&out_map) : "memory");
        if (side_tiles) asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&side_map) : "memory");
    }
    // the messages (and the side information) may be the previous kernel's output
    grid_dependency_wait();

    // Work: a team-unit is kDecTeamWarps adjacent units (32 rows each), one per warp of a team.  CTA c owns the
    // team-units c, c + gridDim.x, ...; its teams draw them from a counter in shared memory, one ahead of the
    // one they work on, so a team that the schedulers favour simply takes more of them and all teams of an SM
    // finish within one unit of each other.  The warps of a team meet before each unit, so that they run through
    // the same code at about the same time (teams of one to four warps measure alike, larger ones are slower).
    __shared__ uint32_t draw_count;
    __shared__ uint32_t drawn[kDecTeams][2];
    const uint32_t team = warp / (uint32_t)kDecTeamWarps;
    const uint32_t tw = warp % (uint32_t)kDecTeamWarps;
    const uint32_t num_tunits = (args.num_units + (uint32_t)kDecTeamWarps - 1u) / (uint32_t)kDecTeamWarps;
    const uint32_t cta_tunits = (blockIdx.x < num_tunits) ? (num_tunits - blockIdx.x - 1u) / gridDim.x + 1u : 0u;
    auto team_meet = [&]() {
        if constexpr (kDecTeams == 1) __syncthreads();
        else if constexpr (kDecTeamWarps == 1) __syncwarp();
        else asm volatile("bar.sync %0, %1;" ::"r"(team + 1u), "n"(kDecTeamWarps * 32) : "memory");
    };
    // unit of this warp in the CTA's j-th team-unit (>= num_units: none)
    auto unit_of = [&](uint32_t j) {
        return (j < cta_tunits) ? (blockIdx.x + j * gridDim.x) * (uint32_t)kDecTeamWarps + tw : 0xFFFFFFFFu;
    };
    if (threadIdx.x == 0) draw_count = 0u;
    __syncthreads();
    if (tw == 0u && lane == 0u) drawn[team][0] = atomicAdd(&draw_count, 1u);
    team_meet();
    uint32_t unit = unit_of(drawn[team][0]);
    const uint32_t whole_rows = args.full_rows - args.first_row;       // rows of the tile maps

    // side information of unit `u` -> tile buffer `b` (lane 0)
    auto issue_side = [&](uint32_t u, uint32_t b) {
        if (u * 32u >= whole_rows) return;                              // a unit that is only the ragged last row
        mbar_expect_tx(bar_side + 8u * b, (uint32_t)kDecTileBytes);
        tma_load_rows(tiles + b * (uint32_t)kDecTileBytes, &side_map, bar_side + 8u * b, (int32_t)(u * 32u));
    };
    // Ask the L2 for every worker's packed words of the unit that starts at row `row0`: lane w (and w + 32)
    // requests the 128-byte lines of worker w, whose words of a unit are 128 * bits contiguous bytes.
    auto prefetch_words = [&](uint32_t row0) {
        if (row0 >= args.full_rows) return;
        for (uint32_t w = lane; w < args.W; w += 32u) {
            const uint32_t* p = args.w[w].packed + (uint64_t)row0 * args.w[w].bits;
            const uint32_t rows_left = args.full_rows - row0;
            const uint32_t lines = (rows_left >= 32u) ? args.w[w].bits : (rows_left * args.w[w].bits + 31u) / 32u;
            for (uint32_t l = 0; l < lines; ++l) prefetch_l2(p + 32u * l);
        }
    };
    if (lane == 0 && side_tiles && unit < args.num_units) issue_side(unit, 0u);
    __syncwarp();

    // bucket of a row (rows past the end take the last row's bucket: their results are never stored)
    auto bucket_of = [&](uint32_t r) {
        const uint32_t rc = (r < args.rows) ? r : args.rows - 1u;
        return (args.rpb_shift != 0xFFFFFFFFu) ? (rc >> args.rpb_shift) : (rc / args.rows_per_bucket);
    };

    // The ragged last row goes first, on the warp that tends to have the least to do: left to the end of the
    // unit that contains it, its serial chains would be what the whole grid waits for.
    if (args.full_rows < args.rows && blockIdx.x == gridDim.x - 1u && warp == (uint32_t)kDecWarps - 1u)
        decode_partial_row<DITH, SIDE>(args, args.full_rows, bucket_of(args.full_rows),
                                       (uint32_t)(args.n - (uint64_t)args.full_rows * 32u), lane);

    const uint32_t swz16 = (lane & 7u) << 4;
    bool gave_up = false;
    uint32_t bucket = bucket_of(args.first_row + (unit < args.num_units ? unit : 0u) * 32u + lane);
    float kappa_next = __ldg(args.w[0].scale + bucket);

#pragma unroll 1
    for (uint32_t it = 0; unit != 0xFFFFFFFFu; ++it) {
        // draw the next team-unit, then meet: everyone has read the previous draw before the one after this
        if (tw == 0u && lane == 0u) drawn[team][(it + 1u) & 1u] = atomicAdd(&draw_count, 1u);
        team_meet();
        const uint32_t unit_next = unit_of(drawn[team][(it + 1u) & 1u]);
        if (unit >= args.num_units) { unit = unit_next; continue; }    // past the end (last team-unit only)
        const uint32_t row = args.first_row + unit * 32u + lane;
        const uint32_t b = it % (uint32_t)kDecTileBuffers;
        const uint32_t tile = tiles + b * (uint32_t)kDecTileBytes;
        const bool more = unit_next < args.num_units;
        const uint32_t bucket_next = more ? bucket_of(args.first_row + unit_next * 32u + lane) : bucket;
        if (more) prefetch_words(args.first_row + unit_next * 32u);
        if (lane == 0) {
            // the store issued two units ago has read its buffer: that buffer takes the next unit's side
            // information now and this unit's output later
            bulk_wait_group_read<1>();
            if (side_tiles && more) issue_side(unit_next, (it + 1u) % (uint32_t)kDecTileBuffers);
        }
        __syncwarp();
        const bool unit_has_tile = unit * 32u < whole_rows;
        if (side_tiles && unit_has_tile &&
            !mbar_wait_bounded(bar_side + 8u * b, (it / (uint32_t)kDecTileBuffers) & 1u, gave_up)) {
            gave_up = true;
            if (lane == 0) atomicOr(args.error_flags, 0x2u);
        }
        const uint32_t row_addr = (tile + lane * 128u) | swz16;
        // lanes past the last whole row compute on the last whole row's words (in bounds) and are never stored
        const uint32_t load_row = (row < args.full_rows) ? row : args.full_rows - 1u;

        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.0f;
        DecLane ln;
        ln.row = row; ln.load_row = load_row; ln.bucket = bucket; ln.bucket_next = bucket_next;
        ln.row_addr = row_addr; ln.kappa_bits_max = 0u; ln.kappa_next = kappa_next;
        if (unit_has_tile) {
            decode_workers<DITH, SIDE>(args, ln, acc);
            kappa_next = ln.kappa_next;
        } else {
            kappa_next = __ldg(args.w[0].scale + bucket_next);
        }
        const uint32_t kappa_bits_max = ln.kappa_bits_max;
        bucket = bucket_next;

        // the mean leaves through the tile buffer: the lane writes its row where it read its side information
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
                v[e] = (args.W == 1u)        ? acc[4 * c + e]                       // the mean of one message is itself
                       : (args.invW != 0.0f) ? __fmul_rn(acc[4 * c + e], args.invW)
                                             : __fdiv_rn(acc[4 * c + e], args.Wf);
            asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};"
                         ::"r"(row_addr ^ (uint32_t)(c << 4)), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3])
                         : "memory");
        }
        fence_proxy_async_shared();
        __syncwarp();
        if (lane == 0 && unit_has_tile) {
            tma_store_rows(&out_map, tile, (int32_t)(unit * 32u));
            bulk_commit_group();
        }
        if (args.status != nullptr && kappa_bits_max >= 0x7F800000u && row < args.full_rows) atomicOr(args.status, 0x1u);
        unit = unit_next;
    }
    // shared memory must stay valid until the last stores have read it
    if (lane == 0) bulk_wait_group_read<0>();
}

}  // namespace dq
