// Host side of the C ABI declared in include/dq.h: argument checks, tensor-map set-up, kernel launches.
// Everything numerical happens in the kernels of dq_encode.cuh / dq_decode.cuh.
#include "dq.h"

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <utility>

#include "dq_decode.cuh"
#include "dq_encode.cuh"
#include "dq_launch.h"
#include "dq_stats.cuh"
#include "dq_ternary.cuh"

// The device's error word: kernels OR DQ_ERR_* bits into it through the address they are given.  In host code
// the name is a handle for the runtime, not an address.
static __device__ unsigned int g_dq_error_flags = 0u;

namespace {

using dq::launch_overlapped;

std::atomic<uint64_t> g_launches{0};

bool is_pow2(uint32_t v) { return v && !(v & (v - 1u)); }

// Address of element 0 of the virtual whole-gradient array whose element `first` is p[0] (integer arithmetic: the
// result may lie outside any allocation and is only ever used with indices >= first).
template <typename T>
T* virtual_base(T* p, uint64_t first)
{
    return reinterpret_cast<T*>(reinterpret_cast<uintptr_t>(p) - first * sizeof(T));
}
bool float_is_pow2(float v)
{
    uint32_t u;
    std::memcpy(&u, &v, sizeof(u));
    return v > 0.0f && (u & 0x007FFFFFu) == 0u && (u >> 23) != 0u && (u >> 23) != 0xFFu;
}
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0u; }

void fill_philox(dq::PhiloxStream& ps, uint64_t seed, uint32_t worker, uint64_t step)
{
    uint32_t k0 = (uint32_t)(seed & 0xFFFFFFFFull), k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        ps.rk[r][0] = k0;
        ps.rk[r][1] = k1;
        k0 += dq::kPhiloxW0;
        k1 += dq::kPhiloxW1;
    }
    ps.c1 = worker;
    ps.c2 = (uint32_t)(step & 0xFFFFFFFFull);
    ps.c3 = (uint32_t)(step >> 32);
    // the block-independent parts of rounds 0..2 (see PhiloxStream)
    const uint64_t p1 = (uint64_t)dq::kPhiloxM1 * (uint64_t)ps.c2;
    const uint32_t u0 = (uint32_t)(p1 >> 32) ^ ps.c1 ^ ps.rk[0][0];
    const uint32_t u1 = (uint32_t)p1;
    const uint64_t p0 = (uint64_t)dq::kPhiloxM0 * (uint64_t)u0;
    ps.v0 = ps.c3 ^ ps.rk[0][1];
    ps.v1 = u1 ^ ps.rk[1][0];
    ps.v2 = (uint32_t)(p0 >> 32) ^ ps.rk[1][1];
    ps.v3 = (uint32_t)p0 ^ ps.rk[2][1];
}

int device_sm_count()
{
    static thread_local int cached_dev = -1, cached_sms = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev != cached_dev) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached_dev = dev;
        cached_sms = sms;
    }
    return cached_sms;
}

dq_status check_params(const dq_params* p, dq_kind kind, uint32_t* levels_out, float* alpha_out)
{
    if (!p) return DQ_ERR_INVALID_ARG;
    if (p->bucket < 32u || p->bucket > 65536u || (p->bucket % 32u) != 0u) return DQ_ERR_INVALID_ARG;
    if (p->bits < 1u || p->bits > 8u) return DQ_ERR_INVALID_ARG;
    if (p->dither_bits != 0u && p->dither_bits != 32u && p->dither_bits != 16u) return DQ_ERR_INVALID_ARG;
    if (kind == DQ_KIND_DQSG) {
        const uint32_t L = p->levels ? p->levels : dq_default_levels(p->bits);
        if (L < 2u || L > (1u << p->bits)) return DQ_ERR_INVALID_ARG;
        *levels_out = L;
        *alpha_out = 1.0f;
    } else if (kind == DQ_KIND_NDQSG) {
        const float alpha = (p->alpha == 0.0f) ? 1.0f : p->alpha;
        if (p->coarse_K < 2u || p->coarse_K > (1u << p->bits)) return DQ_ERR_INVALID_ARG;
        if (!(p->fine_M > 0.0f) || !(alpha > 0.0f) || alpha > 1.0f) return DQ_ERR_INVALID_ARG;
        const float A = alpha * p->fine_M;
        if (!(A > 0.0f)) return DQ_ERR_INVALID_ARG;
        if (A > 1048576.0f) return DQ_ERR_UNSUPPORTED;
        *levels_out = 0u;
        *alpha_out = alpha;
    } else {
        return DQ_ERR_INVALID_ARG;
    }
    return DQ_OK;
}

// cuTensorMapEncodeTiled, looked up at run time so the library loads on machines without a driver.
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_tiled()
{
    static encode_tiled_fn fn = []() -> encode_tiled_fn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<encode_tiled_fn>(p);
    }();
    return fn;
}

// [rows x 32 fp32] view of a flat vector, boxes of `box_rows` rows, 128-byte swizzle.
bool make_row_map(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows)
{
    encode_tiled_fn fn = get_encode_tiled();
    if (!fn) return false;
    const cuuint64_t dims[2] = {32u, rows};
    const cuuint64_t strides[1] = {128u};
    const cuuint32_t box[2] = {32u, box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2u, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kMaxDevices = 64;

// Device address of g_dq_error_flags on the current device; looked up once per device.
unsigned int* error_flags_address()
{
    static std::mutex mu;
    static unsigned int* addr[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_dq_error_flags) != cudaSuccess) return nullptr;
        addr[dev] = static_cast<unsigned int*>(ptr);
    }
    return addr[dev];
}

cudaError_t launch_encode(int mode, uint32_t bits, bool dither16, const CUtensorMap& map, const dq::EncodeArgs& a,
                          uint32_t grid, cudaStream_t st)
{
    switch (mode * 2 + (dither16 ? 1 : 0)) {
        case 0: return dq::launch_encode_m0_d32(bits, map, a, grid, st);
        case 1: return dq::launch_encode_m0_d16(bits, map, a, grid, st);
        case 2: return dq::launch_encode_m1_d32(bits, map, a, grid, st);
        case 3: return dq::launch_encode_m1_d16(bits, map, a, grid, st);
        case 4: return dq::launch_encode_m2_d32(bits, map, a, grid, st);
        case 5: return dq::launch_encode_m2_d16(bits, map, a, grid, st);
        case 6: return dq::launch_encode_m3_d32(bits, map, a, grid, st);
        default: return dq::launch_encode_m3_d16(bits, map, a, grid, st);
    }
}

dq_status encode_common(dq_kind kind, const float* grad, uint64_t n, uint64_t seed, uint32_t worker,
                        uint64_t step, const dq_params* p, uint32_t* out_packed, float* out_scale,
                        cudaStream_t st, uint64_t first_element = 0u)
{
    uint32_t L = 0;
    float alpha = 1.0f;
    dq_status s = check_params(p, kind, &L, &alpha);
    if (s != DQ_OK) return s;
    if (first_element % p->bucket != 0u) return DQ_ERR_INVALID_ARG;      // a range starts at a bucket boundary
    if (n == 0) return DQ_OK;
    if (n >= (1ull << 34) || first_element >= (1ull << 34) || first_element + n >= (1ull << 34))
        return DQ_ERR_UNSUPPORTED;
    if (!grad || !out_packed || !out_scale) return DQ_ERR_INVALID_ARG;
    if (!aligned16(grad) || !aligned16(out_packed) || !aligned16(out_scale)) return DQ_ERR_ALIGNMENT;

    dq::EncodeArgs a;
    std::memset(&a, 0, sizeof(a));
    a.grad = grad;
    a.packed = out_packed;
    a.scale = out_scale;
    a.n = n;
    a.row_offset = (uint32_t)(first_element / 32u);
    a.bucket = p->bucket;
    a.num_buckets = dq_num_buckets(n, p->bucket);
    a.num_words = dq_packed_words(n, p->bits);
    int mode;
    if (kind == DQ_KIND_DQSG) {
        mode = dq::kEncDqsg;
        a.shift = (float)(L - 1u) / 2.0f;
        a.gain_num = a.shift;
        a.kmax = (float)(L - 1u);
    } else {
        // K = 2^bits: the coset is the low `bits` bits of the fine index; a smaller power of two: one mask more;
        // any other K: a modulo
        mode = (p->coarse_K == (1u << p->bits)) ? dq::kEncNdqsgPow2
               : is_pow2(p->coarse_K)           ? dq::kEncNdqsgPow2Mask
                                                : dq::kEncNdqsgAnyK;
        a.gain_num = alpha * p->fine_M;
        a.K = p->coarse_K;
        a.K_offset = ((4194304u + p->coarse_K - 1u) / p->coarse_K) * p->coarse_K;
    }
    fill_philox(a.ps, seed, worker, step);
    a.early_read = (p->flags & DQ_FLAG_INPUT_READY) ? 1u : 0u;
    a.early_store = (a.early_read && (p->flags & DQ_FLAG_OUTPUT_FREE)) ? 1u : 0u;
    a.test_drop_copy = (p->flags & DQ_FLAG_TEST_DROP_COPY) ? 1u : 0u;
    a.error_flags = error_flags_address();
    if (!a.error_flags) return DQ_ERR_CUDA;

    // power-of-two buckets up to 8192: whole work units (a bucket, or 1024 elements for smaller buckets) go
    // through the tile path of the kernel, the rest (and every other bucket size) through its plain-load part,
    // in the same launch
    const int sms = device_sm_count();
    if (sms <= 0) return DQ_ERR_CUDA;
    a.sm_count = (uint32_t)sms;
    const uint32_t B = p->bucket;
    const uint32_t U = (B < 1024u) ? 1024u : B;                     // elements per work unit
    uint64_t tiles = (is_pow2(B) && B <= 8192u) ? n / U : 0u;       // whole units
    if (tiles > 0xFFFFFFFFull) return DQ_ERR_UNSUPPORTED;
    CUtensorMap map;
    std::memset(&map, 0, sizeof(map));
    const bool pair = (B == 2048u || B == 4096u || B == 8192u);     // a warp takes 2048 elements, two halves in time
    const uint32_t wpb = pair ? (B / 2048u) : (B < 1024u) ? 1u : (B / 1024u);
    a.pair_in_time = pair ? 1u : 0u;
    if (tiles > 0) {
        if (!make_row_map(&map, grad, tiles * (U / 32u), 32u)) return DQ_ERR_CUDA;
        a.num_units = (uint32_t)tiles;
        a.lanes_per_bucket = (B < 1024u) ? (B / 32u) : 32u;
        a.warps_per_bucket = wpb;
        uint32_t lg = 0;
        while ((1u << lg) < B) ++lg;
        a.bucket_log2 = lg;
    }
    a.first_bucket = tiles * (U / B);
    const uint64_t rest = a.num_buckets - a.first_bucket;
    const uint32_t slots = (uint32_t)dq::kEncCtasPerSm * (uint32_t)sms;   // resident CTAs
    uint32_t plain = 0;
    if (rest > 0) {
        // buckets of at most 32 rows: a warp takes a window of whole buckets; up to 128 rows: a warp per bucket;
        // larger ones: a CTA per bucket
        uint64_t want = rest;
        if (B <= 1024u) {
            const uint64_t rpb = B / 32u, rows_per_window = (32u / rpb) * rpb;
            const uint64_t rest_rows = (n + 31u) / 32u - a.first_bucket * rpb;
            a.plain_windows = (rest_rows + rows_per_window - 1u) / rows_per_window;
            want = (a.plain_windows + dq::kConsumerWarps - 1u) / dq::kConsumerWarps;
        } else if (B <= dq::kPlainWarpBucketMax) {
            want = (rest + dq::kConsumerWarps - 1u) / dq::kConsumerWarps;           // a warp per bucket
        }
        const uint64_t cap = (tiles > 0) ? (slots / 4u) : (4ull * slots);
        plain = (uint32_t)(want < cap ? want : cap);
        if (plain == 0u) plain = 1u;
    }
    a.plain_ctas = plain;
    uint32_t tile_ctas = 0;
    if (tiles > 0) {
        const uint32_t room = (slots > plain) ? (slots - plain) : 1u;
        const uint64_t groups_per_cta = (uint64_t)dq::kConsumerWarps / wpb;
        const uint64_t want_ctas = (tiles + groups_per_cta - 1u) / groups_per_cta;
        tile_ctas = (uint32_t)(want_ctas < room ? want_ctas : room);
    }
    // the spacing only pays when the first requests of all resident warps saturate HBM
    // (a launch that reads early gets its CTAs one by one, as the previous kernel's CTAs leave: nothing to space)
    a.request_spacing_ns = a.early_read ? 0u : (uint32_t)((uint64_t)dq::kFirstRequestSpacingNs * tile_ctas / slots);
    const bool d16 = (p->dither_bits == 16u);
    if (launch_encode(mode, p->bits, d16, map, a, plain + tile_ctas, st) != cudaSuccess) return DQ_ERR_CUDA;
    g_launches.fetch_add(1);
    return DQ_OK;
}

dq_status decode_common(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step, const float* side_info,
                        float* out_avg, uint32_t* status_word, bool allow_nested, cudaStream_t st,
                        bool running = false, bool half_dithered = false, uint64_t first_element = 0u,
                        bool side_first = false)
{
    if (!msgs || W == 0u || W > DQ_MAX_WORKERS) return DQ_ERR_INVALID_ARG;
    static thread_local dq::DecodeArgs a;    // ~10 KB: keep it off the stack
    std::memset(&a, 0, sizeof(a));
    bool any_nested = false;
    for (uint32_t w = 0; w < W; ++w) {
        const dq_msg& m = msgs[w];
        uint32_t L = 0;
        float alpha = 1.0f;
        dq_status s = check_params(&m.p, m.kind, &L, &alpha);
        if (s != DQ_OK) return s;
        if (m.kind == DQ_KIND_NDQSG && !allow_nested) return DQ_ERR_INVALID_ARG;
        if (m.p.bucket != msgs[0].p.bucket) return DQ_ERR_UNSUPPORTED;
        if (!half_dithered && (m.p.dither_bits == 16u) != (msgs[0].p.dither_bits == 16u)) return DQ_ERR_UNSUPPORTED;
        dq::DecWorker& d = a.w[w];
        // addresses of the (virtual) whole-gradient buffers: see DecodeArgs
        d.packed = virtual_base(m.packed, first_element / 32u * m.p.bits);
        d.scale = virtual_base(m.scale, first_element / m.p.bucket);
        d.unit_lines = m.p.bits;
        fill_philox(d.ps, m.seed, m.worker, step);
        d.bits = m.p.bits;
        uint32_t kind;
        if (m.kind == DQ_KIND_DQSG) {
            kind = dq::kDecDqsg;
            d.s = (float)(L - 1u) / 2.0f;
            d.cconst = 4194304.0f + d.s - 1.5f;
            d.step_mul = is_pow2(L - 1u) && L >= 3u ? 2.0f / (float)(L - 1u) : (L == 2u ? 2.0f : 0.0f);
        } else {
            any_nested = true;
            if (!is_pow2(m.p.coarse_K)) kind = dq::kDecNdqsgAnyK;
            else kind = (alpha == 1.0f) ? dq::kDecNdqsgPow2 : dq::kDecNdqsgPow2Shrink;
            d.cconst = 4194304.0f - 1.5f;
            d.A = alpha * m.p.fine_M;
            d.M1 = m.p.fine_M;
            d.alpha = alpha;
            const float a2 = alpha * alpha;
            d.one_m_alpha2 = 1.0f - a2;
            d.Kf = (float)m.p.coarse_K;
            d.invK = 1.0f / d.Kf;
            d.step_mul = float_is_pow2(m.p.fine_M) ? 1.0f / m.p.fine_M : 0.0f;
            if (running) {
                if (w == 0u) return DQ_ERR_INVALID_ARG;      // nothing decoded yet to serve as side information
                d.rcp_count = 1.0f / (float)w;
            }
        }
        d.variant = kind * 8u + m.p.bits - 1u;
    }
    // runs of equal variants (one routine per run, see decode_workers)
    for (uint32_t w = W; w-- > 0u;)
        a.w[w].group_end = (w + 1u < W && a.w[w + 1u].variant == a.w[w].variant) ? a.w[w + 1u].group_end : w + 1u;
    if (first_element % msgs[0].p.bucket != 0u) return DQ_ERR_INVALID_ARG;   // a range starts at a bucket boundary
    if (n == 0) return DQ_OK;
    if (n >= (1ull << 34) || first_element >= (1ull << 34) || first_element + n >= (1ull << 34))
        return DQ_ERR_UNSUPPORTED;
    if (!out_avg) return DQ_ERR_INVALID_ARG;
    if (side_first && msgs[0].kind != DQ_KIND_DQSG) return DQ_ERR_INVALID_ARG;   // message 0 is decoded on its own
    if (any_nested && !running && !side_first && !side_info) return DQ_ERR_INVALID_ARG;
    if (!aligned16(out_avg) || (side_info && !aligned16(side_info))) return DQ_ERR_ALIGNMENT;
    for (uint32_t w = 0; w < W; ++w) {
        if (!msgs[w].packed || !msgs[w].scale) return DQ_ERR_INVALID_ARG;
        if (!aligned16(msgs[w].packed) || !aligned16(msgs[w].scale)) return DQ_ERR_ALIGNMENT;
    }
    const bool reads_side = any_nested && !running && !side_first;
    const bool from_first = any_nested && !running && side_first;
    a.side = reads_side ? virtual_base(side_info, first_element) : nullptr;
    a.out = virtual_base(out_avg, first_element);
    a.status = status_word;
    a.n = first_element + n;
    a.rows = (uint32_t)((first_element + n + 31u) / 32u);
    a.first_row = (uint32_t)(first_element / 32u);
    a.full_rows = (uint32_t)((first_element + n) / 32u);
    a.num_units = (a.rows - a.first_row + 31u) / 32u;
    a.W = W;
    a.rows_per_bucket = msgs[0].p.bucket / 32u;
    a.rpb_shift = 0xFFFFFFFFu;
    if (is_pow2(a.rows_per_bucket)) {
        a.rpb_shift = 0u;
        while ((1u << a.rpb_shift) < a.rows_per_bucket) ++a.rpb_shift;
    }
    a.has_side = reads_side ? 1u : 0u;
    a.half_bias_bits = 0x4A800000u;
    a.Wf = (float)W;
    a.invW = is_pow2(W) ? 1.0f / (float)W : 0.0f;
    a.error_flags = error_flags_address();
    if (!a.error_flags) return DQ_ERR_CUDA;
    // tile views of the caller's buffers: whole rows only (a ragged last row is handled with plain accesses)
    CUtensorMap side_map, out_map;
    std::memset(&side_map, 0, sizeof(side_map));
    std::memset(&out_map, 0, sizeof(out_map));
    const uint32_t whole_rows = a.full_rows - a.first_row;
    a.use_tiles = whole_rows != 0u ? 1u : 0u;
    if (whole_rows != 0u) {
        if (!make_row_map(&out_map, out_avg, whole_rows, 32u)) return DQ_ERR_CUDA;
        if (reads_side && !make_row_map(&side_map, side_info, whole_rows, 32u)) return DQ_ERR_CUDA;
    }
    const int sms = device_sm_count();
    if (sms <= 0) return DQ_ERR_CUDA;
    const bool d16 = (msgs[0].p.dither_bits == 16u);
    cudaError_t le;
    if (half_dithered) le = dq::launch_decode_d0_r0(side_map, out_map, a, sms, st);
    else if (running && any_nested) le = d16 ? dq::launch_decode_d16_r1(side_map, out_map, a, sms, st)
                                             : dq::launch_decode_d32_r1(side_map, out_map, a, sms, st);
    else if (from_first) le = d16 ? dq::launch_decode_d16_r2(side_map, out_map, a, sms, st)
                                  : dq::launch_decode_d32_r2(side_map, out_map, a, sms, st);
    else le = d16 ? dq::launch_decode_d16_r0(side_map, out_map, a, sms, st)
                  : dq::launch_decode_d32_r0(side_map, out_map, a, sms, st);
    if (le != cudaSuccess) return DQ_ERR_CUDA;
    g_launches.fetch_add(1);
    return DQ_OK;
}

uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1u) / a * a; }

}  // namespace

extern "C" {

uint64_t dq_packed_words(uint64_t n, uint32_t bits) { return (n * (uint64_t)bits + 31u) / 32u; }
uint64_t dq_num_buckets(uint64_t n, uint32_t bucket) { return bucket ? (n + bucket - 1u) / bucket : 0u; }
uint32_t dq_default_levels(uint32_t bits) { return bits == 1u ? 2u : (1u << bits) - 1u; }

const char* dq_status_string(dq_status s)
{
    switch (s) {
        case DQ_OK: return "ok";
        case DQ_ERR_INVALID_ARG: return "invalid argument";
        case DQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case DQ_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case DQ_ERR_CUDA: return "CUDA call failed";
        case DQ_ERR_TOO_LARGE: return "input larger than the built-in scratch buffer";
    }
    return "unknown status";
}

dq_status dqsg_encode(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                      const dq_params* p, uint32_t* out_packed, float* out_scale, void* cuda_stream)
{
    return encode_common(DQ_KIND_DQSG, grad, n, seed, worker, step, p, out_packed, out_scale,
                         static_cast<cudaStream_t>(cuda_stream));
}

dq_status ndqsg_encode(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                       const dq_params* p, uint32_t* out_packed, float* out_scale, void* cuda_stream)
{
    return encode_common(DQ_KIND_NDQSG, grad, n, seed, worker, step, p, out_packed, out_scale,
                         static_cast<cudaStream_t>(cuda_stream));
}

dq_status dqsg_decode_aggregate(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step, float* out_avg,
                                void* cuda_stream)
{
    return decode_common(msgs, W, n, step, nullptr, out_avg, nullptr, false, static_cast<cudaStream_t>(cuda_stream));
}

dq_status ndqsg_decode_aggregate(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                 const float* side_info, float* out_avg, uint32_t* status_word, void* cuda_stream)
{
    return decode_common(msgs, W, n, step, side_info, out_avg, status_word, true,
                         static_cast<cudaStream_t>(cuda_stream));
}

dq_status ndqsg_decode_aggregate_side_first(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step, float* out_avg,
                                            uint32_t* status_word, void* cuda_stream)
{
    return decode_common(msgs, W, n, step, nullptr, out_avg, status_word, true,
                         static_cast<cudaStream_t>(cuda_stream), false, false, 0u, true);
}

dq_status dqsg_decode_aggregate_half_dithered(const dq_msg* msgs, uint32_t W, uint64_t n, float* out_avg,
                                              void* cuda_stream)
{
    return decode_common(msgs, W, n, 0u, nullptr, out_avg, nullptr, false, static_cast<cudaStream_t>(cuda_stream),
                         false, true);
}

dq_status ndqsg_decode_aggregate_running(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step, float* out_avg,
                                         uint32_t* status_word, void* cuda_stream)
{
    return decode_common(msgs, W, n, step, nullptr, out_avg, status_word, true,
                         static_cast<cudaStream_t>(cuda_stream), true);
}

// ------------------------------------------------------------------------------------------------ bucket ranges
dq_status dqsg_encode_range(const float* grad, uint64_t n, uint64_t first_element, uint64_t seed, uint32_t worker,
                            uint64_t step, const dq_params* p, uint32_t* out_packed, float* out_scale,
                            void* cuda_stream)
{
    return encode_common(DQ_KIND_DQSG, grad, n, seed, worker, step, p, out_packed, out_scale,
                         static_cast<cudaStream_t>(cuda_stream), first_element);
}

dq_status ndqsg_encode_range(const float* grad, uint64_t n, uint64_t first_element, uint64_t seed, uint32_t worker,
                             uint64_t step, const dq_params* p, uint32_t* out_packed, float* out_scale,
                             void* cuda_stream)
{
    return encode_common(DQ_KIND_NDQSG, grad, n, seed, worker, step, p, out_packed, out_scale,
                         static_cast<cudaStream_t>(cuda_stream), first_element);
}

dq_status ndqsg_decode_aggregate_range(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t first_element,
                                       uint64_t step, const float* side_info, float* out_avg,
                                       uint32_t* status_word, void* cuda_stream)
{
    return decode_common(msgs, W, n, step, side_info, out_avg, status_word, true,
                         static_cast<cudaStream_t>(cuda_stream), false, false, first_element);
}

dq_status dq_code_histogram(const uint32_t* packed, uint64_t n, uint32_t bits, uint64_t* hist, void* cuda_stream)
{
    if (bits < 1u || bits > 8u) return DQ_ERR_INVALID_ARG;
    if (!hist) return DQ_ERR_INVALID_ARG;
    if (n >= (1ull << 34)) return DQ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(hist, 0, sizeof(uint64_t) << bits, st) != cudaSuccess) return DQ_ERR_CUDA;
    if (n == 0) return DQ_OK;
    if (!packed) return DQ_ERR_INVALID_ARG;
    if (!aligned16(packed) || (reinterpret_cast<uintptr_t>(hist) & 7u) != 0u) return DQ_ERR_ALIGNMENT;
    const int sms = device_sm_count();
    if (sms <= 0) return DQ_ERR_CUDA;
    const uint64_t rows = (n + 31u) / 32u;
    uint64_t grid = (rows + dq::kHistThreads - 1u) / dq::kHistThreads;
    if (grid > (uint64_t)sms * 8u) grid = (uint64_t)sms * 8u;
    static_assert(sizeof(unsigned long long) == sizeof(uint64_t), "histogram counters are 64-bit");
    if (launch_overlapped(dq::code_histogram_kernel, (uint32_t)grid, (uint32_t)dq::kHistThreads, 0, st, packed, n,
                          bits, reinterpret_cast<unsigned long long*>(hist)) != cudaSuccess)
        return DQ_ERR_CUDA;
    g_launches.fetch_add(1);
    return DQ_OK;
}

dq_status dq_code_entropy(const uint64_t* hist_host, uint32_t bits, double* out_bits_per_element)
{
    if (!hist_host || !out_bits_per_element || bits < 1u || bits > 8u) return DQ_ERR_INVALID_ARG;
    long double total = 0.0L;
    for (uint32_t c = 0; c < (1u << bits); ++c) total += (long double)hist_host[c];
    long double h = 0.0L;
    if (total > 0.0L) {
        for (uint32_t c = 0; c < (1u << bits); ++c) {
            if (hist_host[c] == 0u) continue;
            const long double pc = (long double)hist_host[c] / total;
            h -= pc * log2l(pc);
        }
    }
    *out_bits_per_element = (double)h;
    return DQ_OK;
}

// ------------------------------------------------------------------------------------------------ radix-3 container
uint64_t dq_ternary_bytes(uint64_t n) { return (n + 4u) / 5u; }

static_assert(dq::kWarnCodeRange == DQ_WARN_CODE_RANGE, "status bit of the container kernels");

dq_status dq_ternary_pack(const uint32_t* packed, uint64_t n, uint8_t* out_radix, uint32_t* status_word,
                          void* cuda_stream)
{
    if (n >= (1ull << 34)) return DQ_ERR_UNSUPPORTED;
    if (n == 0) return DQ_OK;
    if (!packed || !out_radix) return DQ_ERR_INVALID_ARG;
    if (!aligned16(packed) || !aligned16(out_radix)) return DQ_ERR_ALIGNMENT;
    const uint64_t units = (n + 79u) / 80u;
    const uint64_t grid = (units + dq::kTernaryThreads - 1u) / dq::kTernaryThreads;
    if (launch_overlapped(dq::ternary_pack_kernel, (uint32_t)grid, (uint32_t)dq::kTernaryThreads, 0,
                          static_cast<cudaStream_t>(cuda_stream), packed, n, out_radix, status_word) != cudaSuccess)
        return DQ_ERR_CUDA;
    g_launches.fetch_add(1);
    return DQ_OK;
}

dq_status dq_ternary_unpack(const uint8_t* radix, uint64_t n, uint32_t* out_packed, void* cuda_stream)
{
    if (n >= (1ull << 34)) return DQ_ERR_UNSUPPORTED;
    if (n == 0) return DQ_OK;
    if (!radix || !out_packed) return DQ_ERR_INVALID_ARG;
    if (!aligned16(radix) || !aligned16(out_packed)) return DQ_ERR_ALIGNMENT;
    const uint64_t units = (n + 79u) / 80u;
    const uint64_t grid = (units + dq::kTernaryThreads - 1u) / dq::kTernaryThreads;
    if (launch_overlapped(dq::ternary_unpack_kernel, (uint32_t)grid, (uint32_t)dq::kTernaryThreads, 0,
                          static_cast<cudaStream_t>(cuda_stream), radix, n, out_packed) != cudaSuccess)
        return DQ_ERR_CUDA;
    g_launches.fetch_add(1);
    return DQ_OK;
}

// ------------------------------------------------------------------------------------------------ host buffers
uint64_t dq_encode_workspace_bytes(uint64_t n, const dq_params* p)
{
    if (!p || p->bucket == 0u) return 0u;
    return align_up(n * 4u, 256u) + align_up(dq_packed_words(n, p->bits) * 4u, 256u) +
           align_up(dq_num_buckets(n, p->bucket) * 4u, 256u);
}

uint64_t dq_decode_workspace_bytes(const dq_msg* msgs, uint32_t W, uint64_t n, int has_side_info)
{
    if (!msgs) return 0u;
    uint64_t total = align_up(n * 4u, 256u) * (has_side_info ? 2u : 1u);
    for (uint32_t w = 0; w < W; ++w) {
        if (msgs[w].p.bucket == 0u) return 0u;
        total += align_up(dq_packed_words(n, msgs[w].p.bits) * 4u, 256u) +
                 align_up(dq_num_buckets(n, msgs[w].p.bucket) * 4u, 256u);
    }
    return total;
}

static dq_status encode_host(dq_kind kind, const float* grad, uint64_t n, uint64_t seed, uint32_t worker,
                             uint64_t step, const dq_params* p, uint32_t* out_packed, float* out_scale,
                             void* workspace, uint64_t workspace_bytes, void* cuda_stream)
{
    uint32_t L;
    float alpha;
    dq_status s = check_params(p, kind, &L, &alpha);
    if (s != DQ_OK) return s;
    if (n == 0) return DQ_OK;
    if (n >= (1ull << 34)) return DQ_ERR_UNSUPPORTED;
    if (!grad || !out_packed || !out_scale || !workspace) return DQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0u) return DQ_ERR_ALIGNMENT;
    if (workspace_bytes < dq_encode_workspace_bytes(n, p)) return DQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    float* d_grad = reinterpret_cast<float*>(ws);
    ws += align_up(n * 4u, 256u);
    uint32_t* d_packed = reinterpret_cast<uint32_t*>(ws);
    const uint64_t pbytes = dq_packed_words(n, p->bits) * 4u;
    ws += align_up(pbytes, 256u);
    float* d_scale = reinterpret_cast<float*>(ws);
    const uint64_t sbytes = dq_num_buckets(n, p->bucket) * 4u;
    if (cudaMemcpyAsync(d_grad, grad, n * 4u, cudaMemcpyHostToDevice, st) != cudaSuccess) return DQ_ERR_CUDA;
    s = encode_common(kind, d_grad, n, seed, worker, step, p, d_packed, d_scale, st);
    if (s != DQ_OK) {
        cudaStreamSynchronize(st);          // the copy above may still be reading the caller's buffer
        return s;
    }
    if (cudaMemcpyAsync(out_packed, d_packed, pbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaMemcpyAsync(out_scale, d_scale, sbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

dq_status dqsg_encode_host(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                           const dq_params* p, uint32_t* out_packed, float* out_scale, void* workspace,
                           uint64_t workspace_bytes, void* cuda_stream)
{
    return encode_host(DQ_KIND_DQSG, grad, n, seed, worker, step, p, out_packed, out_scale, workspace,
                       workspace_bytes, cuda_stream);
}

dq_status ndqsg_encode_host(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                            const dq_params* p, uint32_t* out_packed, float* out_scale, void* workspace,
                            uint64_t workspace_bytes, void* cuda_stream)
{
    return encode_host(DQ_KIND_NDQSG, grad, n, seed, worker, step, p, out_packed, out_scale, workspace,
                       workspace_bytes, cuda_stream);
}

static dq_status decode_host(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step, const float* side_info,
                             bool side_first, float* out_avg, void* workspace, uint64_t workspace_bytes,
                             void* cuda_stream)
{
    if (!msgs || W == 0u || W > DQ_MAX_WORKERS) return DQ_ERR_INVALID_ARG;
    if (side_first && msgs[0].kind != DQ_KIND_DQSG) return DQ_ERR_INVALID_ARG;
    for (uint32_t w = 0; w < W; ++w) {
        uint32_t L;
        float alpha;
        dq_status s = check_params(&msgs[w].p, msgs[w].kind, &L, &alpha);
        if (s != DQ_OK) return s;
        if (!msgs[w].packed || !msgs[w].scale) return DQ_ERR_INVALID_ARG;
        // what decode_common would reject, checked here before any copy is queued
        if (msgs[w].p.bucket != msgs[0].p.bucket) return DQ_ERR_UNSUPPORTED;
        if ((msgs[w].p.dither_bits == 16u) != (msgs[0].p.dither_bits == 16u)) return DQ_ERR_UNSUPPORTED;
        if (msgs[w].kind == DQ_KIND_NDQSG && !side_info && !side_first) return DQ_ERR_INVALID_ARG;
    }
    if (n == 0) return DQ_OK;
    if (n >= (1ull << 34)) return DQ_ERR_UNSUPPORTED;
    if (!out_avg || !workspace) return DQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0u) return DQ_ERR_ALIGNMENT;
    if (workspace_bytes < dq_decode_workspace_bytes(msgs, W, n, side_info != nullptr)) return DQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    float* d_out = reinterpret_cast<float*>(ws);
    ws += align_up(n * 4u, 256u);
    float* d_side = nullptr;
    if (side_info) {
        d_side = reinterpret_cast<float*>(ws);
        ws += align_up(n * 4u, 256u);
        if (cudaMemcpyAsync(d_side, side_info, n * 4u, cudaMemcpyHostToDevice, st) != cudaSuccess) return DQ_ERR_CUDA;
    }
    dq_msg dev_msgs[DQ_MAX_WORKERS];
    for (uint32_t w = 0; w < W; ++w) {
        dev_msgs[w] = msgs[w];
        const uint64_t pbytes = dq_packed_words(n, msgs[w].p.bits) * 4u;
        const uint64_t sbytes = dq_num_buckets(n, msgs[w].p.bucket) * 4u;
        uint32_t* d_p = reinterpret_cast<uint32_t*>(ws);
        ws += align_up(pbytes, 256u);
        float* d_s = reinterpret_cast<float*>(ws);
        ws += align_up(sbytes, 256u);
        if (cudaMemcpyAsync(d_p, msgs[w].packed, pbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return DQ_ERR_CUDA;
        if (cudaMemcpyAsync(d_s, msgs[w].scale, sbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return DQ_ERR_CUDA;
        dev_msgs[w].packed = d_p;
        dev_msgs[w].scale = d_s;
    }
    dq_status s = decode_common(dev_msgs, W, n, step, d_side, d_out, nullptr, true, st, false, false, 0u, side_first);
    if (s != DQ_OK) {
        cudaStreamSynchronize(st);          // copies queued above may still be reading the caller's buffers
        return s;
    }
    if (cudaMemcpyAsync(out_avg, d_out, n * 4u, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DQ_ERR_CUDA;
    return DQ_OK;
}

dq_status ndqsg_decode_aggregate_host(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                      const float* side_info, float* out_avg, void* workspace,
                                      uint64_t workspace_bytes, void* cuda_stream)
{
    return decode_host(msgs, W, n, step, side_info, false, out_avg, workspace, workspace_bytes, cuda_stream);
}

dq_status ndqsg_decode_aggregate_side_first_host(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                                 float* out_avg, void* workspace, uint64_t workspace_bytes,
                                                 void* cuda_stream)
{
    return decode_host(msgs, W, n, step, nullptr, true, out_avg, workspace, workspace_bytes, cuda_stream);
}

// ------------------------------------------------------------------------------------------------ no allocation
// Staging area of dqsg_encode_host_static.  In host code this name is only a handle for the runtime, not a
// device address: the address the kernels and copies use is looked up with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[DQ_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_scratch_mutex;
void* g_static_scratch_addr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device; looked up once per device.
dq_status static_scratch_address(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return DQ_ERR_CUDA;
        g_static_scratch_addr[dev] = ptr;
    }
    *out = g_static_scratch_addr[dev];
    return DQ_OK;
}
}  // namespace

dq_status dqsg_encode_host_static(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                                  const dq_params* p, uint32_t* out_packed, float* out_scale, void* cuda_stream)
{
    uint32_t L;
    float alpha;
    dq_status s = check_params(p, DQ_KIND_DQSG, &L, &alpha);
    if (s != DQ_OK) return s;
    if (n == 0) return DQ_OK;
    if (!grad || !out_packed || !out_scale) return DQ_ERR_INVALID_ARG;
    if (n >= (1ull << 34) || dq_encode_workspace_bytes(n, p) > (uint64_t)DQ_STATIC_SCRATCH_BYTES)
        return DQ_ERR_TOO_LARGE;
    void* scratch = nullptr;
    s = static_scratch_address(&scratch);
    if (s != DQ_OK) return s;
    return encode_host(DQ_KIND_DQSG, grad, n, seed, worker, step, p, out_packed, out_scale, scratch,
                       (uint64_t)DQ_STATIC_SCRATCH_BYTES, cuda_stream);
}

dq_status dq_device_error_flags(uint32_t* out_flags)
{
    if (!out_flags) return DQ_ERR_INVALID_ARG;
    unsigned int v = 0u, zero = 0u;
    if (cudaDeviceSynchronize() != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&v, g_dq_error_flags, sizeof(v)) != cudaSuccess) return DQ_ERR_CUDA;
    if (cudaMemcpyToSymbol(g_dq_error_flags, &zero, sizeof(zero)) != cudaSuccess) return DQ_ERR_CUDA;
    *out_flags = v;
    return DQ_OK;
}

uint64_t dq_launch_count(void) { return g_launches.load(); }

}  // extern "C"
