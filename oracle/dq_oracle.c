/*
 * dq_oracle.c  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU implementation of the dithered (DQSG)
 * and nested dithered (NDQSG) gradient quantizers of Abdi & Fekri, "Nested
 * Dithered Quantization for Communication Reduction in Distributed Training",
 * written step by step in the paper's order and notation.  It exists so the
 * CUDA library can be checked against something that shares no code with it.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
 * build, load or call anything in this directory; the library never does.
 *
 * All vector arithmetic is IEEE binary32, round-to-nearest-even, with no
 * contraction except where fmaf() is written (build with -ffp-contract=off).
 * The scalar helpers at the top use double and the paper's symbols directly.
 *
 * Pinned by tests that do not depend on this file's own formulas: the published
 * Philox4x32-10 known-answer vectors, the paper's worked nested example, the
 * uniform-error law of Schuchman's theorem, the selection probabilities of
 * Appendix A, the decoding/MSE statements of the NDQSG theorem, a brute-force
 * nearest-coset search, and a big-integer definition of the bit stream.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define DQO_OK 0
#define DQO_BAD_ARG 1

#define DQO_KIND_DQSG 0u
#define DQO_KIND_NDQSG 1u

/* ------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
 * as 1, 2, 3", SC'11).  The paper only asks for "the same random number
 * generator algorithm and seed number" on both sides (Remark after the
 * dithered-quantization definition; Algorithm 1, worker and server dither
 * steps); a counter-based generator makes "update the seed every iteration"
 * a matter of putting the iteration number in the counter.
 * ---------------------------------------------------------------------- */
void dqo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {            /* Weyl sequence on the key */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32 random bits of element i of worker `worker` at iteration `step`:
 * key = the worker's 64-bit seed, counter = (i/4, worker, step), word i mod 4.
 * i is the index in the whole gradient, so any bucket can be handled alone. */
uint32_t dqo_dither_bits(uint64_t seed, uint32_t worker, uint64_t step, uint64_t i)
{
    uint32_t ctr[4], key[2], out[4];
    ctr[0] = (uint32_t)(i >> 2);
    ctr[1] = worker;
    ctr[2] = (uint32_t)(step & 0xFFFFFFFFu);
    ctr[3] = (uint32_t)(step >> 32);
    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);
    key[1] = (uint32_t)(seed >> 32);
    dqo_philox4x32_10(ctr, key, out);
    return out[i & 3u];
}

/* Dither in units of the fine step: delta = u / Delta, uniform on the grid
 * {(2j+1) 2^-23 - 1/2 : j = 0 .. 2^22-1}, symmetric about 0, never 0 or +-1/2
 * (u ~ U[-Delta/2, Delta/2], Section 3.1).  Every operation here is exact. */
float dqo_dither_from_bits(uint32_t x)
{
    uint32_t odd = ((x >> 10) << 1) | 1u;          /* odd integer below 2^23 */
    return (float)odd * 0x1p-23f - 0.5f;
}

float dqo_dither(uint64_t seed, uint32_t worker, uint64_t step, uint64_t i)
{
    return dqo_dither_from_bits(dqo_dither_bits(seed, worker, step, i));
}

/* Second, cheaper stream ("16-bit dither"): one Philox block serves eight elements.  Element i uses block
 * i/8 (counter = (i/8, worker, step)), word (i mod 8)/2, the low half-word if i is even and the high one if
 * i is odd.  The 16 bits h give delta = (2h+1) 2^-17 - 1/2: a symmetric grid of 65536 points, never 0 or
 * +-1/2.  Any uniform pseudo-random sequence over the step serves Algorithm 1; the coarser grid leaves the
 * error uniform on the step up to 2^-17 of it. */
uint32_t dqo_dither16_half(uint64_t seed, uint32_t worker, uint64_t step, uint64_t i)
{
    uint32_t ctr[4], key[2], out[4];
    ctr[0] = (uint32_t)(i >> 3);
    ctr[1] = worker;
    ctr[2] = (uint32_t)(step & 0xFFFFFFFFu);
    ctr[3] = (uint32_t)(step >> 32);
    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);
    key[1] = (uint32_t)(seed >> 32);
    dqo_philox4x32_10(ctr, key, out);
    uint32_t word = out[(i & 7u) >> 1];
    return (i & 1u) ? (word >> 16) : (word & 0xFFFFu);
}

float dqo_dither16_from_half(uint32_t h)
{
    return (float)(2u * h + 1u) * 0x1p-17f - 0.5f;       /* exact */
}

/* dither of element i in the stream selected by dither_bits (32: one word per element; 16: see above) */
float dqo_dither_stream(uint64_t seed, uint32_t worker, uint64_t step, uint64_t i, uint32_t dither_bits)
{
    /* dither_bits = 0 is the receiver that cannot reproduce the dither ("half-dithered" quantization,
     * Section 2.1: x~_h = Q(x + u), nothing is subtracted); only the decoder accepts it */
    if (dither_bits == 0u) return 0.0f;
    if (dither_bits == 16u)
        return dqo_dither16_from_half(dqo_dither16_half(seed, worker, step, i));
    return dqo_dither(seed, worker, step, i);
}

/* ------------------------------------------------------------------------
 * Scalar definitions in double, the paper's symbols.
 * ---------------------------------------------------------------------- */
/* Q(v) = Delta * round(v / Delta)   (Section 2.1) */
double dqo_Q(double v, double Delta) { return Delta * nearbyint(v / Delta); }

/* x~ = Q(x + u) - u   (definition of dithered quantization) */
double dqo_dithered(double x, double u, double Delta) { return dqo_Q(x + u, Delta) - u; }

/* t = alpha x + u;  s = Q1(t) - Q2(t)   (nested encoder equation) */
double dqo_nested_encode_scalar(double x, double u, double Delta1, double Delta2, double alpha)
{
    double t = alpha * x + u;
    return dqo_Q(t, Delta1) - dqo_Q(t, Delta2);
}

/* r = s - u - alpha y;  x^ = y + alpha (r - Q2(r))   (nested decoder equation) */
double dqo_nested_decode_scalar(double s, double u, double y, double Delta2, double alpha)
{
    double r = s - u - alpha * y;
    return y + alpha * (r - dqo_Q(r, Delta2));
}

/* Raw message size in bits when an index costs log2(levels) bits and every
 * partition sends one 32-bit scale (the accounting behind the raw-bits table). */
double dqo_raw_bits(uint64_t n, uint32_t levels, uint64_t partitions)
{
    return (double)n * log2((double)levels) + 32.0 * (double)partitions;
}

/* ------------------------------------------------------------------------
 * Sizes
 * ---------------------------------------------------------------------- */
uint64_t dqo_packed_words(uint64_t n, uint32_t bits) { return (n * (uint64_t)bits + 31u) / 32u; }
uint64_t dqo_num_buckets(uint64_t n, uint32_t bucket) { return (n + bucket - 1u) / bucket; }
uint32_t dqo_default_levels(uint32_t bits) { return bits == 1u ? 2u : (1u << bits) - 1u; }

/* ------------------------------------------------------------------------
 * Bit stream: element i's b-bit code sits at bit offset i*b of a little-endian
 * stream of 32-bit words (the paper sends "q_p or the corresponding
 * quantization bin", Algorithm 1, and leaves the layout open).
 * ---------------------------------------------------------------------- */
void dqo_pack(const uint32_t *code, uint64_t n, uint32_t bits, uint32_t *words)
{
    uint64_t nw = dqo_packed_words(n, bits);
    memset(words, 0, nw * sizeof(uint32_t));
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t bit = i * bits;
        uint64_t w = bit >> 5;
        uint32_t sh = (uint32_t)(bit & 31u);
        words[w] |= code[i] << sh;
        if (sh + bits > 32u)
            words[w + 1] |= code[i] >> (32u - sh);
    }
}

uint32_t dqo_unpack_one(const uint32_t *words, uint64_t i, uint32_t bits)
{
    uint64_t bit = i * bits;
    uint64_t w = bit >> 5;
    uint32_t sh = (uint32_t)(bit & 31u);
    uint32_t v = words[w] >> sh;
    if (sh + bits > 32u)
        v |= words[w + 1] << (32u - sh);
    return v & ((bits == 32u) ? 0xFFFFFFFFu : ((1u << bits) - 1u));
}

void dqo_unpack(const uint32_t *words, uint64_t n, uint32_t bits, uint32_t *code)
{
    for (uint64_t i = 0; i < n; ++i)
        code[i] = dqo_unpack_one(words, i, bits);
}

/* ------------------------------------------------------------------------
 * Radix-3 container for three-level messages (the paper's raw-bit count for
 * DQSGD with M = 1 is log2(3) = 1.585 bits per element, Section 4, raw-bits
 * table): byte k carries the five ternary codes 5k .. 5k+4 as the number
 *     t_{5k} + 3 t_{5k+1} + 9 t_{5k+2} + 27 t_{5k+3} + 81 t_{5k+4}   (< 243),
 * codes past the end of the vector counting as 0; 8/5 = 1.6 bits per element.
 * A three-level message only holds the codes 0, 1, 2; a code above 2 is
 * stored as 2.
 * ---------------------------------------------------------------------- */
uint64_t dqo_ternary_bytes(uint64_t n) { return (n + 4u) / 5u; }

void dqo_ternary_pack(const uint32_t *code, uint64_t n, uint8_t *bytes)
{
    uint64_t nb = dqo_ternary_bytes(n);
    for (uint64_t k = 0; k < nb; ++k) {
        uint32_t v = 0, weight = 1;
        for (uint32_t q = 0; q < 5u; ++q) {
            uint64_t i = 5u * k + q;
            uint32_t t = (i < n) ? code[i] : 0u;
            if (t > 2u)
                t = 2u;
            v += t * weight;
            weight *= 3u;
        }
        bytes[k] = (uint8_t)v;
    }
}

void dqo_ternary_unpack(const uint8_t *bytes, uint64_t n, uint32_t *code)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t v = bytes[i / 5u];
        for (uint32_t q = 0; q < (uint32_t)(i % 5u); ++q)
            v /= 3u;
        code[i] = v % 3u;
    }
}

/* ------------------------------------------------------------------------
 * Per-bucket scale: kappa_j = max |g_i| over the bucket (kappa = ||g||_inf of
 * Eq. (DQSG), one per partition as in the partitioning paragraph of 3.1).
 * ---------------------------------------------------------------------- */
static float bucket_kappa(const float *g, uint64_t len)
{
    float kappa = 0.0f;
    for (uint64_t i = 0; i < len; ++i) {
        float a = fabsf(g[i]);
        if (a > kappa) kappa = a;
    }
    return kappa;
}

/* gain a_j = num / kappa_j, or 0 for an all-zero (or vanishing) bucket */
static float bucket_gain(float num, float kappa)
{
    return (kappa >= 0x1p-100f) ? num / kappa : 0.0f;
}

static int check_common(uint32_t bucket, uint32_t bits, uint64_t i0)
{
    if (bucket < 32u || bucket > 65536u || (bucket % 32u) != 0u) return DQO_BAD_ARG;
    if (bits < 1u || bits > 8u) return DQO_BAD_ARG;
    if (i0 % bucket != 0u) return DQO_BAD_ARG;
    return DQO_OK;
}

/* ------------------------------------------------------------------------
 * DQSG encoder (Eq. (DQSG); Algorithm 1, worker steps).
 * In index units (dither delta = u/Delta, Delta = 1/s, s = (L-1)/2):
 *     q = round((g/kappa + u)/Delta) = round(g s/kappa + delta),
 * and the transmitted code is k = q + s in {0..L-1}.
 * g points at element i0 of the gradient; n elements are encoded.
 * code_out (optional) receives k per element.
 * ---------------------------------------------------------------------- */
int dqo_dqsg_encode(const float *g, uint64_t n, uint64_t i0,
                    uint64_t seed, uint32_t worker, uint64_t step,
                    uint32_t bucket, uint32_t bits, uint32_t levels, uint32_t dither_bits,
                    uint32_t *packed, float *scale, int32_t *code_out, int threads)
{
    int rc = check_common(bucket, bits, i0);
    if (rc) return rc;
    if (dither_bits != 32u && dither_bits != 16u) return DQO_BAD_ARG;
    if (levels == 0u) levels = dqo_default_levels(bits);
    if (levels < 2u || levels > (1u << bits)) return DQO_BAD_ARG;
    uint64_t nb = dqo_num_buckets(n, bucket);
    uint32_t *code = (uint32_t *)malloc((n ? n : 1) * sizeof(uint32_t));
    if (!code) return DQO_BAD_ARG;
    const float s = (float)(levels - 1u) / 2.0f;
    (void)threads;
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
    for (int64_t j = 0; j < (int64_t)nb; ++j) {
        uint64_t lo = (uint64_t)j * bucket;
        uint64_t len = (n - lo < bucket) ? (n - lo) : bucket;
        float kappa = bucket_kappa(g + lo, len);
        scale[j] = kappa;
        float a = bucket_gain(s, kappa);
        for (uint64_t i = lo; i < lo + len; ++i) {
            float delta = dqo_dither_stream(seed, worker, step, i0 + i, dither_bits);
            float v = fmaf(g[i], a, delta);
            float w = v + s;
            int32_t k = (int32_t)rintf(w);
            if (k < 0) k = 0;
            if (k > (int32_t)levels - 1) k = (int32_t)levels - 1;
            code[i] = (uint32_t)k;
            if (code_out) code_out[i] = k;
        }
    }
    dqo_pack(code, n, bits, packed);
    free(code);
    return DQO_OK;
}

/* ------------------------------------------------------------------------
 * NDQSG encoder (nested encoder equation; Algorithm 2, workers in P2), with
 * the per-bucket normalisation of Algorithm 1.  In units of the fine step
 * Delta_1 = 1/M1:   t/Delta_1 = alpha M1 g/kappa + delta,  q1 = round(.),
 * and the message is the coset m = q1 mod K (K = Delta_2/Delta_1), which
 * carries the same information as s = Q1(t) - Q2(t).
 * q1_out (optional) receives the fine index before the modulo.
 * ---------------------------------------------------------------------- */
int dqo_ndqsg_encode(const float *g, uint64_t n, uint64_t i0,
                     uint64_t seed, uint32_t worker, uint64_t step,
                     uint32_t bucket, uint32_t bits, uint32_t coarse_K, float fine_M, float alpha,
                     uint32_t dither_bits, uint32_t *packed, float *scale, int32_t *q1_out, int threads)
{
    int rc = check_common(bucket, bits, i0);
    if (rc) return rc;
    if (dither_bits != 32u && dither_bits != 16u) return DQO_BAD_ARG;
    if (coarse_K < 2u || coarse_K > (1u << bits)) return DQO_BAD_ARG;
    if (!(fine_M > 0.0f) || !(alpha > 0.0f) || alpha > 1.0f) return DQO_BAD_ARG;
    uint64_t nb = dqo_num_buckets(n, bucket);
    uint32_t *code = (uint32_t *)malloc((n ? n : 1) * sizeof(uint32_t));
    if (!code) return DQO_BAD_ARG;
    const float A = alpha * fine_M;
    const int32_t K = (int32_t)coarse_K;
    (void)threads;
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
    for (int64_t j = 0; j < (int64_t)nb; ++j) {
        uint64_t lo = (uint64_t)j * bucket;
        uint64_t len = (n - lo < bucket) ? (n - lo) : bucket;
        float kappa = bucket_kappa(g + lo, len);
        scale[j] = kappa;
        float a = bucket_gain(A, kappa);
        for (uint64_t i = lo; i < lo + len; ++i) {
            float delta = dqo_dither_stream(seed, worker, step, i0 + i, dither_bits);
            int32_t q1 = (int32_t)rintf(fmaf(g[i], a, delta));
            int32_t m = ((q1 % K) + K) % K;
            code[i] = (uint32_t)m;
            if (q1_out) q1_out[i] = q1;
        }
    }
    dqo_pack(code, n, bits, packed);
    free(code);
    return DQO_OK;
}

/* ------------------------------------------------------------------------
 * One worker's message as the decoder sees it.
 * ---------------------------------------------------------------------- */
typedef struct {
    uint32_t kind;          /* DQO_KIND_DQSG / DQO_KIND_NDQSG */
    uint32_t bucket;
    uint32_t bits;
    uint32_t levels;        /* DQSG */
    uint32_t coarse_K;      /* NDQSG */
    float fine_M;           /* NDQSG */
    float alpha;            /* NDQSG */
    uint32_t worker;
    uint32_t dither_bits;   /* 32 or 16 */
    uint32_t reserved;
    uint64_t seed;
    const uint32_t *packed; /* words for elements [i0, i0+n) */
    const float *scale;     /* scales for the same range */
} dqo_msg;

/* DQSG reconstruction (Algorithm 1, server): g~ = kappa (Delta q - u)
 *   = (kappa/s) ((k - s) - delta). */
static float dqsg_reconstruct(uint32_t k, float s, float c, float delta)
{
    float d = ((float)k - s) - delta;
    return c * d;
}

/* NDQSG reconstruction (nested decoder equation; Algorithm 2, server loop) in
 * fine-step units, y = side information:
 *   r  = m - delta - alpha M1 y / kappa            (r / Delta_1)
 *   Q2(r)/Delta_1 = K round(r / K),  q^1 = m - K round(r/K)
 *   g~ = y + alpha (r - Q2(r)) = (1 - alpha^2) y + (alpha kappa / M1)(q^1 - delta). */
static float ndqsg_reconstruct(uint32_t m, int32_t K, float a, float beta, float alpha,
                               float delta, float y, int32_t *qhat_out)
{
    float r1 = (float)m - delta;
    float r = fmaf(-y, a, r1);
    int32_t jj = (int32_t)rintf(r / (float)K);
    int32_t qhat = (int32_t)m - K * jj;
    float d = (float)qhat - delta;
    if (qhat_out) *qhat_out = qhat;
    if (alpha == 1.0f)
        return beta * d;
    return fmaf(beta, d, (1.0f - alpha * alpha) * y);
}

/* ------------------------------------------------------------------------
 * Decode W messages and average them (Algorithm 1, server: g_bar = 1/P sum g~_p;
 * Algorithm 2 with the side information given as a vector).  Workers are summed
 * in index order.  recon (optional, [W][n]) receives each g~_w, qhat (optional,
 * [W][n]) the resolved fine index of NDQSG workers (k - s is not stored for DQSG;
 * those rows get the code k).
 * ---------------------------------------------------------------------- */
static int decode_aggregate_impl(const dqo_msg *msgs, uint32_t W, uint64_t n, uint64_t i0, uint64_t step,
                                 const float *side_info, int running, float *out_avg,
                                 float *recon, int32_t *qhat, int threads)
{
    if (W == 0u) return DQO_BAD_ARG;
    for (uint32_t w = 0; w < W; ++w) {
        const dqo_msg *m = &msgs[w];
        int rc = check_common(m->bucket, m->bits, i0);
        if (rc) return rc;
        if (m->bucket != msgs[0].bucket) return DQO_BAD_ARG;
        if (m->dither_bits != 32u && m->dither_bits != 16u &&
            !(m->dither_bits == 0u && m->kind == DQO_KIND_DQSG)) return DQO_BAD_ARG;
        if (m->kind == DQO_KIND_DQSG) {
            uint32_t L = m->levels ? m->levels : dqo_default_levels(m->bits);
            if (L < 2u || L > (1u << m->bits)) return DQO_BAD_ARG;
        } else if (m->kind == DQO_KIND_NDQSG) {
            if (m->coarse_K < 2u || m->coarse_K > (1u << m->bits)) return DQO_BAD_ARG;
            if (!(m->fine_M > 0.0f) || !(m->alpha > 0.0f) || m->alpha > 1.0f) return DQO_BAD_ARG;
            if (running ? (w == 0u) : (side_info == NULL)) return DQO_BAD_ARG;
        } else {
            return DQO_BAD_ARG;
        }
    }
    const uint32_t bucket = msgs[0].bucket;
    (void)threads;
#pragma omp parallel for schedule(static) num_threads(threads > 0 ? threads : 1)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        uint64_t j = (uint64_t)i / bucket;
        float acc = 0.0f;
        for (uint32_t w = 0; w < W; ++w) {
            const dqo_msg *m = &msgs[w];
            float kappa = m->scale[j];
            float delta = dqo_dither_stream(m->seed, m->worker, step, i0 + (uint64_t)i, m->dither_bits);
            uint32_t code = dqo_unpack_one(m->packed, (uint64_t)i, m->bits);
            float gt;
            if (m->kind == DQO_KIND_DQSG) {
                uint32_t L = m->levels ? m->levels : dqo_default_levels(m->bits);
                float s = (float)(L - 1u) / 2.0f;
                float c = kappa / s;
                gt = dqsg_reconstruct(code, s, c, delta);
                if (qhat) qhat[(uint64_t)w * n + (uint64_t)i] = (int32_t)code;
            } else {
                float A = m->alpha * m->fine_M;
                float a = bucket_gain(A, kappa);
                float beta = (m->alpha * kappa) / m->fine_M;
                int32_t qh;
                /* Algorithm 2 as written: the side information is the mean of everything decoded so far */
                float y = running ? acc * (1.0f / (float)w) : side_info[i];
                gt = ndqsg_reconstruct(code, (int32_t)m->coarse_K, a, beta, m->alpha, delta, y, &qh);
                if (qhat) qhat[(uint64_t)w * n + (uint64_t)i] = qh;
            }
            if (recon) recon[(uint64_t)w * n + (uint64_t)i] = gt;
            acc = acc + gt;
        }
        out_avg[i] = acc / (float)W;
    }
    return DQO_OK;
}

int dqo_decode_aggregate(const dqo_msg *msgs, uint32_t W, uint64_t n, uint64_t i0, uint64_t step,
                         const float *side_info, float *out_avg,
                         float *recon, int32_t *qhat, int threads)
{
    return decode_aggregate_impl(msgs, W, n, i0, step, side_info, 0, out_avg, recon, qhat, threads);
}

/* Algorithm 2, server loop, as written: the workers are visited in array order; a DQSG message (group P1) is
 * reconstructed directly; an NDQSG message (group P2) is decoded against g_bar = the mean of all reconstructions
 * before it, and g_bar is then updated with the new reconstruction.  With S the running fp32 sum and w the number
 * of workers already decoded, g_bar = S * (1/w) (reciprocal rounded once).  The first message must be DQSG.
 * The result is the mean over all W. */
int dqo_decode_aggregate_running(const dqo_msg *msgs, uint32_t W, uint64_t n, uint64_t i0, uint64_t step,
                                 float *out_avg, float *recon, int32_t *qhat, int threads)
{
    return decode_aggregate_impl(msgs, W, n, i0, step, NULL, 1, out_avg, recon, qhat, threads);
}

/* ------------------------------------------------------------------------
 * Brute-force coset decoder (tests only): among the fine indices congruent to
 * m modulo K, pick the one whose dither-subtracted value lies nearest to the
 * normalised side information, i.e. the point "in the same coarse bin as y".
 * Returns the winning index; *margin receives (second best - best) distance.
 * ---------------------------------------------------------------------- */
int32_t dqo_nearest_coset_bruteforce(uint32_t m, int32_t K, double a, double delta, double y,
                                     int32_t T, double *margin)
{
    double best = INFINITY, second = INFINITY;
    int32_t arg = 0;
    for (int32_t t = -T; t <= T; ++t) {
        int32_t q = (int32_t)m + K * t;
        double dist = fabs(((double)q - delta) - y * a);
        if (dist < best) { second = best; best = dist; arg = q; }
        else if (dist < second) { second = dist; }
    }
    if (margin) *margin = second - best;
    return arg;
}
