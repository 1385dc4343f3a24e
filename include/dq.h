/*
 * dq.h -- C ABI of the dithered / nested dithered gradient quantizer for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-worker encoder and the server-side decode-and-average step of
 * Abdi & Fekri, "Nested Dithered Quantization for Communication Reduction in Distributed Training":
 *
 *   DQSG   (Section 3.1, Eq. (DQSG), Algorithm 1):  g~ = kappa (Q(g/kappa + u) - u),  kappa = ||g||_inf,
 *          u ~ U[-Delta/2, Delta/2] regenerated at the receiver from a shared seed; the worker sends
 *          kappa and the bin index.
 *   NDQSG  (Section 3.2, nested encoder / decoder equations, Algorithm 2):  t = alpha g + u,
 *          s = Q1(t) - Q2(t);  r = s - u - alpha y,  g^ = y + alpha (r - Q2(r))  with side information y.
 *
 * Conventions shared by every entry point
 *   - A gradient is a flat fp32 vector of n elements, cut into buckets of `bucket` elements (the paper's
 *     equal partitions, one scale kappa each; the last bucket may be short).
 *   - The dither of element i of worker `worker` at iteration `step` is word (i mod 4) of
 *     Philox4x32-10(key = seed, counter = (i / 4, worker, lo32(step), hi32(step))), mapped to the open
 *     grid {(2j+1) 2^-23 - 1/2} in units of the fine quantization step.  With dq_params.dither_bits = 16
 *     one block serves eight elements instead: block i / 8, word (i mod 8) / 2, low half-word for even i
 *     and high half-word for odd i, mapped to {(2h+1) 2^-17 - 1/2}; this halves the generator's cost,
 *     which dominates both kernels.  Encoder and decoder must be given the same (seed, worker, step) and
 *     the same dither_bits.
 *   - A message is `scale` (one fp32 per bucket) plus `packed`: element i's b-bit code at bit offset
 *     i*b of a little-endian stream of 32-bit words; pad bits of the last word are written as 0.
 *   - "device" pointers are CUDA device memory on the current device, 16-byte aligned, owned by the
 *     caller.  The library allocates nothing at run time and keeps no state between calls, with two
 *     exceptions that live in its device image: one error word per GPU (dq_device_error_flags) and the
 *     fixed staging array of dqsg_encode_host_static.  It is asynchronous on the given stream (it never
 *     synchronises), except for the *_host entry points, which return after the results are in the
 *     caller's host buffers.
 *   - Outputs must not alias inputs.  Inputs are assumed finite.
 *   - The integer decisions are taken in fp32 with the rounding constant 1.5 * 2^23, which is exact for
 *     magnitudes below 2^22: DQSG needs (L-1)/2 + 1 < 2^22 (always true for b <= 8); NDQSG needs
 *     alpha*M1 <= 2^20 (checked) and, at the decoder, |alpha*M1*y/kappa| < 2^21 for every element, i.e. side
 *     information that is not millions of coarse cells away from the gradient -- in particular a message
 *     whose bucket scale kappa is almost zero (below about 1e-6 of |y|) must not be paired with ordinary
 *     side information.  Beyond that bound the resolved coset is undefined (no fault, no diagnostic).
 *   - Errors are return codes only.  Invalid arguments are rejected before anything is launched.
 *   - n must be below 2^34.
 */
#ifndef DQ_H_
#define DQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DQ_OK = 0,
    DQ_ERR_INVALID_ARG = 1,   /* NULL pointer, n or W out of range, bits/levels/K/alpha out of range      */
    DQ_ERR_UNSUPPORTED = 2,   /* valid in the paper's terms but not handled (e.g. mixed bucket sizes)     */
    DQ_ERR_ALIGNMENT = 3,     /* a device pointer is not 16-byte aligned                                  */
    DQ_ERR_CUDA = 4,          /* a CUDA call or launch failed; see cudaGetLastError of the calling thread */
    DQ_ERR_TOO_LARGE = 5      /* the input does not fit the library's built-in scratch buffer              */
} dq_status;

typedef enum { DQ_KIND_DQSG = 0, DQ_KIND_NDQSG = 1 } dq_kind;

/* Bits of the optional decode status word and of dq_device_error_flags(). */
#define DQ_WARN_NONFINITE_SCALE 0x1u   /* a received scale was NaN or Inf                                   */
#define DQ_ERR_COPY_TIMEOUT     0x2u   /* a bounded wait for an asynchronous tile copy ran out; the tile
                                          was skipped and its outputs are undefined                        */
#define DQ_WARN_CODE_RANGE      0x4u   /* dq_ternary_pack met a code 3 (not a three-level message); it was
                                          stored as 2                                                      */

/* One quantizer description.  Plain data, read during the call. */
typedef struct {
    uint32_t bucket;    /* B: multiple of 32 in [32, 65536]                                               */
    uint32_t bits;      /* b: 1..8 bits per element on the wire                                           */
    uint32_t levels;    /* DQSG: number of levels L, 2..2^b (odd L = the paper's 2M+1, Delta = 2/(L-1));
                           0 selects L = 2 for b = 1 and 2^b - 1 otherwise.  Ignored for NDQSG.           */
    uint32_t coarse_K;  /* NDQSG: K = Delta_2 / Delta_1, 2..2^b.  Ignored for DQSG.                       */
    float    fine_M;    /* NDQSG: M1 = 1/Delta_1 in units of kappa, 0 < alpha*M1 <= 2^20.                 */
    float    alpha;     /* NDQSG: shrinkage, 0 < alpha <= 1; 0 selects 1.                                 */
    uint32_t dither_bits; /* random bits per dither value: 32 (0 selects it) or 16, see above              */
    uint32_t flags;     /* DQ_FLAG_* bits, 0 for none                                                     */
} dq_params;

/*
 * DQ_FLAG_INPUT_READY (encoders only; ignored elsewhere).  By default an encode kernel touches no memory
 * before the previous kernel of its stream has completed.  With this flag the caller declares that `grad`
 * was completely written before that previous kernel was launched and is not written by it -- the usual case
 * when a gradient produced by the backward pass is encoded after some unrelated kernel, or when several
 * gradients are encoded back to back.  The encoder then requests and quantizes its first tiles while the
 * previous kernel is still draining; its stores to out_packed and out_scale still wait for that kernel to
 * complete, so outputs may be shared with it.  Results are identical with and without the flag.
 */
#define DQ_FLAG_INPUT_READY 0x1u
/*
 * DQ_FLAG_OUTPUT_FREE (encoders only; has an effect only together with DQ_FLAG_INPUT_READY).  The caller
 * additionally declares that the previous kernel of the stream neither reads nor writes out_packed and
 * out_scale -- e.g. the encodes of different workers' gradients into different message buffers, back to back.
 * Then nothing in the encoder waits for that kernel except its own end: the two kernels overlap wherever the
 * GPU has room (the tail of one runs beside the head of the next), while a later kernel that waits for this
 * one still sees both complete.  Results are identical with and without the flag.
 * "Neither reads nor writes" is about the memory, not the pointer: a buffer that a stream-ordered allocator
 * hands out may be memory that the previous kernel still reads (its input, freed by the host a moment ago);
 * such a buffer is not free in this sense.
 */
#define DQ_FLAG_OUTPUT_FREE 0x2u
/*
 * DQ_FLAG_TEST_DROP_COPY (encoders only; for tests of the error path, never for production calls).  One warp
 * of the encoder announces the tile copy of its last work unit but does not issue it.  Its bounded wait for
 * that copy runs out after about 20 ms; the kernel then finishes normally, DQ_ERR_COPY_TIMEOUT is set in the
 * device's error word (dq_device_error_flags) and the codes of that one unit are undefined.  Nothing faults
 * and nothing waits longer than the bound.  Without effect for gradients so short that the warp has one unit.
 */
#define DQ_FLAG_TEST_DROP_COPY 0x80000000u

/* One worker's message as the decoder sees it. */
typedef struct {
    const uint32_t* packed;  /* dq_packed_words(n, p.bits) words                                          */
    const float*    scale;   /* dq_num_buckets(n, p.bucket) scales                                        */
    uint64_t        seed;    /* the worker's dither seed                                                  */
    uint32_t        worker;  /* the worker's index as used by its encoder                                 */
    dq_kind         kind;
    dq_params       p;
} dq_msg;

#define DQ_MAX_WORKERS 64u

/* Message sizes: ceil(n*bits/32) words and ceil(n/bucket) scales. */
uint64_t dq_packed_words(uint64_t n, uint32_t bits);
uint64_t dq_num_buckets(uint64_t n, uint32_t bucket);
/* The level count used when dq_params.levels is 0. */
uint32_t dq_default_levels(uint32_t bits);
const char* dq_status_string(dq_status s);

/*
 * dqsg_encode -- worker side of Algorithm 1 (Eq. (DQSG)): per bucket kappa = max|g|, dither from
 * (seed, worker, step), index q = round((g/kappa + u)/Delta) stored as k = q + (L-1)/2 in b bits.
 *   grad        device, fp32[n], read once
 *   out_packed  device, uint32[dq_packed_words(n, p->bits)], fully overwritten
 *   out_scale   device, fp32[dq_num_buckets(n, p->bucket)], fully overwritten
 *   cuda_stream a cudaStream_t (NULL = default stream)
 * n = 0 is a no-op returning DQ_OK.
 */
dq_status dqsg_encode(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                      const dq_params* p, uint32_t* out_packed, float* out_scale, void* cuda_stream);

/*
 * ndqsg_encode -- worker side of Algorithm 2 for a worker in P2 (nested encoder equation), with the
 * per-bucket normalisation of Algorithm 1: q1 = round(alpha*M1*g/kappa + u/Delta_1), and the message is
 * the coset q1 mod K in [0, K), which determines s = Q1(t) - Q2(t).  Same buffers as dqsg_encode.
 */
dq_status ndqsg_encode(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                       const dq_params* p, uint32_t* out_packed, float* out_scale, void* cuda_stream);

/*
 * dqsg_decode_aggregate -- server side of Algorithm 1: regenerate every worker's dither, reconstruct
 * g~_w = kappa_w (Delta q_w - u_w) and write the mean over the W workers, summed in array order.
 *   msgs     host array of W messages (1 <= W <= DQ_MAX_WORKERS), all of kind DQSG, of one bucket size
 *            and one dither_bits; read during the call, the device buffers they point to are read by
 *            the kernel
 *   out_avg  device, fp32[n], fully overwritten
 */
dq_status dqsg_decode_aggregate(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                float* out_avg, void* cuda_stream);

/*
 * ndqsg_decode_aggregate -- server side of Algorithm 2 with the side information given as a vector
 * (nested decoder equation): DQSG messages are reconstructed as above; an NDQSG message is resolved to
 * the fine index congruent to its code that lies in the coarse cell around alpha*M1*y/kappa, and
 * reconstructed as g^ = (1 - alpha^2) y + (alpha kappa / M1)(q1^ - u/Delta_1); the mean of all W
 * reconstructions is written.  Kinds, bits, levels, K, M1 and alpha may differ per worker.
 *   side_info    device, fp32[n]; required when any message is NDQSG, may be NULL otherwise
 *   status_word  device uint32, optional (NULL to skip): DQ_WARN_* bits are OR-ed into it
 */
dq_status ndqsg_decode_aggregate(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                 const float* side_info, float* out_avg, uint32_t* status_word,
                                 void* cuda_stream);

/*
 * ndqsg_decode_aggregate_side_first -- the server of Algorithm 2 with one worker in P1: message 0 (which must be
 * a DQSG message) is decoded first and its reconstruction g~_0 is the side information y of every NDQSG message
 * that follows; the mean of all W reconstructions is written.  The result is bit-identical to
 *     dqsg_decode_aggregate(msgs, 1, ..., y);  ndqsg_decode_aggregate(msgs, W, ..., y, out_avg, ...)
 * but y never exists in global memory: no side-information vector is read and the first pass is not launched.
 * Other arguments as for ndqsg_decode_aggregate.
 */
dq_status ndqsg_decode_aggregate_side_first(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                            float* out_avg, uint32_t* status_word, void* cuda_stream);

/*
 * dqsg_decode_aggregate_half_dithered -- the receiver that cannot reproduce the dither (Section 2.1,
 * "half-dithered quantization" x~_h = Q(x + u); by Lemma 1 this is M-level stochastic quantization): every
 * DQSG message is reconstructed as kappa * Delta * q with nothing subtracted, and the mean is written.  No
 * random numbers are generated, so this kernel shows the memory-bound limit of the decoder.  Seeds, worker
 * indices and dither_bits of the messages are ignored.  Arguments as for dqsg_decode_aggregate.
 */
dq_status dqsg_decode_aggregate_half_dithered(const dq_msg* msgs, uint32_t W, uint64_t n, float* out_avg,
                                              void* cuda_stream);

/*
 * ndqsg_decode_aggregate_running -- the server loop of Algorithm 2 as written: the messages are visited in
 * array order; a DQSG message (group P1) is reconstructed directly; an NDQSG message (group P2) is resolved
 * against g_bar = the mean of all reconstructions before it, which is then updated with the new one ("update
 * g_bar using g_p").  g_bar is S * (1/w) with S the running fp32 sum and w the number of messages already
 * decoded, so no side-information vector is read.  msgs[0] must be a DQSG message.  The mean of all W
 * reconstructions is written.  Other arguments as for ndqsg_decode_aggregate.
 */
dq_status ndqsg_decode_aggregate_running(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                         float* out_avg, uint32_t* status_word, void* cuda_stream);

/*
 * Bucket ranges.  Buckets are independent and the dither of an element depends on its index in the whole
 * gradient only (Algorithm 1: every worker quantizes its own coordinates with its own seed; partitioning
 * paragraph of Section 3.1: one scale per partition), so a gradient can be encoded and decoded in pieces: by
 * layer as the backward pass produces them, in chunks that overlap with a transfer, or one bucket range per GPU.
 * The *_range calls work on the elements [first_element, first_element + n) of a longer vector:
 *   first_element   index of the first element in the whole gradient; a multiple of p->bucket (of the messages'
 *                   bucket size for the decoder), else DQ_ERR_INVALID_ARG; first_element + n < 2^34
 *   grad, side_info, out_avg, out_packed, out_scale and the packed / scale pointers inside msgs
 *                   point at the RANGE's data (element first_element is at index 0), sized for n elements
 * Because a range starts at a bucket boundary it starts at a word boundary of the bit stream: the messages of
 * consecutive ranges, concatenated, are bit-identical to the message of one call over the whole vector, and the
 * decoded ranges are the corresponding slices of the whole result.  first_element = 0 is the plain call.
 * Every pointer must still be 16-byte aligned: a range may write straight into its slice of whole-gradient
 * buffers only where that slice is so aligned (first_element * bits a multiple of 128 for the bit stream,
 * first_element / bucket a multiple of 4 for the scales); otherwise give it buffers of its own.
 */
dq_status dqsg_encode_range(const float* grad, uint64_t n, uint64_t first_element, uint64_t seed, uint32_t worker,
                            uint64_t step, const dq_params* p, uint32_t* out_packed, float* out_scale,
                            void* cuda_stream);
dq_status ndqsg_encode_range(const float* grad, uint64_t n, uint64_t first_element, uint64_t seed, uint32_t worker,
                             uint64_t step, const dq_params* p, uint32_t* out_packed, float* out_scale,
                             void* cuda_stream);
dq_status ndqsg_decode_aggregate_range(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t first_element,
                                       uint64_t step, const float* side_info, float* out_avg,
                                       uint32_t* status_word, void* cuda_stream);

/*
 * dq_code_histogram -- counts how often each code occurs in a packed message: hist[c] = number of elements
 * whose b-bit code is c.  This is the input of the paper's rate accounting (Section 4: raw bits are
 * log2(levels) per element, the entropy of the index stream is what an entropy coder approaches).
 *   packed  device, dq_packed_words(n, bits) words
 *   hist    device, uint64[2^bits], 8-byte aligned; zeroed and filled by the call
 */
dq_status dq_code_histogram(const uint32_t* packed, uint64_t n, uint32_t bits, uint64_t* hist, void* cuda_stream);

/*
 * dq_code_entropy -- the empirical entropy H = -sum_c p_c log2 p_c, p_c = hist[c] / sum(hist), of a code
 * histogram, in bits per element: the rate that the entropy coding of the index stream approaches (Section 4,
 * the paragraph on entropy coding and the entropy-coded columns of the tables).  Host arithmetic on at most 256
 * counters.
 *   hist_host             HOST memory, uint64[2^bits] (a copy of dq_code_histogram's result)
 *   out_bits_per_element  HOST, receives H; 0 for an empty histogram
 */
dq_status dq_code_entropy(const uint64_t* hist_host, uint32_t bits, double* out_bits_per_element);

/*
 * Radix-3 container for three-level DQSG messages (levels = 3, bits = 2).  Section 4 counts log2(3) = 1.585
 * bits per element for the three-level quantizer (raw-bits table, DQSGD row); the 2-bit stream spends 2.  The
 * container stores five codes per byte,
 *     byte k = t_{5k} + 3 t_{5k+1} + 9 t_{5k+2} + 27 t_{5k+3} + 81 t_{5k+4}   (codes past n count as 0),
 * i.e. 1.6 bits per element: 20 % fewer bytes on the wire, within 1 % of the paper's count.  The scales are
 * sent unchanged.  The encode and decode-aggregate kernels keep working on the 2-bit stream; these two calls
 * convert a message between the two forms on the device and touch only the packed data.
 *   dq_ternary_bytes   ceil(n / 5), the size of the container
 *   dq_ternary_pack    packed: device, dq_packed_words(n, 2) words whose codes are 0, 1 or 2 (a code 3 is
 *                      stored as 2 and DQ_WARN_CODE_RANGE is OR-ed into *status_word when that is not NULL);
 *                      out_radix: device, dq_ternary_bytes(n) bytes, 16-byte aligned, fully overwritten
 *   dq_ternary_unpack  radix: device, dq_ternary_bytes(n) bytes (a byte above 242 is read as its five
 *                      low base-3 digits); out_packed: device, dq_packed_words(n, 2) words, fully
 *                      overwritten, pad bits 0 -- bit-identical to the stream that was packed
 */
uint64_t dq_ternary_bytes(uint64_t n);
dq_status dq_ternary_pack(const uint32_t* packed, uint64_t n, uint8_t* out_radix, uint32_t* status_word,
                          void* cuda_stream);
dq_status dq_ternary_unpack(const uint8_t* radix, uint64_t n, uint32_t* out_packed, void* cuda_stream);

/*
 * Host-buffer variants.  Every data pointer (grad, out_packed, out_scale, the packed/scale pointers
 * inside msgs, side_info, out_avg) is HOST memory (pinned memory makes the copies asynchronous);
 * `workspace` is device memory of at least the stated size, 256-byte aligned, provided by the caller.
 * Each call copies its inputs to the workspace, runs the same kernels as the device entry points,
 * copies the results back and synchronises the stream before returning.
 */
uint64_t dq_encode_workspace_bytes(uint64_t n, const dq_params* p);
uint64_t dq_decode_workspace_bytes(const dq_msg* msgs, uint32_t W, uint64_t n, int has_side_info);
dq_status dqsg_encode_host(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                           const dq_params* p, uint32_t* out_packed, float* out_scale,
                           void* workspace, uint64_t workspace_bytes, void* cuda_stream);
dq_status ndqsg_encode_host(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                            const dq_params* p, uint32_t* out_packed, float* out_scale,
                            void* workspace, uint64_t workspace_bytes, void* cuda_stream);
dq_status ndqsg_decode_aggregate_host(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                      const float* side_info, float* out_avg,
                                      void* workspace, uint64_t workspace_bytes, void* cuda_stream);
/* ndqsg_decode_aggregate_side_first from host buffers; workspace of dq_decode_workspace_bytes(msgs, W, n, 0). */
dq_status ndqsg_decode_aggregate_side_first_host(const dq_msg* msgs, uint32_t W, uint64_t n, uint64_t step,
                                                 float* out_avg, void* workspace, uint64_t workspace_bytes,
                                                 void* cuda_stream);

/*
 * dqsg_encode_host_static -- dqsg_encode_host for callers that cannot provide device memory.
 * (The paper has no counterpart: this is a packaging variant of the DQSG encoder above.)
 *
 * Some users of this library cannot allocate on the GPU at the point where they need to encode: a
 * training process whose framework has already claimed the device's memory for its own pool, a plug-in
 * that is only handed host buffers, or a latency-critical loop in which cudaMalloc (which can block and
 * synchronise the device) is not acceptable.  For them the device-side staging area that dqsg_encode_host
 * takes as `workspace` lives inside the library instead: a fixed array of DQ_STATIC_SCRATCH_BYTES bytes
 * in device global memory.  Every GPU on which the library is loaded holds that array until the process
 * exits, whether or not this function is ever called.
 *
 *   grad, out_packed, out_scale   HOST memory, as for dqsg_encode_host (pinned memory keeps the copies
 *                                 asynchronous); results are complete when the call returns
 *   returns DQ_ERR_TOO_LARGE      when dq_encode_workspace_bytes(n, p) > DQ_STATIC_SCRATCH_BYTES
 *                                 (about 7.8 million elements at 2 bits); nothing is copied or launched
 *
 * The call performs no cudaMalloc / cudaFree and calls no allocating library routine.  The array is part of
 * the library's device image: the driver reserves it when that image is loaded on a device, which with lazy
 * loading is the first use of ANY entry point there; if the memory cannot be reserved, every entry point fails
 * with DQ_ERR_CUDA.  The first call of this function on each device additionally looks up the array's device
 * address (once per device, with that device current); make one warm-up call per device at start-up, outside
 * any stream capture and outside the latency-critical loop.  The address is cached for the life of the
 * process: cudaDeviceReset is not supported once it has been looked up.  The array is shared by all calls and keeps whatever the last call
 * left in it.  Nothing in it has to start at zero: the gradient is copied over its input region and the
 * kernel writes every packed word and every scale before they are copied back.  Two calls that overlap in
 * time on one device (different host threads or streams) use the same bytes and race; serialise them.
 */
#define DQ_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
dq_status dqsg_encode_host_static(const float* grad, uint64_t n, uint64_t seed, uint32_t worker, uint64_t step,
                                  const dq_params* p, uint32_t* out_packed, float* out_scale,
                                  void* cuda_stream);

/*
 * dq_device_error_flags -- reads (and clears) the current device's error word: DQ_ERR_COPY_TIMEOUT is
 * set if any kernel of this library gave up waiting for one of its own asynchronous copies.
 * Synchronises the device.
 */
dq_status dq_device_error_flags(uint32_t* out_flags);

/* Number of kernel launches issued by this library in the calling process so far. */
uint64_t dq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DQ_H_ */
