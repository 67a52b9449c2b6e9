/*
 * co3.h — C ABI of the CO3 uplink pipeline for NVIDIA B200 (sm_100a).
 *
 * CO3 ("Convert, Compress, Correct", arXiv 2204.08211) sends, per client and per round, the
 * gradient g corrected by a decayed error memory m, converted to a low-resolution floating-point
 * format and entropy-coded:
 *     v = g + gamma * m            Sec. IV-A (iii), error correction with memory decay gamma
 *     ghat = Q_fp(v)               Sec. IV-A (i), level form in Sec. V-B
 *     b = h_Hf(ghat)               Sec. IV-A (ii), element-wise Huffman coding, one code per layer
 *     m = v - ghat                 Algorithm 1, memory update (= gamma*m + g - ghat)
 * and the parameter server decodes all clients and averages, Sec. II-B (iv):
 *     avg = (1/U) * sum_u ghat^(u)
 *
 * Conventions for every entry point unless stated otherwise
 *   - Pointers marked [device] are CUDA device pointers owned by the caller; pointers marked
 *     [host] are ordinary host pointers.  The library allocates no memory and keeps no state
 *     between calls; scratch space is the caller's `workspace` (device, 256-byte aligned, size
 *     from co3_workspace_bytes), whose contents are undefined after a call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue
 *     work and return; they never synchronise.
 *   - The int return value reports what the host can see at once (null or misaligned pointers,
 *     unsupported sizes, workspace or capacity too small for the fixed part, launch failures).
 *     Everything that depends on device data (descriptor contents, a symbol without codeword, a
 *     payload that does not fit, a corrupt stream) is reported in the device-side co3_result,
 *     valid once the stream has been synchronised.  After a device-side error the outputs of
 *     that client are undefined but nothing is written outside the buffers given.  CO3_ERR_CUDA
 *     in a co3_result (a copy inside a kernel never completed) is reported for every client of
 *     the call: the kernels stop within about one time-out, and the error memories and streams
 *     of all clients of that call are undefined.
 *   - A gradient of one client is a flat fp32 vector of n_elem elements, cut into n_seg segments
 *     (layers) that are contiguous and in order: segs[0].elem_off == 0,
 *     segs[k+1].elem_off == segs[k].elem_off + segs[k].n_elem, sum of n_elem == n_elem.
 *     Segment k uses fmts[k] and codes[k] for every client: one code per layer, shared by
 *     all users (Sec. IV-A (ii)).  Clients are batched: client u's vector starts
 *     client_stride_elems * u elements after the base pointer.
 *   - fp32 buffers and streams must be 16-byte aligned.
 */
#ifndef CO3_H_
#define CO3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CO3_OK 0
#define CO3_ERR_INVALID_ARG 1  /* bad pointer/size, or descriptor contents rejected on the device */
#define CO3_ERR_CAPACITY 2     /* stream or workspace too small; nothing is written past the end */
#define CO3_ERR_NO_CODEWORD 3  /* a symbol occurred whose code length is 0 */
#define CO3_ERR_NONFINITE 4    /* NaN/Inf seen (count in n_nonfinite); the stream is still valid */
#define CO3_ERR_CORRUPT 5      /* decoder: header/offset mismatch or a bit pattern that is no codeword */
#define CO3_ERR_CUDA 6         /* a CUDA runtime call failed */

#define CO3_MAX_CODE_LEN 16    /* longest codeword */
#define CO3_CHUNK_SYMS 2048    /* the only chunk size supported */
#define CO3_SUB_SYMS 128       /* symbols per sub-chunk offset */

#define CO3_FMT_FLUSH_SUBNORMALS 1u

/*
 * Target format [sgn, exp, mant] of Sec. IV-A (i) / Sec. V-B, 1 + exp_bits + mant_bits <= 8,
 * exp_bits >= 2.  Levels for the scaled input t = v * scale are c_mant * 2^c_exp with
 * c_mant in {1 + a_1/2 + ... + a_mant/2^mant}, c_exp in {-(2^(exp-1)-2) .. 2^(exp-1)-1}; exponent
 * code 0 holds zero and, unless CO3_FMT_FLUSH_SUBNORMALS is set, the evenly spaced values below
 * the smallest normal level; the all-ones exponent code is never produced (inputs beyond the
 * largest level saturate to it).  Rounding is to the nearest level, ties to the even code.
 * `scale` is the exponent bias written as a multiplier (c_scale = 1/scale); the reconstructed
 * value is level * inv_scale with the stored inv_scale (normally fl32(1/scale)).
 * A symbol is sign << (exp+mant) | exponent code << mant | mantissa code; zero has sign 0.
 */
typedef struct {
    uint8_t exp_bits;
    uint8_t mant_bits;
    uint16_t flags;
    float scale;
    float inv_scale;
} co3_fmt;

/* Prefix code of one layer: len[s] in 0..CO3_MAX_CODE_LEN (0 = symbol s has no codeword),
 * bits[s] the codeword right-aligned, its most significant bit is transmitted first. */
typedef struct {
    uint8_t len[256];
    uint16_t bits[256];
} co3_code;

typedef struct {
    uint64_t elem_off;
    uint64_t n_elem;
} co3_seg;

/* Written on the device, one per client (encode/convert) or one per call (decode). */
typedef struct {
    int32_t status;           /* CO3_OK or the first error seen for this client */
    uint32_t first_bad_chunk; /* smallest chunk index that failed (CO3_ERR_CORRUPT / NO_CODEWORD) */
    uint64_t payload_bits;    /* r: sum of the codeword lengths (Sec. II-B (iii)) */
    uint64_t container_bytes; /* total stream size including header, tables and padding */
    uint64_t n_saturated;     /* finite inputs beyond the largest level (Sec. V-B boundary +-B) */
    uint64_t n_nonfinite;     /* NaN (sent as zero) and +-Inf (sent as +-B); their memory restarts at 0 */
} co3_result;

/* Text for a status code; never NULL. */
const char* co3_status_string(int status);

/*
 * Bytes of device workspace needed by any entry point for vectors of n_elem elements in n_seg
 * segments with n_clients clients per encode call (pass n_clients = 0 if only co3_convert,
 * co3_decode and co3_decode_aggregate are used).  Returns CO3_ERR_INVALID_ARG for an
 * unsupported chunk_syms or out == NULL.
 */
int co3_workspace_bytes(uint64_t n_elem, uint32_t n_seg, uint32_t n_clients, uint32_t chunk_syms,
                        size_t* out /* [host] */);

/* Upper bound of the size of one client's stream (every codeword CO3_MAX_CODE_LEN bits long). */
int co3_stream_capacity_bytes(uint64_t n_elem, uint32_t n_seg, uint32_t chunk_syms,
                              size_t* out /* [host] */);

/*
 * Correct, convert, update memory (Algorithm 1, the conversion and memory steps) for
 * n_clients clients, without coding.
 *   grad [device]  fp32, read only;  mem [device] fp32, updated in place: m <- v - ghat
 *   sym_out [device, nullable]  one byte per element, same strides as grad
 *   hist_out [device, nullable] uint64[n_seg][256]: occurrences of each symbol per segment summed
 *                               over the clients of this call (the statistics the code is fitted
 *                               to); overwritten, not accumulated
 *   res [device] co3_result[n_clients]
 */
int co3_convert(const float* grad, float* mem, float decay,
                const co3_fmt* fmts /* [device] n_seg */, const co3_seg* segs /* [device] n_seg */,
                uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                uint8_t* sym_out, uint64_t* hist_out, co3_result* res,
                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Symbol statistics alone (Sec. IV-A (ii): a Huffman code is designed for the distribution of its source, here the
 * symbols of Q_fp(g + decay * m) of this round): hist_out exactly as co3_convert would fill it, and nothing else is
 * written: grad and mem are both read only, so that the code can be fitted before the round is encoded in one pass by
 * co3_encode.  res [device] co3_result[n_clients] receives the saturation and non-finite counts the round will see.
 */
int co3_histogram(const float* grad, const float* mem, float decay,
                  const co3_fmt* fmts /* [device] n_seg */, const co3_seg* segs /* [device] n_seg */,
                  uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                  uint64_t* hist_out /* [device] uint64[n_seg][256] */, co3_result* res,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * The conversion with dithered rounding, which Sec. II-B (ii) allows for (the quantizer may be a stochastic mapping,
 * so that non-subtractive dither quantization can be implemented).  Reading: the dither is uniform over the step
 * between the two levels around the scaled value t, i.e. the upper level is taken iff
 *     R < (|t| - lower) / (upper - lower) * 2^24,
 * R a uniform 24-bit integer, so that the result averages to t itself; a t that is a level stays where it is, beyond
 * the largest level it saturates as in co3_convert, NaN and infinities are treated as there.  R is word p % 4, top
 * 24 bits, of Philox-4x32-10 (Salmon, Moraes, Dror, Shaw, SC 2011) with key (seed, 0) and counter (p / 4 low word,
 * p / 4 high word, client, layer index) for the element at place p of its layer: give every round another seed.
 * Everything else (arguments, outputs, statuses) is as in co3_convert, co3_histogram and co3_encode; the parameter
 * server needs neither the seed nor to know that the stream was dithered (co3_decode_aggregate as usual).
 */
int co3_convert_dither(const float* grad, float* mem, float decay,
                       const co3_fmt* fmts /* [device] n_seg */, const co3_seg* segs /* [device] n_seg */,
                       uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                       uint32_t seed, uint8_t* sym_out, uint64_t* hist_out, co3_result* res,
                       void* workspace, size_t workspace_bytes, void* stream);
int co3_histogram_dither(const float* grad, const float* mem, float decay,
                         const co3_fmt* fmts /* [device] n_seg */, const co3_seg* segs /* [device] n_seg */,
                         uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                         uint32_t seed, uint64_t* hist_out, co3_result* res,
                         void* workspace, size_t workspace_bytes, void* stream);
int co3_encode_dither(const float* grad, float* mem, float decay,
                      const co3_fmt* fmts, const co3_code* codes /* [device] n_seg */, const co3_seg* segs,
                      uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                      uint32_t seed, uint8_t* streams_out, size_t stream_capacity, uint32_t chunk_syms,
                      void* workspace, size_t workspace_bytes, co3_result* res, void* stream);

/*
 * co3_convert without a workspace argument (the paper has no counterpart; this exists for the host
 * program's sake).  Some callers are not allowed to obtain device memory at the point where they run
 * the conversion: a plug-in inside a server that handed all device memory to its own pool at start-up,
 * or a latency-bound loop that must never enter the CUDA allocator because an allocation can stall the
 * whole device.  For them the scratch space is a fixed array of CO3_STATIC_SCRATCH_BYTES inside the
 * library image (each GPU that loads the library carries one copy until the process ends).  This call,
 * and everything it calls, performs no cudaMalloc / cudaFree and no other allocating routine; inputs,
 * outputs and `res` are still the caller's, with the same meaning as in co3_convert.
 *   - Layouts whose workspace need (co3_workspace_bytes(n_elem, n_seg, 0, ...)) exceeds
 *     CO3_STATIC_SCRATCH_BYTES are refused with CO3_ERR_CAPACITY before anything is enqueued; the
 *     18-layer residual network layout (62 segments, 11.2 M elements) fits.
 *   - The first call on each device looks the array's device address up (with that device current) and
 *     keeps it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, which still holds the previous call's tables; whatever
 *     must start from zero is cleared at the start of each call.  Two calls whose kernels can overlap on
 *     the GPU (different streams without an ordering between them) race on it: order them.
 *   - Leave profiling (co3_profile_enable) off if event creation counts as allocation for you.
 */
#define CO3_STATIC_SCRATCH_BYTES (2u << 20)
int co3_convert_static(const float* grad, float* mem, float decay,
                       const co3_fmt* fmts /* [device] n_seg */, const co3_seg* segs /* [device] n_seg */,
                       uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                       uint8_t* sym_out, uint64_t* hist_out, co3_result* res, void* stream);

/*
 * Huffman code for one layer from 256 integer weights (Sec. IV-A (ii)); host function, all
 * pointers [host].  Every symbol fmt can produce takes part with weight max(w, 1); other symbols
 * get length 0.  Ties: a leaf before a merged node, leaves by symbol, merged nodes by age.
 * If the longest codeword would exceed CO3_MAX_CODE_LEN all weights are halved (not below 1) and
 * the construction repeats.  Codewords are canonical: sorted by (length, symbol), consecutive
 * values.  Returns CO3_ERR_INVALID_ARG for a bad fmt or a weight sum >= 2^63.
 */
int co3_code_build(const uint64_t* weights, const co3_fmt* fmt, co3_code* out);

/*
 * The same construction for n_seg layers at once on the device (one thread block per layer), so that a
 * code fitted to this round's histogram (co3_convert's hist_out) never leaves the GPU.  Tables are
 * identical, entry for entry, to co3_code_build's for the same weights and formats.
 *   weights   [device] uint64[n_seg][256]
 *   fmts      [device] n_seg
 *   codes_out [device] n_seg, fully overwritten (length 0, bits 0 for symbols without codeword)
 *   res       [device] one co3_result: CO3_ERR_INVALID_ARG if any layer has a bad fmt or a weight sum >= 2^63
 *                      (that layer's table is all zero then); 8-byte aligned
 * Asynchronous on `stream`; the return value covers only the host-side argument checks.
 */
int co3_code_build_device(const uint64_t* weights, const co3_fmt* fmts, uint32_t n_seg, co3_code* codes_out,
                          co3_result* res, void* stream);

/*
 * Fit of every layer's multiplier to this round's data, on the device (Sec. III: a layer's gradient entries
 * are modelled as zero-mean generalized normal, GenNorm(alpha, beta), with kurtosis
 * Gamma(5/beta) Gamma(1/beta) / Gamma(3/beta)^2 and variance alpha^2 Gamma(3/beta) / Gamma(1/beta);
 * Sec. IV-A (i): the bias is the one that minimises the expected squared conversion error under that model,
 * found numerically once per shape and tabulated, Sec. IV-B).  Per layer k, over all n_clients vectors:
 *     v = g + decay * m (v = g when mem is NULL);  sigma^2 = sum v^2 / N;  kurtosis = N sum v^4 / (sum v^2)^2
 *     beta = the shape with that kurtosis, kept inside the table's range [beta0, beta0 + (n_beta-1) dbeta]
 *     alpha = sigma * sqrt(Gamma(1/beta) / Gamma(3/beta))
 *     fmts[k].scale = exp(table(beta)) / alpha,  fmts[k].inv_scale = fl32(1 / scale)
 * where table is row seg_tab[k] (row 0 if seg_tab is NULL) of log_tab and is interpolated linearly; its entry i
 * is the natural logarithm of the best multiplier for alpha = 1 at shape beta0 + i * dbeta.  Sums are fp64 in a
 * fixed order (results do not depend on the launch shape or on timing); the other fields of fmts are not read.
 *   grad, mem [device]  as in co3_convert, both read only; mem nullable
 *   fmts [device]       n_seg entries; scale and inv_scale of every fitted layer are overwritten
 *   log_tab [device]    float[n_tab][n_beta];  seg_tab [device, nullable] uint32[n_seg], entries < n_tab
 *   stats_out [device, nullable] double[n_seg][4]: sigma, kurtosis, beta, alpha of every fitted layer
 *   res [device]        one co3_result: CO3_ERR_INVALID_ARG if a layer is empty, all zero or holds a non-finite
 *                       value, or its table index is out of range (first_bad_chunk = smallest such layer); those
 *                       layers' formats are left untouched
 *   workspace           sized by co3_workspace_bytes with this n_clients (>= 1)
 */
int co3_fit_scale(const float* grad, const float* mem, float decay, co3_fmt* fmts, const co3_seg* segs,
                  uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                  const float* log_tab, const uint32_t* seg_tab, uint32_t n_tab, uint32_t n_beta,
                  float beta0, float dbeta, double* stats_out, co3_result* res,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Error magnitude (Sec. VI, "Error magnitude": the memory term m_t against the gradient term g_t, the figure the
 * memory decay gamma is chosen by): per client u and layer k
 *     norms_out[(u * n_seg + k) * 2 + 0] = sum |g_i|,   norms_out[(u * n_seg + k) * 2 + 1] = sum |m_i|
 * over the layer's elements, fp64 sums in a fixed order (independent of the launch shape and of timing).  A
 * NaN in a layer gives NaN for that layer, an infinity gives infinity; nothing is reported as an error.
 *   grad, mem [device]  as in co3_convert, both read only
 *   norms_out [device]  double[n_clients][n_seg][2], fully overwritten
 *   res [device]        one co3_result (CO3_ERR_INVALID_ARG if the segment table is inconsistent)
 *   workspace           sized by co3_workspace_bytes with this n_clients (>= 1)
 */
int co3_error_magnitude(const float* grad, const float* mem, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
                        uint32_t n_clients, uint64_t client_stride_elems, double* norms_out, co3_result* res,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Huffman weights of every layer from its fitted model instead of from counted symbols (Sec. IV-A (ii): the code
 * is designed for the GenNorm distribution of the layer).  The weight of a symbol is floor(p * 2^30), p the
 * GenNorm(0, alpha, beta) mass of the inputs that the converter, with the layer's multiplier, sends to that
 * symbol's level (between the midpoints to the neighbouring levels; beyond the last level everything; zero
 * collects both signs); symbols the format never produces get 0.  Feed the result to co3_code_build_device.
 *   fmts [device]        n_seg formats with their multipliers (as left by co3_fit_scale, or the caller's)
 *   stats [device]       double[n_seg][4] laid out as co3_fit_scale's stats_out: beta at [2], alpha at [3]
 *   weights_out [device] uint64[n_seg][256], fully overwritten
 *   res [device]         one co3_result: CO3_ERR_INVALID_ARG if a layer's format, beta or alpha is unusable
 *                        (first_bad_chunk = smallest such layer; its weights are all zero)
 */
int co3_model_weights(const co3_fmt* fmts, const double* stats, uint32_t n_seg, uint64_t* weights_out,
                      co3_result* res, void* stream);

/*
 * Client uplink for n_clients clients, the three per-user updates of Algorithm 1 in one call, codes given:
 *     v = g + decay * m,  ghat = Q_fp(v)   (Sec. IV-A (iii), (i));   b = h_Hf(ghat): the codewords of the symbols
 *     of ghat concatenated element by element (Sec. II-B (iii), Sec. IV-A (ii));   m <- v - ghat.
 *   grad, mem, decay, fmts, segs, strides: as in co3_convert; mem is updated in place
 *   codes [device]        n_seg prefix-code tables; a symbol that occurs must have a codeword
 *   streams_out [device]  client u's container starts at streams_out + u * stream_capacity
 *                         (stream_capacity a multiple of 16); layout below
 *   res [device] co3_result[n_clients]
 * Container (little-endian; every section 16-byte aligned):
 *   header 64 B: u32 magic 'CO3S', u32 version 1, u32 n_seg, u32 chunk_syms, u32 sub_syms, u32 0,
 *                u64 n_elem, u64 n_chunks, u64 payload_words, u64 payload_bits, u64 total_bytes
 *   n_seg x { u64 n_elem, u64 first_chunk, u64 payload_bits }
 *   u64 word_off[n_chunks + 1]             payload word at which each chunk starts
 *   u16 bit_off[n_chunks][16]              bit offset of each run of 128 symbols inside its chunk
 *   u32 payload[payload_words]
 * A chunk holds up to 2048 consecutive symbols of one segment; its codewords are concatenated in
 * element order, bit j of the chunk is bit 31-(j%32) of its word j/32, unused bits are 0.
 */
int co3_encode(const float* grad, float* mem, float decay,
               const co3_fmt* fmts, const co3_code* codes /* [device] n_seg */, const co3_seg* segs,
               uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
               uint8_t* streams_out, size_t stream_capacity, uint32_t chunk_syms,
               void* workspace, size_t workspace_bytes, co3_result* res, void* stream);

/* The coding step alone, b = h_Hf(ghat) (Sec. II-B (iii), Sec. IV-A (ii)): the same container from symbols that
 * co3_convert produced, for the flow in which the code is fitted to this round's symbol statistics between
 * conversion and coding (Sec. IV-A (ii): the code is designed for the distribution of the source).
 * sym [device]: one byte per element, strides as for grad. */
int co3_encode_symbols(const uint8_t* sym, const co3_code* codes, const co3_seg* segs,
                       uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                       uint8_t* streams_out, size_t stream_capacity, uint32_t chunk_syms,
                       void* workspace, size_t workspace_bytes, co3_result* res, void* stream);

/*
 * Parameter server: decode n_clients streams and average (Sec. II-B (iv), Algorithm 1):
 * avg_out[i] = (ghat_i^(0) + ghat_i^(1) + ...) / n_clients, fp32 additions in client order and
 * one fp32 division.
 *   streams [device]  array of n_clients device pointers, each to a container of at least
 *                     stream_bytes readable bytes
 *   res [device]      one co3_result (payload_bits and container_bytes summed over clients)
 */
int co3_decode_aggregate(const uint8_t* const* streams, size_t stream_bytes, uint32_t n_clients,
                         const co3_fmt* fmts, const co3_code* codes, const co3_seg* segs,
                         uint32_t n_seg, uint64_t n_elem, uint32_t chunk_syms, float* avg_out,
                         void* workspace, size_t workspace_bytes, co3_result* res, void* stream);

/*
 * The same with the model update of Algorithm 1's last step folded in (w_{t+1} = w_t - eta/U * sum_u ghat^(u),
 * Sec. II-B (iv)): params[i] <- params[i] - lr * avg[i] with avg[i] exactly as co3_decode_aggregate forms
 * it; one fp32 multiplication and one fp32 subtraction per element, each rounded on its own.
 *   params [device]   n_elem model parameters, updated in place; 16-byte aligned
 *   avg_out [device]  nullable: the average itself, if the caller wants it too
 */
int co3_decode_aggregate_update(const uint8_t* const* streams, size_t stream_bytes, uint32_t n_clients,
                                const co3_fmt* fmts, const co3_code* codes, const co3_seg* segs,
                                uint32_t n_seg, uint64_t n_elem, uint32_t chunk_syms, float lr, float* params,
                                float* avg_out, void* workspace, size_t workspace_bytes, co3_result* res,
                                void* stream);

/* One stream: reconstructed values and/or symbols (either output may be NULL, not both). */
int co3_decode(const uint8_t* stream_in, size_t stream_bytes,
               const co3_fmt* fmts, const co3_code* codes, const co3_seg* segs,
               uint32_t n_seg, uint64_t n_elem, uint32_t chunk_syms,
               float* ghat_out, uint8_t* sym_out,
               void* workspace, size_t workspace_bytes, co3_result* res, void* stream);

/*
 * Diagnostics (no counterpart in the paper).  With profiling enabled every kernel launched by the
 * entry points above is bracketed by a CUDA event pair on the caller's stream; co3_profile_read
 * waits for those events, adds up the elapsed time and the number of launches per kernel kind
 * (arrays of CO3_KERNEL_COUNT entries, [host]) and clears the records.  Off by default; at most
 * 16384 launches are recorded between reads.  Not thread-safe, and not to be left on inside a
 * stream capture.
 */
#define CO3_KERNEL_PREPARE 0  /* descriptor (and, when decoding, stream header) validation, derived tables */
#define CO3_KERNEL_CONVERT 1  /* correct + convert + memory update (+ symbols, histogram) */
#define CO3_KERNEL_PACK 2     /* (correct + convert + memory update +) codeword lookup, scan, bit packing */
#define CO3_KERNEL_SCAN 3     /* chunk offsets, header, tables */
#define CO3_KERNEL_COMPACT 4  /* payload compaction */
#define CO3_KERNEL_CODE_BUILD 5 /* Huffman tables from weights on the device */
#define CO3_KERNEL_DECODE 6   /* decode + cross-client accumulate */
#define CO3_KERNEL_FIT 7      /* moments, multiplier fit, model weights, error magnitude */
#define CO3_KERNEL_CLEAR 8    /* zeroing of the call state, results and histogram at the start of a call */
#define CO3_KERNEL_COUNT 9
int co3_profile_enable(int on);
int co3_profile_read(double* total_ms /* [host] */, uint32_t* launches /* [host] */);

#ifdef __cplusplus
}
#endif
#endif /* CO3_H_ */
