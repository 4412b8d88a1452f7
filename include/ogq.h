/*
 * ogq.h -- C ABI of the optimal-gradient-quantization library (CUDA, sm_100a).
 *
 * The library implements the per-tensor quantization path of "Optimal Gradient
 * Quantization Condition for Communication-Efficient Distributed Training":
 * runtime level solvers for BinGrad-b, BinGrad-pb and ORQ, quantize + bit-pack,
 * and the server-side unpack + dequantize + sum over K workers.
 *
 * Conventions shared by every entry point
 *   - A bucket is a flat fp32 array `grad` of `total_elems` elements holding T
 *     tensors back to back: tensor t is grad[off[t] .. off[t+1]), off[0] = 0,
 *     off[T] = total_elems, off non-decreasing.  Empty tensors are allowed.
 *   - Pointers named d_* are DEVICE pointers owned by the caller; pointers named
 *     h_* are HOST pointers.  d_grad, d_out and every packed buffer must be
 *     16-byte aligned; tensor offsets need no alignment (tensors whose offset
 *     is not a multiple of 4 elements take a scalar-load path).
 *   - The library allocates no memory and keeps no state between calls on the data
 *     path (only the measurement helpers at the end keep host-side records).  Scratch
 *     memory is the caller's `d_ws` of at least ogq_workspace_bytes(...) bytes,
 *     256-byte aligned; its contents need not be preserved or initialised.
 *   - Calls only enqueue work on `stream` and return at once.  The return code
 *     reports argument validation and launch errors.  Conditions that depend on
 *     the data are reported per tensor in d_status (bits OGQ_ST_*), never by a
 *     trap.  There is no CPU fallback.
 *   - Levels are fp32 because they are what a worker sends next to its codes.
 *   - Size limit of the selection solvers (ogq_levels_orq, ogq_levels_bingrad with
 *     OGQ_BINGRAD_PB): total_elems below 2^32, because they count a tensor's elements in
 *     32-bit cells; larger buckets return OGQ_ERR_UNSUPPORTED and enqueue nothing.
 */
#ifndef OGQ_H_
#define OGQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *ogq_stream_t; /* a cudaStream_t */

typedef enum {
    OGQ_OK = 0,
    OGQ_ERR_INVALID_ARG = 1,
    OGQ_ERR_UNSUPPORTED = 2,
    OGQ_ERR_WORKSPACE = 3,
    OGQ_ERR_CUDA = 4,
    OGQ_ERR_LIMIT = 5 /* the request exceeds a fixed capacity of the entry point */
} ogq_status;

typedef enum { OGQ_BINGRAD_PB = 0, OGQ_BINGRAD_B = 1, OGQ_ORQ = 2 } ogq_scheme;

/* per-tensor status bits written to d_status */
#define OGQ_ST_EMPTY 1      /* tensor has no elements; its levels are 0 */
#define OGQ_ST_NONFINITE 2  /* NaN or Inf seen; levels are 0 (ORQ, pb) or unspecified (b) */
#define OGQ_ST_CONSTANT 4   /* all elements equal (one side of the split empty): all levels equal */
#define OGQ_ST_ITER_CAP 8   /* an iteration limit was reached before convergence */
#define OGQ_ST_INTERNAL 16  /* a solver bracket failed to contain its target (should not happen) */

/* Library version string (static storage). */
const char *ogq_version(void);

/* Code width in bits for s levels: 1 for s = 2, ceil(log2 s) otherwise; 0 if s < 2 or s > 32. */
int ogq_bits_for_levels(int s);

/*
 * Packed layout (the paper's Algorithm 2 only says "encode"; this is the wire
 * format of this library).  Per tensor a little-endian bit stream of 32-bit
 * words: the code of element i occupies stream bits [i*bits, (i+1)*bits),
 * stream bit j is bit (j mod 32) of word j/32, and each tensor's region is zero
 * padded to a multiple of 4 words.  Fills h_packed_off[0..T] (in words) from
 * the host copy of the element offsets.  Host-only; no device work.
 */
ogq_status ogq_packed_layout(const int64_t *h_off, int T, int bits, int64_t *h_packed_off);

/*
 * Upper bound of the scratch bytes any level solver needs for a bucket of
 * `num_tensors` tensors and `total_elems` elements with at most `max_levels`
 * levels.  Host-only.
 */
size_t ogq_workspace_bytes(int num_tensors, int64_t total_elems, int max_levels);

/*
 * BinGrad levels (Section "Binary Quantization").
 *   variant OGQ_BINGRAD_B : Eq. (bingrad-b optimal condition).  b_0 starts at the
 *     tensor mean; b_{-1}, b_1 are the means of {v < b_0} and {v >= b_0}.  With
 *     lloyd_iters = I > 0 the update b_0 = (b_{-1} + b_1)/2 followed by new means
 *     is applied up to I times, stopping when the split no longer changes
 *     (OGQ_ST_ITER_CAP if it still changed after I updates).  b_0 is rounded to
 *     fp32 at every step, since it is the threshold the quantizer compares with.
 *   variant OGQ_BINGRAD_PB: Eq. (bingrad-pb optimal condition) on |v|: b_1 is where
 *     g(b) = b n - sum_{|v| >= b} |v| changes sign (the minimiser of the
 *     quantizer's squared error); levels are {-b_1, +b_1}; lloyd_iters is ignored.
 * Outputs: d_levels [T][2] = {b_{-1}, b_1}; d_thresh [T] = b_0 (B only, may be
 * NULL for PB); d_status [T].
 */
ogq_status ogq_levels_bingrad(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems,
                              int variant, int lloyd_iters, float *d_levels, float *d_thresh,
                              int32_t *d_status, void *d_ws, size_t ws_bytes, ogq_stream_t stream);

/*
 * BinGrad-b levels without caller-provided scratch.  The paper has no counterpart; this exists
 * for callers that must not allocate device memory: code that runs where the allocator is off
 * limits (a plugin or communication hook invoked in the middle of a training step, a process
 * whose memory pool is owned and fully reserved by another component, a strict real-time loop
 * where cudaMalloc's implicit synchronisation is unacceptable) and that cannot size and keep an
 * ogq_workspace_bytes() buffer either.  Same results as ogq_levels_bingrad(..., OGQ_BINGRAD_B,
 * ...): the same kernels run, but their partial-sum slots and counters live in a fixed array
 * inside the library image instead of d_ws.
 *   - Capacity: at most OGQ_NOALLOC_MAX_TENSORS tensors per call (any element count).  More
 *     returns OGQ_ERR_LIMIT and enqueues nothing.  The array costs every GPU that loads the
 *     library about 304 KB of device memory until the process exits.
 *   - The call allocates and frees nothing.  The first call on each device looks up the array's
 *     device address (with that device current); make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array.  The part a call uses is cleared on `stream`
 *     before its kernels run, so leftovers of earlier calls do no harm, but two calls whose
 *     work overlaps on the GPU (different streams, no ordering between them) race on it and
 *     give wrong levels.  Order such calls, or use ogq_levels_bingrad with separate scratch.
 *   - OGQ_ERR_LIMIT comes only from the tensor-count check above; a failing CUDA call is
 *     OGQ_ERR_CUDA.  Host threads may make the first call on a device concurrently (the
 *     address lookup is idempotent and its result is stored atomically).
 */
#define OGQ_NOALLOC_MAX_TENSORS 1024
ogq_status ogq_levels_bingrad_b_noalloc(const float *d_grad, const int64_t *d_off, int T,
                                        int64_t total_elems, int lloyd_iters, float *d_levels,
                                        float *d_thresh, int32_t *d_status, ogq_stream_t stream);

/*
 * ORQ levels (Algorithm 1 with the discrete form of the simplified optimal
 * condition).  s in {3, 5, 9, 17}.  The end levels are the tensor's minimum and
 * maximum (Corollary 1); every other level is the middle of its two bracket
 * levels L < R: with T = sum_{L <= v <= R} (v - L) / (R - L), it is the
 * (floor(T) + 1)-th largest element of {L <= v <= R}, so every level is one of
 * the tensor's own values, found by exact selection (no sampling, no
 * approximation of ranks).  T itself is evaluated in fp64 from exact integer
 * partial sums; where T lies within fp64 rounding of an integer, the data value
 * next to the one a higher-precision evaluation picks may be returned (both
 * then satisfy the condition to rounding).
 * Output: d_levels [T][s] ascending, d_status [T].
 */
ogq_status ogq_levels_orq(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems, int s,
                          float *d_levels, int32_t *d_status, void *d_ws, size_t ws_bytes,
                          ogq_stream_t stream);

/*
 * Quantize and pack (the random-rounding equation of Section "Multi-level
 * Quantization", Eq. (bingrad-pb), Eq. (bingrad-b), then "encode").
 *   ORQ / BINGRAD_PB (s = 2): segment k = 1 + #{interior levels <= v}, lo = b_{k-1},
 *     hi = b_k; the code is k if  (float)u * (hi - lo) < (v - lo) * 2^24  (each
 *     operation in fp32, round to nearest), else k - 1; u is the top 24 bits of
 *     word (i mod 4) of Philox4x32-10 with key (seed low, seed high) and counter
 *     (i/4 low, i/4 high, tensor index, stream_id), i the index inside the tensor.
 *     Values outside [b_0, b_{s-1}] get the nearest end code.
 *   BINGRAD_B: code = [v >= d_thresh[t]]; no random numbers; d_levels is unused.
 * d_levels is [T][s], d_thresh is [T] (B only), d_packed_off [T+1] comes from
 * ogq_packed_layout, d_packed receives d_packed_off[T] words (all of them are
 * written, padding included).
 */
ogq_status ogq_quantize_pack(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems,
                             ogq_scheme scheme, int s, const float *d_levels, const float *d_thresh,
                             uint64_t seed, uint32_t stream_id, const int64_t *d_packed_off,
                             uint32_t *d_packed, ogq_stream_t stream);

/*
 * Server step of Algorithm 2: out[i] = scale * sum_{k<K} levels_k[t][code_k[i]],
 * summed in fp32 in worker order k = 0..K-1.  d_packed_k and d_levels_k are
 * DEVICE arrays of K device pointers (worker k's packed buffer and its [T][s]
 * level table).  1 <= K <= 64.  scale = 1/K gives the broadcast average.
 */
ogq_status ogq_unpack_sum(const uint32_t *const *d_packed_k, const float *const *d_levels_k, int K,
                          const int64_t *d_off, const int64_t *d_packed_off, int T, int64_t total_elems,
                          int s, float scale, float *d_out, ogq_stream_t stream);

/*
 * Quantization error per tensor, d_err [T] in fp64 (a diagnostic, not on the encode path).
 *   ogq_quant_error: the realised error of bit-packed codes, sum_i (levels[code_i] - v_i)^2,
 *     the ||Q(G) - G||^2 the paper records during training (Section "Performance" of the CIFAR
 *     experiments and its training-curve figure).  s = 2 decodes 1-bit codes of either BinGrad.
 *   ogq_expected_error: its expectation over the random rounding, sum_i (v_i - lo_i)(hi_i - v_i)
 *     with lo, hi the levels around v_i (the functional in the proof of Theorem 1); a value
 *     outside the levels counts with its squared distance to the end level.
 * Sums are fp64 per thread, combined with one fp64 atomic per CTA and tensor piece: the last
 * bits can differ from run to run.
 */
ogq_status ogq_quant_error(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems, int s,
                           const float *d_levels, const int64_t *d_packed_off, const uint32_t *d_packed,
                           double *d_err, ogq_stream_t stream);
ogq_status ogq_expected_error(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems, int s,
                              const float *d_levels, double *d_err, ogq_stream_t stream);

/*
 * Entropy-dense wire format (Tables of the CIFAR-100 and ImageNet results: compression ratios
 * x20.2, x13.8, x10.1 for 3, 5, 9 levels, i.e. 32 / log2(s): a code is taken to cost log2(s)
 * bits).  The closest whole-word format: M consecutive codes of a tensor are the base-s digits,
 * least significant first, of one 32-bit word, M = ogq_dense_digits(s) the largest count with
 * s^M <= 2^32 (s = 3: 20, 5: 13, 9: 10, 17: 7; 0 for other s), so ratios x20 / x13 / x10 / x7
 * against x16 / x10.7 / x8 / x6.4 of the bit-packed format.  Word j of a tensor holds elements
 * j M ... j M + M - 1, missing elements count as code 0, and regions are zero padded to a
 * multiple of 4 words (ogq_dense_layout, host-only, fills h_packed_off[0..T]).
 *   ogq_quantize_pack_dense: the ORQ quantizer of ogq_quantize_pack (same segment search, same
 *     Philox counters, same rounding decision, hence the same codes), packed in this format.
 *   ogq_unpack_sum_dense: ogq_unpack_sum for this format.
 */
int ogq_dense_digits(int s);
ogq_status ogq_dense_layout(const int64_t *h_off, int T, int s, int64_t *h_packed_off);
ogq_status ogq_quantize_pack_dense(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems,
                                   int s, const float *d_levels, uint64_t seed, uint32_t stream_id,
                                   const int64_t *d_packed_off, uint32_t *d_packed, ogq_stream_t stream);
ogq_status ogq_unpack_sum_dense(const uint32_t *const *d_packed_k, const float *const *d_levels_k, int K,
                                const int64_t *d_off, const int64_t *d_packed_off, int T,
                                int64_t total_elems, int s, float scale, float *d_out,
                                ogq_stream_t stream);

/*
 * Gradient clipping (Section "Experiments", paragraph after the list of methods):
 * clip(v) = sign(v) min(|v|, c sigma), sigma^2 the variance of the gradient being quantized
 * (here: of each tensor, about its mean, over all its elements), c = 2.5 in the ImageNet runs,
 * 1.7 or 2.5 in the clipping-factor table.
 *   ogq_clip_threshold: d_tau[t] = fp32(c * sigma_t) from one streaming read; d_status[t] gets
 *     OGQ_ST_EMPTY or OGQ_ST_NONFINITE (then d_tau[t] = 0), else 0.  Scratch as for
 *     ogq_levels_bingrad (ogq_workspace_bytes).
 *   ogq_levels_orq_clipped / ogq_levels_bingrad_clipped: the level solvers on the clipped
 *     gradient; the clamp to [-d_tau[t], d_tau[t]] is applied as the values are read, the clipped
 *     gradient is never written out.  ORQ's end levels become the clipped extremes.  A non-finite
 *     value is clipped like any other, so it is ogq_clip_threshold that reports it.
 *   ogq_quantize_pack_clipped: ogq_quantize_pack with the same clamp applied first, so that the
 *     codes are exactly those of the clipped gradient (plain ogq_quantize_pack with the clipped
 *     levels decodes to the same values but may pick another of several equal levels for a value
 *     beyond +-tau).
 */
ogq_status ogq_clip_threshold(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems,
                              float c, float *d_tau, int32_t *d_status, void *d_ws, size_t ws_bytes,
                              ogq_stream_t stream);
ogq_status ogq_levels_orq_clipped(const float *d_grad, const int64_t *d_off, int T, int64_t total_elems,
                                  int s, const float *d_tau, float *d_levels, int32_t *d_status,
                                  void *d_ws, size_t ws_bytes, ogq_stream_t stream);
ogq_status ogq_levels_bingrad_clipped(const float *d_grad, const int64_t *d_off, int T,
                                      int64_t total_elems, int variant, int lloyd_iters,
                                      const float *d_tau, float *d_levels, float *d_thresh,
                                      int32_t *d_status, void *d_ws, size_t ws_bytes,
                                      ogq_stream_t stream);
ogq_status ogq_quantize_pack_clipped(const float *d_grad, const int64_t *d_off, int T,
                                     int64_t total_elems, ogq_scheme scheme, int s,
                                     const float *d_levels, const float *d_thresh, const float *d_tau,
                                     uint64_t seed, uint32_t stream_id, const int64_t *d_packed_off,
                                     uint32_t *d_packed, ogq_stream_t stream);

/*
 * Fixed-length bucket mode (Section "Experiments", first paragraph: "bucket-based quantization
 * ... evenly divides the whole gradient into buckets of the same length d and quantizes each
 * bucket independently"; d = 2048 on CIFAR, 512 on ImageNet, 128 ... 32768 in the bucket-size
 * table).  One call does levels + quantize + pack for every bucket of d_grad[0 .. total_elems):
 * bucket j is elements [j d, min((j+1) d, total_elems)), nb = ceil(total_elems / d) buckets.
 * Each bucket is read from HBM once, sorted in shared memory, solved and packed by one CTA.
 * The results are those of ogq_levels_* followed by ogq_quantize_pack on a bucket of nb tensors
 * with offsets j d: same level definitions, Philox tensor index = j, and the packed layout of
 * ogq_packed_layout for those offsets (bucket j starts at word j * d * bits / 32;
 * ogq_bucket_packed_words gives the total).  ogq_unpack_sum decodes it with the same offsets.
 *   d      multiple of 128, 128 <= d <= 32768 (else OGQ_ERR_UNSUPPORTED)
 *   scheme OGQ_ORQ (s in {3, 5, 9, 17}), OGQ_BINGRAD_B or OGQ_BINGRAD_PB (s = 2)
 *   iters  OGQ_ORQ: refinement sweeps after Algorithm 1 (0 = the paper's greedy levels).  One
 *          sweep re-solves every interior level, in ascending order, from its two current
 *          neighbours, b_k = Q*(b_{k-1}, b_{k+1}); sweeps stop early when one changes nothing
 *          (the paper's conclusion names the greedy algorithm as open to improvement; each
 *          sweep cannot increase the expected quantization error).
 *          OGQ_BINGRAD_B: Lloyd updates, as lloyd_iters of ogq_levels_bingrad.  PB: ignored.
 *   clip_c 0: no clipping.  > 0: every bucket is first clipped to +-clip_c times its own standard
 *          deviation (see ogq_clip_threshold; ImageNet setting of the paper: d = 512, c = 2.5).
 * Outputs: d_levels [nb][s], d_thresh [nb] (B only, may be NULL otherwise), d_status [nb],
 * d_packed.  No scratch memory is needed.
 */
int64_t ogq_bucket_packed_words(int64_t total_elems, int d, int bits);
ogq_status ogq_bucket_encode(const float *d_grad, int64_t total_elems, int d, ogq_scheme scheme, int s,
                             int iters, float clip_c, uint64_t seed, uint32_t stream_id, float *d_levels,
                             float *d_thresh, int32_t *d_status, uint32_t *d_packed,
                             ogq_stream_t stream);

/*
 * Server step of Algorithm 2 for fixed-length buckets: out[i] = scale * sum_{k<K}
 * levels_k[i / d][code_k[i]], fp32 sum in worker order, the result ogq_unpack_sum gives for
 * offsets j d.  d_packed_k / d_levels_k: DEVICE arrays of K device pointers to the workers' packed
 * buffers and [nb][s] level tables as ogq_bucket_encode wrote them.  1 <= K <= 64.  No scratch.
 */
ogq_status ogq_bucket_decode_sum(const uint32_t *const *d_packed_k, const float *const *d_levels_k, int K,
                                 int64_t total_elems, int d, int s, float scale, float *d_out,
                                 ogq_stream_t stream);

/*
 * Measurement helpers (no counterpart in the paper; they do not touch the data path).
 * ogq_launch_count: number of kernels this library has launched in this process so far.
 * ogq_profile_enable(1): from now on every kernel launch of the library is bracketed by two CUDA
 *   events recorded on the launch stream; ogq_profile_enable(0) stops recording.  Turning it on
 *   discards earlier records.  Process-wide and not thread-safe: use it from one thread, around
 *   whole calls, and never while a stream is being captured.
 * ogq_profile_collect: waits for the recorded events, then writes up to max_records entries:
 *   h_ms[i] is the device time of launch i in milliseconds and h_names receives the kernel
 *   names, each padded to name_stride bytes (NUL terminated).  Returns the number of records
 *   written and clears them.
 */
unsigned long long ogq_launch_count(void);
int ogq_profile_enable(int on);
int ogq_profile_collect(float *h_ms, char *h_names, int name_stride, int max_records);

#ifdef __cplusplus
}
#endif
#endif /* OGQ_H_ */
