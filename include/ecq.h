/*
 * ecq.h -- C ABI of the B200 (sm_100a) ECQ-SGD gradient codec.
 *
 * The library implements the per-worker, per-iteration codec of "Error
 * Compensated Quantized SGD" (Wu, Huang, Huang, Zhang, ICML 2018), Section 4,
 * on a flat fp32 gradient of d entries cut into contiguous buckets of `bucket`
 * entries (the last bucket may be shorter); each bucket carries its own scale.
 *
 * Conventions for every call
 *   - Returns an int status (ECQ_OK == 0); never throws, never exits.
 *   - Unless a parameter says "host", data pointers are DEVICE pointers owned
 *     by the caller; the library never frees or reallocates them.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL
 *     is the default stream) and the call returns without synchronising,
 *     unless stated otherwise.  Stream order is kept: a kernel of this library
 *     may be scheduled while the work ahead of it in the stream is finishing
 *     (programmatic dependent launch), but touches no global memory before
 *     that work has completed, so buffers may be reused from call to call.
 *   - `grad`, `err`, `out`, `codes` must be 16-byte aligned; `scales` 4-byte.
 *   - A context is immutable after creation (except the ecq_set_* calls) and may
 *     be used from several host threads on different streams.
 *   - Inputs must be finite.  A bucket whose compensated values contain NaN or
 *     Inf is sent as all-zero levels with scale 0, its accumulator entries are
 *     left unchanged, and ECQ_ERR_NONFINITE is recorded in the context's sticky
 *     device status word (see ecq_status).
 *
 * Wire format of one worker's message (paragraph after Eq. 9: r bits per entry
 * plus one fp32 scale per scaled vector, here per bucket)
 *   - scales[b], b < nb = ceil(d / bucket): the bucket's l-infinity norm of the
 *     compensated gradient (0 for an all-zero or non-finite bucket).
 *   - codes: a dense little-endian bit stream, entry i occupying stream bits
 *     [i*r, i*r + r), r = ceil(log2(2s+1)); stream bit k is bit (k mod 32) of
 *     32-bit word (k div 32).  Entry i holds q_i + s, q_i in [-s, s] the signed
 *     level.  Because bucket % 32 == 0 every bucket starts on a word boundary;
 *     the stream is padded with zero bits to ecq_codes_words() words.
 */
#ifndef ECQ_H_
#define ECQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ecq_ctx ecq_ctx;

#define ECQ_MAX_WORKERS 64          /* workers (messages) one kernel launch serves */
#define ECQ_MAX_WORKERS_TOTAL 1024  /* most workers ecq_encode_batch / ecq_decode_mean[_update] take */

enum {
    ECQ_OK = 0,
    ECQ_ERR_ARG = 1,        /* null / misaligned pointer, size or range violation */
    ECQ_ERR_CUDA = 2,       /* a CUDA runtime or driver call failed */
    ECQ_ERR_NONFINITE = 3,  /* NaN or Inf met in a compensated gradient (sticky, device) */
    ECQ_ERR_TIMEOUT = 4,    /* a bounded in-kernel wait on an async copy ran out (sticky, device) */
    ECQ_ERR_ALLOC = 5,      /* host or device allocation failed in ecq_create */
    ECQ_ERR_TOO_LARGE = 6,  /* ecq_step_static: the messages do not fit the built-in scratch */
    ECQ_ERR_CAPACITY = 7,   /* ecq_huffman_encode: the stream does not fit the buffer (sticky, device) */
    ECQ_ERR_SYMBOL = 8      /* a level without a code word / a bit pattern that is no word (sticky, device) */
};

/*
 * Create a codec context.
 *   d       entries of the flat gradient (>= 1)
 *   bucket  entries per bucket: multiple of 32, >= 32
 *   levels  s of Eq. 9, the number of non-zero quantisation levels, 1..32767
 *   alpha   compensation coefficient of Eq. 7 (>= 0)
 *   beta    time-decay factor of Eq. 5/6 (0 <= beta <= 1)
 *   seed    64-bit key of the Philox4x32-10 stream that drives Eq. 9
 * The context owns only constants and one 4-byte device status word on the
 * device that is current at the time of the call (device ordinals 0..63; beyond
 * that ECQ_ERR_CUDA).  ECQ_ERR_ARG on a range violation, ECQ_ERR_ALLOC /
 * ECQ_ERR_CUDA otherwise.
 */
int ecq_create(ecq_ctx** out, uint64_t d, uint32_t bucket, uint32_t levels,
               float alpha, float beta, uint64_t seed);

/* Release the context (NULL is allowed).  Synchronises nothing: do not destroy
 * a context with work in flight. */
void ecq_destroy(ecq_ctx* ctx);

/*
 * Choose what the error-accumulator update books.
 *   0 (default)  Eq. 6 as printed: h <- beta*h + (g - g~), g the raw gradient.
 *   1            h <- beta*h + ((g + alpha*h) - g~), the compensated value.
 */
int ecq_set_error_mode(ecq_ctx* ctx, int mode);

/*
 * Choose the scaling factor ||v|| of Eq. 8 (the paper leaves the norm open and names l2 and
 * l-infinity), taken per bucket.
 *   0 (default)  l-infinity: max |v_i|
 *   1            l2: sqrt(sum v_i^2).  The fp32 sum has a fixed order so that results do not
 *                depend on the kernel's shape: every run of 32 consecutive entries is summed
 *                front to back with one fused multiply-add per entry, the run sums are added
 *                pairwise in index order, level by level.  Entries below about 1e-19 in
 *                magnitude square to zero; a sum that overflows (entries beyond about 1e19)
 *                is reported as ECQ_ERR_NONFINITE.  Buckets that are not a power of two
 *                or exceed 4096 entries may have at most 32768 entries (else ECQ_ERR_ARG).
 * The receiver side is the same for both.
 */
int ecq_set_norm(ecq_ctx* ctx, int norm);

/*
 * Choose how the receiver side (Eq. 4; ecq_decode_mean and ecq_decode_mean_update) is
 * launched.  The result does not depend on the choice: every kernel sums the W terms of an
 * output in ascending worker order with one fused multiply-add per term.
 *   kernel    ECQ_DECODE_AUTO (default): by shape and length;
 *             ECQ_DECODE_WARP: tiles of 1024 outputs, every warp copies its own code words;
 *             ECQ_DECODE_RING: tiles of 30720 outputs, one bulk copy per (tile, worker)
 *             shared by the CTA (what AUTO takes for r <= 8 once a CTA has enough tiles:
 *             3 with 12 messages or more of up to 4 bits, 5 with 8 or more of 2 bits or
 *             12 or more of up to 8 bits, 12 otherwise).
 *             A shape that a kernel does not cover (bucket not a power of two, r > 9, more
 *             than bucket/4 workers for buckets under 1024; for RING also `out` or
 *             `params` not 32-byte aligned) falls through to the next one.
 *   max_ctas  upper limit on the CTAs of a launch; 0 = fill the device.
 * ECQ_ERR_ARG on an unknown kernel.
 */
#define ECQ_DECODE_AUTO 0
#define ECQ_DECODE_WARP 1
#define ECQ_DECODE_RING 2
int ecq_set_decode_plan(ecq_ctx* ctx, int kernel, uint32_t max_ctas);

/*
 * Set how many times a kernel polls for an asynchronous copy (a TMA or bulk load into
 * shared memory) before it gives up.  The paper has no counterpart: this is the library's
 * guard against a copy that never completes.  A wait that runs out makes its CTA stop,
 * records ECQ_ERR_TIMEOUT in the sticky status word (ecq_status), lets the copies still in
 * flight land -- that last wait always keeps the built-in limit of 2^22 polls, whatever is
 * set here -- and returns; buffers the CTA had not finished are left partly written, and
 * the context stays usable.  Default 2^22 (a fraction of a second; no copy takes that
 * long).  0 makes every wait give up at once without polling: the only use of small
 * values is to exercise that path.
 */
#define ECQ_WAIT_LIMIT_DEFAULT (1u << 22)
int ecq_set_wait_limit(ecq_ctx* ctx, uint32_t polls);

/* r = ceil(log2(2s+1)): bits per entry (paragraph after Eq. 9). */
uint32_t ecq_code_bits(const ecq_ctx* ctx);
/* nb = ceil(d / bucket): floats in one worker's `scales`. */
uint64_t ecq_num_buckets(const ecq_ctx* ctx);
/* ceil(d*r / 32): 32-bit words in one worker's `codes`. */
uint64_t ecq_codes_words(const ecq_ctx* ctx);

/*
 * Sender side, one worker, one iteration (Algorithm 1, phase 1: the quantisation step,
 * which applies Eq. 7, and the accumulator step, which applies Eq. 6, fused):
 *   v = grad + alpha*err                            (Eq. 7)
 *   scale_b = max over the bucket of |v_i|          (Eq. 8, l-infinity norm)
 *   level m_i in {floor(x), floor(x)+1}, x = s|v_i|/scale_b, going up with
 *   probability x - floor(x), decided by the Philox word of counter
 *   (i/4, worker, step) under key `seed`            (Eq. 9)
 *   q_i = sgn(v_i) m_i,  g~_i = q_i * (scale_b / s) (Eq. 8)
 *   err_i <- beta*err_i + (grad_i - g~_i)           (Eq. 6; see ecq_set_error_mode)
 *   codes, scales <- the message                    (wire format above)
 *
 *   worker, step  identify the random stream; the same (seed, worker, step)
 *                 always gives the same draws
 *   grad   [d]    in, never written
 *   err    [d]    in/out, the accumulator h of this worker; must be zero before
 *                 the first iteration (h(0) = 0)
 *   codes  [ecq_codes_words()]  out
 *   scales [ecq_num_buckets()]  out
 * Buffers of different workers must not overlap.  ECQ_ERR_ARG on null or
 * misaligned pointers; ECQ_ERR_CUDA if the launch fails.
 */
int ecq_encode(ecq_ctx* ctx, uint32_t worker, uint32_t step, const float* grad,
               float* err, uint32_t* codes, float* scales, void* cuda_stream);

/*
 * ecq_encode for workers 0..W-1 of one iteration in ONE kernel launch (Algorithm 1,
 * the loop over the P nodes of phase 1, on a single GPU that holds all P workers'
 * slices).  Results are identical to W calls of ecq_encode(ctx, w, step, grads[w],
 * errs[w], codes[w], scales[w]); a single launch spares W-1 launch ramps and tails,
 * which matters for vectors of tens of megabytes.  Beyond ECQ_MAX_WORKERS workers there
 * is one launch per ECQ_MAX_WORKERS of them, with the same results.
 *   W       1..ECQ_MAX_WORKERS_TOTAL
 *   grads, errs, codes, scales   HOST arrays of W device pointers each, with the
 *           meaning, sizes and alignment of ecq_encode's arguments; read before the
 *           call returns
 */
int ecq_encode_batch(ecq_ctx* ctx, uint32_t W, uint32_t step, const float* const* grads,
                     float* const* errs, uint32_t* const* codes, float* const* scales,
                     void* cuda_stream);

/*
 * Receiver side (Eq. 4 and Algorithm 1, phase 2, global-gradient step):
 *   out_i = (1/W) * sum_{w<W} q_{w,i} * (scales_w[b(i)] / s)
 *   W       number of messages, 1..ECQ_MAX_WORKERS_TOTAL
 *   codes   HOST array of W device pointers to the workers' code streams
 *   scales  HOST array of W device pointers to the workers' scales
 *   out [d] the averaged dequantised gradient
 * The two pointer arrays are read before the call returns.  Up to ECQ_MAX_WORKERS
 * messages are summed in one launch; beyond that there is one launch per
 * ECQ_MAX_WORKERS messages, each continuing the sum of the previous one (kept in
 * `out` meanwhile) in the same ascending order of w, so the result is the same
 * chain of fp32 operations as a single pass.  The long-vector kernels carry the
 * level steps times a power of two (2^-22, and 1/W when W is a power of two):
 * exact, except that level steps below 2^-94 may lose low-order bits, an error
 * far below any gradient that matters.
 */
int ecq_decode_mean(ecq_ctx* ctx, uint32_t W, const uint32_t* const* codes,
                    const float* const* scales, float* out, void* cuda_stream);

/*
 * Receiver side with the model update fused in (Algorithm 1, phase 2: the global-gradient
 * step followed by the model-update step, w(t+1) = w(t) - eta * g~(t)):
 *   g~_i     = the mean ecq_decode_mean would produce
 *   params_i <- fma(-eta, g~_i, params_i)       (one rounding)
 *   out_i    = g~_i when out is not NULL
 *   params [d]  in/out, 16-byte aligned; out [d] or NULL, must not alias params
 *   W       as in ecq_decode_mean; with more than ECQ_MAX_WORKERS messages `out` is
 *           required (it carries the running sum between launches; ECQ_ERR_ARG if NULL)
 * Saves the separate pass over the decoded gradient that an optimiser step would make.
 */
int ecq_decode_mean_update(ecq_ctx* ctx, uint32_t W, const uint32_t* const* codes,
                           const float* const* scales, float eta, float* params, float* out,
                           void* cuda_stream);

/*
 * Level statistics of one message (paragraph after Eq. 9: with d_k entries on the k-th
 * of the 2s+1 levels, an entropy code needs at most sum_k d_k log2(d / d_k) bits).
 *   codes   [ecq_codes_words()] device, one worker's code stream
 *   counts  [2s+1] device uint64, 8-byte aligned: counts[k] = entries whose level is k - s;
 *           zeroed and filled by the call (asynchronously on the stream)
 */
int ecq_code_histogram(ecq_ctx* ctx, const uint32_t* codes, uint64_t* counts, void* cuda_stream);

/* sum_k d_k log2(d / d_k) over the non-empty bins of HOST counts, d = sum_k d_k. */
double ecq_entropy_bound_bits(const uint64_t* counts_host, uint32_t n_bins);

/*
 * Entropy-coded message.  The paragraph after Eq. 9 notes that the r-bit codes can be
 * compressed further by an entropy code (the paper names Huffman coding as one) with at most
 * sum_k d_k log2(d / d_k) bits, and the linear-model experiments count their
 * communication that way.  The paper fixes no format; this one is the library's:
 *   - a prefix code over the 2s+1 level indices, optimal among codes whose words have at
 *     most ECQ_HUFFMAN_MAX_LEN bits (Huffman's code whenever that has no longer word);
 *   - canonical words: symbols ordered by (length, index), the first word all zeros, each
 *     next one = (previous + 1) shifted left by the growth in length;
 *   - a word's bits are sent first-bit first into a stream of 32-bit words, bit k of the
 *     stream being bit k mod 32 of word k / 32;
 *   - entries are cut into chunks of ECQ_HUFFMAN_CHUNK; every chunk starts on a word
 *     boundary; offsets[c] is the first word of chunk c, offsets[n_chunks] the stream
 *     length in words;
 *   - quarters[3c + j] (j = 0, 1, 2) is the bit, counted from the first word of chunk c,
 *     at which entry 256 (j + 1) of that chunk starts (the chunk's end if it has fewer
 *     entries): four readers can share a chunk.
 *     A message on the wire is (lengths, offsets, quarters, stream, scales).
 * Available for levels <= 2047 (r <= 12); ECQ_ERR_ARG beyond.
 *
 * ecq_huffman_lengths   HOST only: lengths_host[k] (k < 2s+1) from the level counts of
 *                       ecq_code_histogram, 0 for a level that does not occur, 1 when a
 *                       single level occurs.
 * ecq_huffman_chunks    ceil(d / ECQ_HUFFMAN_CHUNK).
 * ecq_huffman_stream_bound   HOST only: words that are always enough for the stream of a
 *                       message with these counts under these lengths.
 * ecq_huffman_tables    builds the encoder and decoder tables of a code from its lengths
 *                       (HOST, ECQ_ERR_ARG if they are no prefix code) and copies them to
 *                       tables_dev (ECQ_HUFFMAN_TABLE_BYTES, 16-byte aligned, device) on
 *                       the stream; lengths_host may be reused when the call returns.
 * ecq_huffman_encode    codes [ecq_codes_words()] -> stream_words [capacity_words],
 *                       offsets [ecq_huffman_chunks() + 1] and quarters
 *                       [3 * ecq_huffman_chunks()], all device.  If the stream
 *                       needs more than capacity_words nothing is written to stream_words
 *                       and ECQ_ERR_CAPACITY becomes pending; a level without a word makes
 *                       ECQ_ERR_SYMBOL pending (both are read by ecq_status).
 * ecq_huffman_decode    the inverse: stream_words [stream_len_words] (16-byte aligned),
 *                       offsets, quarters -> codes [ecq_codes_words()], bit-identical to what was encoded.  Nothing
 *                       beyond stream_len_words is read, whatever the offsets say.  A bit
 *                       pattern that is no word ends its chunk (rest zero) and makes
 *                       ECQ_ERR_SYMBOL pending.
 */
#define ECQ_HUFFMAN_MAX_LEN 12
#define ECQ_HUFFMAN_CHUNK 1024
#define ECQ_HUFFMAN_TABLE_BYTES (4096 * 4 + 4096 * 4 + 16)
int ecq_huffman_lengths(const ecq_ctx* ctx, const uint64_t* counts_host, uint8_t* lengths_host);
uint64_t ecq_huffman_chunks(const ecq_ctx* ctx);
uint64_t ecq_huffman_stream_bound(const ecq_ctx* ctx, const uint64_t* counts_host,
                                  const uint8_t* lengths_host);
int ecq_huffman_tables(ecq_ctx* ctx, const uint8_t* lengths_host, void* tables_dev,
                       void* cuda_stream);
int ecq_huffman_encode(ecq_ctx* ctx, const void* tables_dev, const uint32_t* codes,
                       uint32_t* stream_words, uint64_t capacity_words, uint32_t* offsets,
                       uint16_t* quarters, void* cuda_stream);
int ecq_huffman_decode(ecq_ctx* ctx, const void* tables_dev, const uint32_t* stream_words,
                       uint64_t stream_len_words, const uint32_t* offsets,
                       const uint16_t* quarters, uint32_t* codes, void* cuda_stream);

/*
 * One whole iteration from HOST gradients to a HOST result: for every worker
 * copy its gradient to the device, ecq_encode it, then ecq_decode_mean all W
 * messages and copy the mean back.  Copies of worker w+1 overlap the encode of
 * worker w.  The call returns after `out_host` is complete.
 *   grads_host  HOST array of W HOST pointers, [d] floats each (pinned memory
 *               makes the copies asynchronous; pageable memory also works)
 *   err_dev     [W*d] device floats: the W accumulators, worker-major, kept by
 *               the caller between iterations (zero before the first one)
 *   workspace_dev, workspace_bytes
 *               caller-owned device scratch of at least
 *               ecq_step_host_workspace_bytes(ctx, W) bytes, 256-byte aligned
 *   out_host    [d] HOST floats
 */
uint64_t ecq_step_host_workspace_bytes(const ecq_ctx* ctx, uint32_t W);
int ecq_step_host(ecq_ctx* ctx, uint32_t W, uint32_t step,
                  const float* const* grads_host, float* err_dev,
                  void* workspace_dev, uint64_t workspace_bytes,
                  float* out_host, void* cuda_stream);

/*
 * One whole iteration on DEVICE buffers for callers that must not allocate.
 * (The paper has no counterpart: this entry point exists for the embedding, not
 * for the method.)
 *
 * Who needs it: code that runs where device allocation is forbidden or cannot be
 * afforded -- inside a memory pool that owns all of the GPU's memory, in a plugin
 * called from another framework's hot loop, in a process whose allocator must not
 * be re-entered.  ecq_create and the caller-owned message buffers of ecq_encode /
 * ecq_decode_mean both need allocations; this call needs neither a context nor
 * message buffers.  It runs W encodes and one decode-mean exactly like
 * ecq_encode (worker w, iteration `step`, error mode 0) and ecq_decode_mean
 * would, keeping the W messages and the status word in a scratch array that is
 * compiled into the library: ECQ_STATIC_SCRATCH_BYTES of device memory that every
 * GPU on which the library is loaded holds until the process exits.
 *
 *   d, bucket, levels, alpha, beta, seed   as in ecq_create
 *   W        1..ECQ_MAX_WORKERS
 *   grads    HOST array of W device pointers, [d] floats each (read only)
 *   err      [W*d] device floats, worker-major accumulators (in/out)
 *   out      [d] device floats, the decoded mean
 * The scratch must hold 256 + W * (roundup256(4*ceil(d*r/32)) + roundup256(4*ceil(d/bucket)))
 * bytes; larger problems are refused with ECQ_ERR_TOO_LARGE before anything is
 * launched.  d must be a multiple of 4 when W > 1 (16-byte aligned accumulators).
 *
 * The call enqueues on `cuda_stream`, waits for it, and returns ECQ_OK,
 * ECQ_ERR_NONFINITE or ECQ_ERR_TIMEOUT like ecq_status would.  It calls no
 * cudaMalloc / cudaFree and no allocating library routine (a host thread's first
 * call binds the device's primary context with cudaSetDevice; kernels are loaded
 * by the CUDA runtime on first use as for any library).  The first call on a
 * device (ordinals 0..63; beyond that ECQ_ERR_CUDA) looks up the scratch array's
 * device address (with that device current); make that first call outside any
 * stream capture.  All calls on a device share
 * the one array and it keeps the last call's contents: the status word is cleared
 * at the start of every call, the messages are fully overwritten; two calls that
 * overlap on the GPU (different streams or host threads) race on it and must be
 * serialised by the caller.
 */
#define ECQ_STATIC_SCRATCH_BYTES (4u << 20)
int ecq_step_static(uint64_t d, uint32_t bucket, uint32_t levels, float alpha, float beta,
                    uint64_t seed, uint32_t W, uint32_t step, const float* const* grads,
                    float* err, float* out, void* cuda_stream);

/*
 * Synchronise `cuda_stream`, then return and clear the context's sticky device
 * status: ECQ_OK, ECQ_ERR_NONFINITE, ECQ_ERR_TIMEOUT, or ECQ_ERR_CUDA if the
 * stream itself reports an error.
 */
int ecq_status(ecq_ctx* ctx, void* cuda_stream);

/* Number of kernels this library has launched in this process (all contexts). */
uint64_t ecq_launch_count(void);

/* Static description of a status code. */
const char* ecq_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ECQ_H_ */
