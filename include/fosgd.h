/*
 * libfosgd: the gradient-compression round trip of FO-SGD ("flattened one-bit SGD",
 * arXiv 2405.11095) on one NVIDIA B200 (sm_100a).
 *
 * One iteration of the protocol (paper, Section 4): every worker n flips the signs of its
 * gradient with a random eps_n, applies the orthonormal Walsh-Hadamard transform H, adds
 * a uniform dither in [-lambda, lambda] and keeps one sign bit per coordinate (uplink).  The
 * server decodes every worker with that worker's eps_n, averages, and encodes the average
 * again with its own eps^s, amplitude lambda^s and K dithers (downlink).  Workers decode.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers owned by the caller.  The library allocates
 *     nothing and does not synchronise: work is enqueued on `stream` and the call returns
 *     (the one exception is the health check fosgd_async_timeouts, which waits for the device).
 *     Its only state between calls is diagnostic (the last CUDA error and the trace hooks per
 *     host thread, the timeout counter per device) plus the built-in scratch of
 *     fosgd_decode_noalloc.
 *   - d is the true gradient length; d' = fosgd_padded_dim(d, block_log2) is the length the
 *     transform runs on.  block_log2 = 0: one transform of length d' = next power of two
 *     (>= 32).  block_log2 = b in [5, 30]: independent transforms on consecutive blocks of
 *     2^b coordinates, d' = d rounded up to a multiple of 2^b (a variant outside the
 *     paper's Theorem 5.5; the paper itself only treats d = 2^k).
 *   - Packed format (Remark 3.3): coordinate i lives in 32-bit word i >> 5 at bit i & 31;
 *     bit 1 means +1.  For K dithers the count c_i in {0..K} of non-negative signs is stored
 *     as P = fosgd_planes(K) bit planes, plane p (d'/32 words) holding bit p of c_i, and the
 *     encoder value of Def. 3.7 is 2 c_i - K.
 *   - Randomness is a pure function of (seed, step, id, coordinate): Philox4x32-10 with
 *     counter (c, domain, lo32 step, id) and key (lo32 seed, hi32 seed ^ hi32 step).
 *     Domain 0 gives eps (word j of 32 flips = output j&3 of counter j>>2; set bit = -1).
 *     Domain 1+k gives dither k: coordinate i = 128 G + 32 r + l uses output r of counter
 *     32 G + l; its top 24 bits k24 give tau = lambda * (2 k24 + 1 - 2^24) * 2^-24.
 *     id is the worker id, or FOSGD_SERVER_ID for the downlink.  The transmitted eps of the
 *     paper is replaced by this shared (seed, step, id).
 *   - sgn(0) = +1.
 *   - Pointers must be 16-byte aligned, worker_stride * sizeof(element) a multiple of 16.
 *   - `ws` is scratch, contents undefined on entry and exit.  fosgd_workspace_bytes gives
 *     the minimum (one worker in flight); the calls that take several workers batch as many
 *     per launch as a larger `ws` allows.  Transforms that fit one thread block's tile
 *     (length <= 2^15) need none (ws may be NULL, ws_bytes 0).  A decoder from one packed
 *     plane whose transform is longer than 2^25 keeps the output of its first pass in fp16
 *     beside the fp32 intermediate where `ws` has 1.5 times the minimum for at least one
 *     worker (it then batches ws_bytes / (1.5 * minimum) workers per launch): less traffic,
 *     same result bit for bit.  The optional one-kernel
 *     encoder (fosgd_set_fused_encoder) keeps 16 + 4 bytes per worker of progress words
 *     behind the intermediates: with FOSGD_FUSED_SYNC_BYTES(M) more than M times the minimum
 *     all M workers go in one launch, with exactly M times the minimum the last worker
 *     gets a launch of its own.
 *   - Return value: FOSGD_OK or a negative status.  On an argument, alignment, workspace,
 *     size or limit error (every status but FOSGD_ECUDA) nothing has been enqueued.
 *     FOSGD_ECUDA means a launch or a runtime call failed, possibly after earlier kernels of
 *     the same call were enqueued: outputs, scratch and the accumulator are then undefined;
 *     fosgd_last_cuda_error() (thread local) returns the cudaError_t.
 */
#ifndef FOSGD_H
#define FOSGD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* fosgd_stream; /* == cudaStream_t */

enum { FOSGD_F32 = 0, FOSGD_BF16 = 1 };
enum { FOSGD_AGG_BEGIN = 1, FOSGD_AGG_END = 2 };
enum {
    FOSGD_OP_ENCODE = 0,
    FOSGD_OP_DECODE = 1,
    FOSGD_OP_AGGREGATE = 2,
    FOSGD_OP_DOWNLINK_DECODE = 3,
    FOSGD_OP_FLATTEN = 4,
    FOSGD_OP_AMPLITUDES = 5,       /* fosgd_amplitudes, per_block = 0 */
    FOSGD_OP_BLOCK_AMPLITUDES = 6  /* fosgd_amplitudes, per_block = 1 */
};
enum {
    FOSGD_OK = 0,
    FOSGD_EINVAL = -1,       /* null pointer, d < 1, M < 1, K outside [1,255], bad lambda, bad block_log2, bad flags */
    FOSGD_EALIGN = -2,       /* pointer or worker stride not 16-byte aligned */
    FOSGD_EWORKSPACE = -3,   /* ws missing or smaller than fosgd_workspace_bytes */
    FOSGD_EUNSUPPORTED = -4, /* unknown dtype or op, d' > 2^31 */
    FOSGD_ECUDA = -5,        /* a kernel launch returned an error */
    FOSGD_ELIMIT = -6        /* size beyond the built-in scratch of fosgd_decode_noalloc */
};

#define FOSGD_SERVER_ID 0xFFFFFFFFu

/* d' (see above); -1 if d < 1, block_log2 is invalid or d' would exceed 2^31. */
int64_t fosgd_padded_dim(int64_t d, int block_log2);

/* P = ceil(log2(K + 1)) bit planes (Remark 3.3); 0 if K is outside [1, 255]. */
int fosgd_planes(int K);

/* Dither amplitudes of Theorem 5.5 (natural logarithm): lambda = alpha * B * sqrt(ln d_eff / d_eff)
 * and lambda^s = alpha^s * lambda * sqrt(ln d_eff); d_eff is the transform length (d' in
 * global mode, 2^block_log2 in blocked mode), B an a-priori bound on the gradient norm. */
float fosgd_lambda(double B, double alpha, int64_t d_eff);
float fosgd_lambda_server(double lambda, double alpha_s, int64_t d_eff);

/* Minimum scratch bytes for one call of `op` (FOSGD_OP_*) on these sizes -> *out. */
int fosgd_workspace_bytes(int op, int64_t d, int M, int dtype, int block_log2, int K, size_t* out);

/* Uplink encoder E_{eps,lambda} (Def. 3.7, Section 4 "Workers-to-server", K = 1) for workers
 * worker_id0 .. worker_id0 + M - 1.  grads: M gradients of d elements of `dtype`, worker n
 * starting at element n * worker_stride; coordinates d..d'-1 are taken as zero.
 * bits: [M][d'/32] words out. */
int fosgd_encode(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                 uint32_t worker_id0, uint64_t seed, uint64_t step, float lambda, int block_log2,
                 uint32_t* bits, void* ws, size_t ws_bytes, fosgd_stream stream);

/* The flattening transform alone (Def. 3.5): out[n][0..d') = H D_{eps_n} x_n, orthonormal
 * scaling, fp32, same inputs as fosgd_encode.  out: [M][d'] floats. */
int fosgd_flatten(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                  uint32_t worker_id0, uint64_t seed, uint64_t step, int block_log2,
                  float* out, void* ws, size_t ws_bytes, fosgd_stream stream);

/* Decoder D_{eps,lambda} (Def. 3.8) for one worker: out[0..d) = lambda * D_eps * H^T * q,
 * q_i = +-1 from bits ([d'/32] words).  out: d floats. */
int fosgd_decode(const uint32_t* bits, int64_t d, uint32_t worker_id, uint64_t seed, uint64_t step,
                 float lambda, int block_log2, float* out, void* ws, size_t ws_bytes,
                 fosgd_stream stream);

/* Server side (Section 4, "Decoding", eq. (4.1), "Server-to-workers: Encoding").
 * Adds the M workers of this chunk (ids worker_id0 .. +M-1, bits [M][d'/32]) into the fp32
 * accumulator acc[d']: acc (=, with FOSGD_AGG_BEGIN, else +=) sum_n D_{eps_n} H^T q_n in
 * unnormalised integer units.  With FOSGD_AGG_END the sum is scaled by
 * lambda / (N_total * sqrt(transform length)), so that acc holds the average gbar of all
 * N_total workers on all d' coordinates, and, if down_bits is not NULL, gbar is encoded with
 * (FOSGD_SERVER_ID, lambda_s, K) into P = fosgd_planes(K) planes of d'/32 words.
 * A single call with flags = BEGIN | END handles all workers at once; chunked calls must
 * pass the same N_total, lambda, seed, step and cover each worker exactly once.
 * lambda_s and K are read only when END is set and down_bits is not NULL. */
int fosgd_server_aggregate(const uint32_t* bits, int64_t d, int M, uint32_t worker_id0, int N_total,
                           uint64_t seed, uint64_t step, float lambda, int block_log2,
                           float* acc, int flags, float lambda_s, int K, uint32_t* down_bits,
                           void* ws, size_t ws_bytes, fosgd_stream stream);

/* Downlink decoder D_{eps^s,lambda^s,K} (Def. 3.8, Section 4 "Server-to-workers: Decoding"):
 * out[0..d) = (lambda_s / K) * D_{eps^s} * H^T * (2c - K).  down_bits: [P][d'/32]. */
int fosgd_downlink_decode(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step,
                          float lambda_s, int K, int block_log2, float* out, void* ws,
                          size_t ws_bytes, fosgd_stream stream);

/* Amplitudes measured on the device and left there, so that no host round trip separates the
 * norm pass from the encoder (the paper takes the norm bound B as known a priori: this pass over
 * the gradients is an optional convenience, not part of the encode path).
 *   per_block = 0 (Theorem 5.5 with B = max_n ||g_n||_2 over the M gradients of the call):
 *     lambda_dev[0] = alpha * B * sqrt(ln n / n), lambda_s_dev[0] = alpha_s * lambda * sqrt(ln n),
 *     n the transform length.  ws: M * 2048 bytes (FOSGD_OP_AMPLITUDES).
 *   per_block = 1 (blocked mode only, block_log2 = b >= 5; nb = d' >> b blocks): every worker and
 *     block gets the amplitude of its own norm, lambda_dev[n * nb + k] = alpha * ||g_n restricted
 *     to block k||_2 * sqrt(ln 2^b / 2^b) (the flattening bound of Lemma 3.6 applied to each
 *     block's transform), and lambda_s_dev[k] = alpha_s * max_n lambda_dev[n * nb + k] *
 *     sqrt(ln 2^b), because ||Z(x)||_2 <= lambda sqrt(n) (Remark 5.2) bounds the averaged block.
 *     Amplitudes are floored at 1e-30, so that the bits of an all-zero block are still decided by
 *     the dither; such a block decodes to values of that size.  ws: FOSGD_OP_BLOCK_AMPLITUDES.
 * lambda_s_dev may be NULL (not written).  Sums of squares are taken in fp64 in a fixed order:
 * the result is reproducible.  Device pointers; alpha, alpha_s > 0. */
int fosgd_amplitudes(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M, double alpha,
                     double alpha_s, int block_log2, int per_block, float* lambda_dev, float* lambda_s_dev,
                     void* ws, size_t ws_bytes, fosgd_stream stream);

/* The three calls of the round trip with the amplitudes read from device memory, in either
 * layout of fosgd_amplitudes.  Same definitions and arguments as fosgd_encode,
 * fosgd_server_aggregate and fosgd_downlink_decode otherwise.  With per_block = 1 row n of
 * lambda_dev belongs to worker worker_id0 + n of the call, and the server average weights each
 * worker's decoded block by that worker's amplitude (Def. 3.8 per block).  lambda_s_dev is read
 * only where the downlink is encoded or decoded.  The amplitudes are not range-checked. */
int fosgd_encode_dev(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M,
                     uint32_t worker_id0, uint64_t seed, uint64_t step, const float* lambda_dev, int per_block,
                     int block_log2, uint32_t* bits, void* ws, size_t ws_bytes, fosgd_stream stream);
int fosgd_server_aggregate_dev(const uint32_t* bits, int64_t d, int M, uint32_t worker_id0, int N_total,
                               uint64_t seed, uint64_t step, const float* lambda_dev, const float* lambda_s_dev,
                               int per_block, int block_log2, float* acc, int flags, int K, uint32_t* down_bits,
                               void* ws, size_t ws_bytes, fosgd_stream stream);
int fosgd_downlink_decode_dev(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step,
                              const float* lambda_s_dev, int per_block, int K, int block_log2, float* out, void* ws,
                              size_t ws_bytes, fosgd_stream stream);

/* The server's downlink encoder alone (Section 4 downlink "Encoding": E_{eps^s, lambda^s, K} of
 * Def. 3.7 applied to the average), for servers whose average is completed outside
 * fosgd_server_aggregate (partial averages summed across GPUs).  gbar: d' = fosgd_padded_dim(d,
 * block_log2) floats (every entry is input: the transform of the average has no padding of its
 * own); down_bits: [P][d'/32] words out, identical to what fosgd_server_aggregate writes for the
 * same average.  lambda^s by value (lambda_s_dev NULL, per_block 0) or from device memory in either
 * layout of fosgd_amplitudes. */
int fosgd_downlink_encode(const float* gbar, int64_t d, uint64_t seed, uint64_t step, float lambda_s,
                          const float* lambda_s_dev, int per_block, int K, int block_log2, uint32_t* down_bits,
                          void* ws, size_t ws_bytes, fosgd_stream stream);

/* Worker update of Section 4, eq. (4.2), fused into the downlink decoder: x[i] <- x[i] -
 * step_size * g^d[i] for i < d, where g^d = D_{eps^s, lambda^s, K}(down_bits) is what
 * fosgd_downlink_decode returns; the decoded vector itself is not stored.  x: d floats in device
 * memory, read and written.  lambda^s by value (lambda_s_dev NULL, per_block 0) or from device
 * memory in either layout of fosgd_amplitudes (then lambda_s is ignored).  step_size finite and
 * non-zero.  Other arguments and errors as fosgd_downlink_decode. */
int fosgd_downlink_apply(const uint32_t* down_bits, int64_t d, uint64_t seed, uint64_t step, float lambda_s,
                         const float* lambda_s_dev, int per_block, int K, int block_log2, float step_size,
                         float* x, void* ws, size_t ws_bytes, fosgd_stream stream);

/* fosgd_amplitudes (one amplitude for all workers, per_block = 0) and fosgd_encode_dev in one call, for the
 * usual case that the gradients just encoded are the ones whose norm sets the amplitude (Theorem 5.5 with
 * B = max_n ||g_n||_2 over the M workers of the call).  lambda_dev (and lambda_s_dev, nullable) receive the
 * amplitudes as fosgd_amplitudes writes them; the packed signs are those of fosgd_encode_dev with that lambda.
 * Where the first strided pass of the encoder can carry the sums (fp32 gradients, transform length 2^20 ..
 * 2^24 in global or blocked mode, `ws` holding all M workers) the gradients are read once instead of twice;
 * elsewhere the call runs the two calls one after the other.  The sums are added in a fixed order, so the
 * amplitudes are reproducible, but in another order than fosgd_amplitudes uses: the two may differ in the
 * last bit.  amp_ws: scratch of fosgd_workspace_bytes(FOSGD_OP_AMPLITUDES, ..., M, ...) bytes. */
int fosgd_encode_measured(const void* grads, int dtype, int64_t d, int64_t worker_stride, int M, uint32_t worker_id0,
                          uint64_t seed, uint64_t step, double alpha, double alpha_s, int block_log2, float* lambda_dev,
                          float* lambda_s_dev, uint32_t* bits, void* ws, size_t ws_bytes, void* amp_ws,
                          size_t amp_ws_bytes, fosgd_stream stream);

/* fosgd_decode without a scratch argument (the paper has no counterpart; it computes exactly
 * what fosgd_decode computes).  For callers that must not allocate device memory where they
 * decode (no allocator reachable from their code, cudaMalloc banned because it synchronises,
 * or no memory left to ask for), the scratch is a fixed array of FOSGD_NOALLOC_SCRATCH_BYTES
 * inside the library image; every GPU that loads the library holds it until the process ends.
 *   - Limit: the scratch that fosgd_workspace_bytes(FOSGD_OP_DECODE, ...) asks for must fit,
 *     i.e. a decoder whose transform takes several passes (transform length above 2^15, in
 *     global or blocked mode) is accepted up to d' = 2^20 coordinates (d' floats of scratch);
 *     single-pass decoders need no scratch and are accepted at any size.  Beyond the limit the
 *     call returns FOSGD_ELIMIT and enqueues nothing.  The decoder's own argument checks
 *     (FOSGD_EINVAL, FOSGD_EALIGN) come first.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.  Later calls only launch.
 *   - The call allocates nothing and frees nothing.
 *   - All calls on a device share the one array.  Nothing in it needs clearing between calls
 *     (each call overwrites what it reads), but two calls whose kernels may run at the same
 *     time on one GPU (different streams, or different host threads) race on it: serialise them. */
#define FOSGD_NOALLOC_SCRATCH_BYTES ((size_t)4 << 20)
int fosgd_decode_noalloc(const uint32_t* bits, int64_t d, uint32_t worker_id, uint64_t seed,
                         uint64_t step, float lambda, int block_log2, float* out, fosgd_stream stream);

/* Health check (no counterpart in the paper).  The streaming kernels wait for their asynchronous
 * tile copies with a bounded number of polls; a thread block whose wait runs out stops working
 * and bumps a device counter instead of spinning forever.  *count receives the number of such
 * events on the current device since the library was loaded: 0 in a healthy run, anything else
 * means the outputs of some call are incomplete.  This call synchronises the device. */
int fosgd_async_timeouts(int* count);

/* Profiling aid (no counterpart in the paper).  events: HOST array of 2*capacity cudaEvent_t
 * handles created by the caller with timing enabled, or NULL to switch tracing off.  While set,
 * every kernel launch issued by the calling thread records events[2k] before and events[2k+1]
 * after launch number k (k < capacity, at most 256), so that cudaEventElapsedTime gives each
 * kernel's duration.  Setting the array resets the launch counter.  Thread local. */
int fosgd_trace_passes(void** events, int capacity);
int fosgd_trace_count(void);            /* launches recorded since the array was set */
const char* fosgd_trace_label(int k);   /* e.g. "col10:f32->ws@4", "row14:ws->pack1@4", "row14:ws16->final@srv" (kernel, source->sink,
                                           workers of the launch, or "srv" for the server's own vector on the downlink); valid until the next call */

/* Which passes of a decoder that starts from one packed plane (fosgd_decode, fosgd_server_aggregate,
 * the downlink decoder with K = 1; transform lengths 2^20 .. 2^25) run on the tensor cores.  The
 * recursion H_k = H_1 (x) H_{k-1} below Def. 3.4 makes every Kronecker factor H_128 a legal 128 x 128
 * matrix product, and on the decode side all operands are exact small integers (Def. 3.8: q_i = +-1).
 *   FOSGD_TC_STRIDED     the ten strided stages as H_8 on packed bytes plus a 128 x 128 x 128 8-bit integer
 *                        product per block (tcgen05 kind::i8), instead of packed fp16 arithmetic on the
 *                        plain ALUs (launches of fewer than 256 tiles of 2^17 coordinates stay on the
 *                        plain ALUs: too few tiles to repay a block's set-up);
 *   FOSGD_TC_CONTIGUOUS  the contiguous pass on tiles of 2^14 (transform length 2^24) as H_4 in packed
 *                        fp16 while staging, a 128 x 128 x 128 fp16 product with fp32 accumulators in tensor
 *                        memory per tile and worker (tcgen05 kind::f16), and H_32, flip and the sum over
 *                        the workers in registers, instead of fp32 butterflies on the plain ALUs (launches
 *                        that sum fewer than three workers stay on the plain ALUs, which are faster there).
 *   FOSGD_TC_ANY_SIZE    apply the chosen passes also to launches below the size thresholds named above.
 * Either way the results are the same bit for bit (all values are integers below 2^24 in magnitude).
 * Default: FOSGD_TC_STRIDED | FOSGD_TC_CONTIGUOUS (each measured faster than its plain-ALU kernel on a B200).  Process-wide; returns the
 * previous mask. */
enum { FOSGD_TC_STRIDED = 1, FOSGD_TC_CONTIGUOUS = 2, FOSGD_TC_ANY_SIZE = 4 };
int fosgd_set_tensor_core_pass(int mask);

/* Kernel choice for the uplink encoder of fp32 gradients when the transform length is 2^24 (ten strided
 * stages, then contiguous tiles of 2^14).  With on == 0 (the default) the two passes run as two kernels, one
 * after the other.  With on != 0 both run as one persistent kernel: half of every thread block stages strided
 * tiles through the tensor copy engine while the other half transforms, dithers and packs the contiguous
 * tiles of workers whose strided pass is complete.  Same bits either way; measured on a B200 the two kernels
 * are the faster form, so the one-kernel form is an option, not the default.  Process-wide; returns the
 * previous setting. */
int fosgd_set_fused_encoder(int on);
#define FOSGD_FUSED_SYNC_BYTES(M) ((((size_t)(M) + 4) * 4 + 15) & ~(size_t)15)

/* Issue-rate probe (measurement aid; no counterpart in the paper).  Enqueues one kernel that
 * keeps every scheduler of every SM busy with independent register-resident chains of one
 * instruction kind: fp32 add, fp32 fused multiply-add, three-input integer logic, or 32-bit
 * integer multiply-add.  *lane_ops (HOST pointer) receives the number of lane operations the
 * kernel executes (threads x iters x operations per iteration); divided by the kernel's duration,
 * timed by the caller with events on `stream`, it is the rate the plain ALUs sustain on this
 * device at the clock it runs.  sink: DEVICE pointer to at least 4 writable bytes (never written
 * in practice).  iters in [1, 2^24]. */
enum { FOSGD_PROBE_FADD = 0, FOSGD_PROBE_FFMA = 1, FOSGD_PROBE_LOP3 = 2, FOSGD_PROBE_IMAD = 3 };
int fosgd_probe_issue_rate(int kind, int iters, double* lane_ops, uint32_t* sink, fosgd_stream stream);

const char* fosgd_strerror(int status);
int fosgd_last_cuda_error(void);
const char* fosgd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FOSGD_H */
