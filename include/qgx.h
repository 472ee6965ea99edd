/*
 * qgx -- the data-parallel hot path of Q-GenX (quantized generalized extra-gradient,
 * arXiv 2308.09187) for one NVIDIA B200 (sm_100a), as a C library.
 *
 * The paper's K processors are K slices of one GPU's memory: a "[K][d]" array holds worker
 * k's vector at offset k*d.  A vector is cut into buckets of `bucket` coordinates (the last
 * one may be shorter; nb = ceil(d / bucket)); Definition 1 is applied to every bucket on its
 * own, with the bucket's own norm.
 *
 * Conventions for every entry point unless its comment says otherwise:
 *  - pointers marked [dev] are device pointers, owned by the caller, and must stay valid until
 *    the context's stream has run the call; pointers marked [host] are read (or written) before
 *    the call returns;
 *  - calls are asynchronous on the stream given to qgx_create and return a qgx_status for what
 *    the host could check; errors found on the device (non-finite norm, capacity, corrupt
 *    stream, a bounded wait that ran out) are latched in the context and reported by
 *    qgx_sync_status, which synchronizes the stream.  No call aborts, traps or prints;
 *  - the library allocates device memory only inside qgx_create and when a call needs a larger
 *    workspace than any call before it (the fused calls and qgx_update_levels).
 *
 * Symbol byte: bits 0..4 level index, bit 7 sign (set only when the level index is nonzero).
 * Stream: 32-bit words, bit p of a stream is bit (p & 31) of word (p >> 5).
 */
#ifndef QGX_H_
#define QGX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QGX_OK = 0,
  QGX_ERR_INVALID_ARG = 1,
  QGX_ERR_BAD_LEVELS = 2,   /* nlev outside [2,32], endpoints not 0 and 1, or not strictly increasing */
  QGX_ERR_CAPACITY = 3,     /* a worker's stream does not fit cap_words */
  QGX_ERR_CORRUPT = 4,      /* a stream that no encoder could have produced */
  QGX_ERR_NONFINITE = 5,    /* a bucket norm is NaN or infinite */
  QGX_ERR_TIMEOUT = 6,      /* a bounded device-side wait ran out */
  QGX_ERR_CUDA = 7,         /* the CUDA runtime reported an error */
  QGX_ERR_TOO_LARGE = 8     /* the problem exceeds the fixed scratch of qgx_encode_noalloc */
} qgx_status;

enum { QGX_NORM_L2 = 0, QGX_NORM_LINF = 1 };
enum { QGX_CODE_FIXED = 0, QGX_CODE_HUFFMAN = 1, QGX_CODE_ELIAS = 2 };
enum { QGX_OP_DENSE_AFFINE = 0, QGX_OP_BILINEAR = 1, QGX_OP_DIAGONAL = 2 };
enum { QGX_REFIT_NONE = 0, QGX_REFIT_CONTINUE = 1, QGX_REFIT_FIRST = 2 };
/* flag of qgx_quantize: `norms` is an input (the caller's norms are used as they are) */
enum { QGX_NORMS_SUPPLIED = 1 };

enum { QGX_MAX_LEVELS = 32, QGX_MAX_CODE_LEN = 12, QGX_MAX_BUCKET = 16384 };

typedef struct qgx_ctx qgx_ctx;

/* Prefix code Psi of App. J over the level indices.  code[j] holds the codeword of level j as an
 * integer of len[j] bits whose most significant bit is sent first.  subblock = number of
 * coordinates per sub-block of a bucket (a multiple of 4); <= 0 or >= bucket means none. */
typedef struct {
  int32_t nlev;
  int32_t maxlen;
  int32_t subblock;
  uint8_t len[32];
  uint32_t code[32];
} qgx_codebook;

/* Quantizer configuration (Definition 1 + Sec. 3.2).  levels[0] = 0 < ... < levels[nlev-1] = 1.
 * nlev counts every entry of the table, the end points 0 and 1 among them.  Definition 1 writes the table as
 * 0 = l_0 < l_1 < ... < l_s < l_{s+1} = 1, so its s (the free levels between the end points) is nlev - 2; where the
 * paper's experiments speak of "s levels" of a uniform quantizer with s quantization intervals, the table has
 * nlev = s + 1 entries (the convention of the benchmark's configurations). */
typedef struct {
  int32_t nlev;
  int32_t bucket;           /* multiple of 4, <= QGX_MAX_BUCKET */
  int32_t norm_type;        /* QGX_NORM_L2 | QGX_NORM_LINF */
  int32_t code_type;        /* what a refit rebuilds: QGX_CODE_FIXED | QGX_CODE_HUFFMAN | QGX_CODE_ELIAS */
  int32_t nbins;            /* histogram bins of the level refit (Sec. 3.3) */
  int32_t pad;
  uint64_t seed;            /* key of the counter-based generator */
  float levels[32];
  qgx_codebook cb;
} qgx_quant_cfg;

enum { QGX_NOISE_ADDITIVE = 0, QGX_NOISE_RELATIVE = 1 };

/* Monotone operator A of the VI (Sec. 2).  DENSE_AFFINE: A(x) = M x + b, M row-major d x d.
 * BILINEAR: the game min_x max_y x^T A y with z = (x, y), A n x n row-major, d = 2n,
 * A(z) = (A y, -A^T x).  DIAGONAL: A(x) = D .* x.  mat and bias are [dev]. */
typedef struct {
  int32_t kind;
  int32_t noise_model;      /* how a worker's noise array enters its dual vector: QGX_NOISE_ADDITIVE (Assumption 2)
                             * V_k = A(x) + U_k; QGX_NOISE_RELATIVE (Assumption 3, e.g. random player updating)
                             * V_k = A(x) .* S_k with non-negative scales of mean one */
  uint64_t d;
  const float *mat;
  const float *bias;        /* DENSE_AFFINE only; may be NULL */
} qgx_operator;

/* State of Algorithm 1.  The vectors are [dev] float[d], caller-owned.  scalars is [dev]
 * double[2] = { sum of squared differences, gamma_t }; t (host) counts iterations from 1. */
typedef struct {
  uint64_t d;
  int32_t K;
  int32_t t;
  float *X;                 /* X_t */
  float *Y;                 /* Y_t */
  float *Xbar;              /* (1/t) sum of X_{i+1/2}: the ergodic average of Theorems 3 and 4 */
  float *Xhalf;             /* X_{t+1/2} of the last step */
  const float *anchor;      /* X_1; the update is X_{t+1} = anchor + gamma_{t+1} Y_{t+1} */
  double *scalars;
} qgx_eg_state;

/* ---- context ------------------------------------------------------------------------------ */

/* Creates a context on `device` whose calls run on `cuda_stream` (a cudaStream_t; NULL = the
 * default stream).  Allocates a small status block.  Returns QGX_ERR_CUDA if there is no usable
 * device: there is no CPU fallback. */
qgx_status qgx_create(qgx_ctx **ctx, int device, void *cuda_stream);
void qgx_destroy(qgx_ctx *ctx);
/* Synchronizes the stream and returns the first error latched by a device-side check since the
 * last call of this function (QGX_OK if none), clearing it. */
qgx_status qgx_sync_status(qgx_ctx *ctx);
const char *qgx_status_str(qgx_status s);
/* How many kernels of this library the context has launched so far. */
uint64_t qgx_launch_count(const qgx_ctx *ctx);

/* Per-kernel device timing for benchmarks (no counterpart in the paper).  qgx_timing_enable
 * allocates `max_records` event pairs (0 switches timing off and frees them); while on, every
 * launch of the kernels named below is bracketed by two events on the context's stream.
 * qgx_timing_read synchronizes, returns the number of recorded launches of `kernel` and their
 * summed duration in milliseconds, and forgets the records read so far of every kernel when
 * `reset` is nonzero. */
enum { QGX_KERNEL_ENCODE = 0, QGX_KERNEL_DECODE = 1, QGX_KERNEL_HISTOGRAM = 2, QGX_KERNEL_OPERATOR = 3,
       QGX_KERNEL_FINISH = 4, QGX_KERNEL_COUNT = 5 };
qgx_status qgx_timing_enable(qgx_ctx *ctx, int max_records);
qgx_status qgx_timing_read(qgx_ctx *ctx, int kernel, int reset, int *launches /*[host] out*/,
                           double *total_ms /*[host] out*/);

/* ---- host helpers ------------------------------------------------------------------------- */

/* QGX_OK iff the table is admissible for Definition 1. */
qgx_status qgx_check_levels(const float *levels /*[host]*/, int nlev);
/* Worst-case 32-bit words of one worker's stream: per bucket 32 (norm, C_b of App. E) +
 * 16 per sub-block + (maxlen + 1) per coordinate bits, rounded up to whole words. */
size_t qgx_stream_capacity_words(size_t d, int bucket, int subblock, int maxlen);
/* Fixed-length code: every level index costs ceil(log2 nlev) bits. */
qgx_status qgx_build_codebook_fixed(int nlev, int subblock, qgx_codebook *cb /*[host] out*/);
/* Huffman code (App. J) for symbol weights p[nlev] [host]; canonical codewords ordered by
 * (length, index); if the longest codeword would exceed QGX_MAX_CODE_LEN the weights are
 * flattened by adding 2^(m-16), m = 0, 1, ..., until it fits. */
qgx_status qgx_build_codebook_huffman(const double *p, int nlev, int subblock, qgx_codebook *cb);
/* Elias' recursive code (App. J: the choice when the distribution of the levels is unknown but small
 * levels are known to be frequent): level j is sent as the codeword of the integer j + 1 -- the bit 0
 * preceded by groups, the last group the binary form of the integer, each earlier group the binary
 * form of the following group's bit count minus one.  At most 12 bits for 32 levels; independent of
 * any weights.  cb [host] out. */
qgx_status qgx_build_codebook_elias(int nlev, int subblock, qgx_codebook *cb);
/* Level fit of Sec. 3.3 on a histogram hist[nbins] [host] of normalized magnitudes, read as a
 * piecewise-uniform density: coordinate descent on the (QAda) objective, each interior level
 * moved to the root of the objective's derivative with its neighbours fixed; at most 32 sweeps.
 * first_fit != 0 starts from the mass quantiles, otherwise from levels[] as passed in.
 * levels [host] in/out. */
qgx_status qgx_fit_levels(const double *hist, int nbins, float *levels, int nlev, int first_fit);
/* Symbol weights p[nlev] [host] out of the proposition on the code pmf (App. E). */
qgx_status qgx_symbol_pmf(const double *hist, int nbins, const float *levels, int nlev, double *p);

/* ---- the four steps of one exchange (Algorithm 1: quantize, encode | decode, aggregate) ---- */

/* Definition 1 per bucket.  v [dev] float[K][d] -> norms [dev] float[K][nb] (L2: square root
 * of the fp64 sum of squares, rounded once to fp32; with QGX_NORMS_SUPPLIED in flags norms is
 * read instead) and sym [dev] uint8[K][d].  Coordinate i of worker k in exchange `exchange_id`
 * rounds up iff (w >> 8) * 2^-24 < xi, w = word (i & 3) of Philox4x32-10 with key = seed and
 * counter = (i >> 2 low, i >> 2 high, k, exchange_id).  levels is [host].
 * Device-side error: QGX_ERR_NONFINITE (that bucket's symbols are all zero). */
qgx_status qgx_quantize(qgx_ctx *ctx, const float *v, int K, size_t d, int bucket,
                        const float *levels, int nlev, int norm_type, uint64_t seed,
                        uint32_t exchange_id, int flags, float *norms, uint8_t *sym);

/* CODE o Q of Sec. 3.2 / App. J.  Worker k's stream is stream[k*cap_words ...] [dev]; bucket b
 * starts on a word boundary, after the buckets before it, and holds: the 32 bits of the norm;
 * if sub-blocks are on, one 16-bit length (bits) per sub-block; then per coordinate its
 * codeword, first code bit first, and one sign bit iff the level index is nonzero.
 * bucket_bits [dev] uint32[K][nb] receives each bucket's length in bits, total_bits [dev]
 * uint64[K] their sum.  Words the buckets do not use up to each worker's end are left untouched.
 * Device-side errors: QGX_ERR_CAPACITY (nothing is written for that worker), QGX_ERR_CORRUPT
 * for a level index >= nlev in sym. */
qgx_status qgx_encode(qgx_ctx *ctx, const float *norms, const uint8_t *sym, int K, size_t d,
                      int bucket, const qgx_codebook *cb /*[host]*/, uint32_t *stream,
                      size_t cap_words, uint32_t *bucket_bits, uint64_t *total_bits);

/* qgx_encode for callers that must not allocate device memory.  (The paper has no counterpart: this is
 * a packaging variant of the call above, not another method.)  Who needs it: code that runs where
 * cudaMalloc is off limits -- a communication hook or an inner loop that is being recorded into a CUDA
 * stream capture, a process whose memory is handed out up front by a pool or a scheduler, or a library
 * embedded in another runtime that forbids allocations after start-up.  qgx_encode keeps the buckets'
 * word offsets and per-worker overflow flags in a workspace that it grows with cudaMalloc; this entry
 * point keeps them in a fixed array inside the library image instead (about 516 KB, present on every GPU
 * that loads the library until the process ends) and calls no cudaMalloc, cudaFree or other allocating
 * routine.  Arguments, stream layout, outputs and device-side errors are those of qgx_encode; the results
 * are identical.
 *  - Limits: K <= 1024 and K * nb <= 65536 buckets; beyond that the call returns QGX_ERR_TOO_LARGE and
 *    launches nothing.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 *    device current); make that first call before any stream capture begins.
 *  - All calls on a device share the one array and find in it what the previous call left; the call
 *    overwrites everything it reads.  Two calls that overlap on the GPU (different streams or contexts)
 *    race on it: run them one after the other. */
qgx_status qgx_encode_noalloc(qgx_ctx *ctx, const float *norms, const uint8_t *sym, int K, size_t d,
                              int bucket, const qgx_codebook *cb /*[host]*/, uint32_t *stream,
                              size_t cap_words, uint32_t *bucket_bits, uint64_t *total_bits);

/* DEQ o CODE: the exact inverse of qgx_encode, driven by bucket_bits.  Every read is bounded by
 * the bucket's length; a codeword that runs past it, an unassigned bit pattern, a sub-block whose
 * length disagrees with its header, or lengths that exceed cap_words latch QGX_ERR_CORRUPT. */
qgx_status qgx_decode(qgx_ctx *ctx, const uint32_t *stream, size_t cap_words,
                      const uint32_t *bucket_bits, int K, size_t d, int bucket,
                      const qgx_codebook *cb /*[host]*/, float *norms, uint8_t *sym);

/* Aggregation of Algorithm 1: out[i] = (1/K) sum_k norm_{k,b(i)} * s * l_idx, the fp32 sum taken
 * in the order k = 0..K-1 and divided once by K.  out [dev] float[d]. */
qgx_status qgx_average(qgx_ctx *ctx, const float *norms, const uint8_t *sym, int K, size_t d,
                       int bucket, const float *levels /*[host]*/, int nlev, float *out);

/* ---- fused exchange ------------------------------------------------------------------------ */

/* quantize -> encode -> decode -> average in two kernels, same streams and same mean as the four
 * calls above in sequence.  v [dev] float[K][d]; mean_out [dev] float[d]; total_bits [dev]
 * uint64[K] (may be NULL).  The streams live in the context's workspace (slot 0 or 1, so that
 * the two exchanges of one iteration can both be kept); the workspace grows on first use (cudaMalloc) and is
 * freed by qgx_destroy.  The code must have sub-blocks of 32, 64 or 128 coordinates that divide the bucket
 * (QGX_ERR_INVALID_ARG otherwise: use the four calls).  Device-side errors: QGX_ERR_NONFINITE,
 * QGX_ERR_CAPACITY, QGX_ERR_TIMEOUT (a bounded wait between CTAs ran out), QGX_ERR_CORRUPT. */
qgx_status qgx_exchange(qgx_ctx *ctx, const float *v, int K, size_t d, const qgx_quant_cfg *cfg /*[host]*/,
                        uint32_t exchange_id, int slot, float *mean_out, uint64_t *total_bits);
/* Layer-wise exchange: v [dev] float[K][d] holds nseg tensors back to back (segment s = coordinates
 * [offset, offset + length) of every worker, offsets multiples of 4, the segments tiling [0, d) in order);
 * every segment is exchanged with its own table and code (segs[s].cfg), buckets never cross a segment, and
 * coordinate offset + i of worker k uses the generator counter of coordinate offset + i.  mean_out [dev]
 * float[d]; total_bits [dev] uint64[K] (may be NULL) receives the stream bits summed over segments.  With more
 * than one segment the tensors run side by side on a few streams and workspaces of the context's own, forked
 * from and joined back into the context's stream (the call stays asynchronous and ordered on that stream); their
 * streams are not reachable through qgx_exchange_streams. */
typedef struct {
  size_t offset;
  size_t length;
  const qgx_quant_cfg *cfg;   /* [host] */
} qgx_segment;
qgx_status qgx_exchange_segments(qgx_ctx *ctx, const float *v, int K, size_t d, const qgx_segment *segs /*[host]*/,
                                 int nseg, uint32_t exchange_id, float *mean_out, uint64_t *total_bits);
/* How the decode pass of the fused calls spreads its work.  By default (QGX_SPLIT_AUTO) vectors with few
 * sub-blocks are decoded one worker per thread, followed by a kernel that adds the workers' values in worker
 * order (same results, K times more threads, K * d floats of workspace, at most 256 MB); large vectors are decoded
 * by one thread per sub-block over all workers.  QGX_SPLIT_NEVER / QGX_SPLIT_ALWAYS force one way (ALWAYS still
 * falls back when the workspace would exceed 256 MB).  QGX_SPLIT_SYMBOLS decodes in two passes: the walk alone, one
 * worker per thread, writes every worker's symbol bytes (K * d bytes of workspace unless the exchange keeps its
 * symbols anyway), and a second kernel forms the ordered sums, the squared differences and the state update from
 * them -- same results; exchanges that compare with and overwrite the kept symbols in one go stay in one pass. */
enum { QGX_SPLIT_AUTO = 0, QGX_SPLIT_NEVER = 1, QGX_SPLIT_ALWAYS = 2, QGX_SPLIT_SYMBOLS = 3 };
qgx_status qgx_set_decode_split(qgx_ctx *ctx, int mode);
/* Which kernel the encode pass of the fused calls uses (no counterpart in the paper; the streams are the same bit
 * for bit).  QGX_ENCODE_REGISTERS: one CTA per bucket, the bucket held in registers between the norm and the
 * rounding.  QGX_ENCODE_STAGED: whole buckets of 1024, 2048, 4096, 8192 or 16384 coordinates of 16-byte aligned
 * vectors whose rows lie a multiple of 32 floats apart are staged in shared memory by bulk tensor copies, three
 * buffers deep, and packed 32 coordinates per lane; what does not qualify (other bucket sizes, a short last
 * bucket) still goes through the first kernel.  QGX_ENCODE_AUTO (the default) takes the kernel that measured
 * faster on B200: the first. */
enum { QGX_ENCODE_AUTO = 0, QGX_ENCODE_REGISTERS = 1, QGX_ENCODE_STAGED = 2 };
qgx_status qgx_set_encode_path(qgx_ctx *ctx, int mode);
/* The receiving side alone (Algorithm 1: decode, aggregate): decodes the streams that the last qgx_exchange with
 * the same K, d and bucket left in `slot` -- as they are now, so also after the caller has changed them -- and writes
 * their mean to mean_out [dev] float[d].  cfg [host] must carry the level table and code they were made with.
 * Device-side error: QGX_ERR_CORRUPT for streams that no encoder could have produced (every read stays inside
 * the slot's buffers). */
qgx_status qgx_exchange_decode(qgx_ctx *ctx, int K, size_t d, const qgx_quant_cfg *cfg, int slot, float *mean_out);
/* How many times a device-side wait (one bucket waiting for the word count of an earlier bucket of its worker)
 * polls before it gives up with QGX_ERR_TIMEOUT; the default, 2^22, is seconds.  No counterpart in the paper. */
qgx_status qgx_set_wait_limit(qgx_ctx *ctx, int polls);
/* Diagnostic (no counterpart in the paper): the next fused exchange on this context leaves the first `buckets`
 * buckets of every worker unencoded, so that the buckets after them wait for word counts that never come.  With a
 * small wait limit this shows the bounded wait at work: the waiting buckets give up, QGX_ERR_TIMEOUT is latched,
 * nothing is written for them, the kernel ends, and the context stays usable. */
qgx_status qgx_debug_skip_buckets(qgx_ctx *ctx, size_t buckets);
/* Where the last qgx_exchange on `slot` left its streams: all [dev], valid until the next call
 * that uses the slot.  Any output pointer may be NULL. */
qgx_status qgx_exchange_streams(qgx_ctx *ctx, int slot, const uint32_t **stream, size_t *cap_words,
                                const uint32_t **bucket_bits, const uint64_t **total_bits);

/* ---- choice of the code by measured bits (App. J) -------------------------------------------- */

/* App. J gives two kinds of prefix code: Huffman's when the frequencies of the levels are known or can be
 * estimated, Elias' recursive code when they are not.  Between refits the frequencies drift, so the library can
 * measure instead of assuming: counts[j] = coordinates of an exchange that were sent as level j, and a code costs
 * sum_j counts[j] * (len[j] + [j != 0]) bits on them (the bucket headers cost the same under every code).
 *
 * qgx_set_keep_symbols: qgx_exchange keeps its decoded symbols in the workspace too (one byte per coordinate
 * and worker), as the iteration calls always do for their last exchange but one.
 * qgx_level_counts: counts [dev] uint64[32] of the exchange whose symbols the context keeps (asynchronous);
 * QGX_ERR_INVALID_ARG if it keeps none.
 * qgx_code_bits: the cost of a code on counts [host].
 * qgx_choose_code_host: candidates 0 the code in *cb, 1 a Huffman code built from the counts (only if
 * allow_rebuild), 2 Elias' recursive code, 3 the fixed-length code; bits [host] uint64[4] receives their costs
 * (all ones for a candidate that is not allowed), *cb the cheapest (the earlier one on ties), *winner its number.
 * qgx_choose_code: qgx_level_counts into counts [dev] uint64[32], then qgx_choose_code_host on cfg->cb, for
 * the exchanges that follow; synchronizes the stream.  cfg->code_type (what a refit builds) is left as it is. */
qgx_status qgx_set_keep_symbols(qgx_ctx *ctx, int on);
qgx_status qgx_level_counts(qgx_ctx *ctx, uint64_t *counts);
qgx_status qgx_code_bits(const uint64_t *counts, const qgx_codebook *cb, uint64_t *bits);
qgx_status qgx_choose_code_host(const uint64_t *counts, qgx_codebook *cb, int allow_rebuild, uint64_t *bits, int *winner);
qgx_status qgx_choose_code(qgx_ctx *ctx, qgx_quant_cfg *cfg /*[host] in/out*/, int allow_rebuild, uint64_t *counts,
                           uint64_t *bits, int *winner);

/* ---- level adaptation (Sec. 3.3; Algorithm 1, "t in U") ------------------------------------- */

/* Sufficient statistics and refit in one call: hist [dev] double[nbins] receives the histogram of
 * the normalized magnitudes u of all K*nb buckets of v, each coordinate weighted by its bucket's
 * squared norm (the weights lambda_j of Eq. QAda); then, on the host, cfg->levels is refitted
 * (qgx_fit_levels, first fit iff refit == QGX_REFIT_FIRST) and cfg->cb rebuilt per cfg->code_type
 * from the symbol weights.  Synchronizes the stream.  cfg [host] in/out; hist_host [host]
 * double[nbins] out, may be NULL. */
qgx_status qgx_update_levels(qgx_ctx *ctx, const float *v, int K, size_t d, qgx_quant_cfg *cfg,
                             int refit, double *hist, double *hist_host);
/* The histogram alone (asynchronous).  weighted == 0 counts coordinates instead. */
qgx_status qgx_histogram(qgx_ctx *ctx, const float *v, int K, size_t d, int bucket, int norm_type,
                         int nbins, int weighted, double *hist);

/* ---- the iteration (Algorithm 1, Eq. Q-GenX, step size of Theorem 3) ------------------------ */

/* Sets Y = 0, X = anchor, Xbar = 0, scalars = {0, K}, t = 1 (gamma_1 = K). */
qgx_status qgx_eg_init(qgx_ctx *ctx, qgx_eg_state *st /*[host]*/);
/* One iteration in the dual-extrapolation instance (two oracle calls, two exchanges):
 *   V_{k,t} = A(X_t) + U_{k,t};  [refit of levels and code on V_{.,t} if refit != 0];
 *   X_{t+1/2} = X_t - gamma_t mean_k Vhat_{k,t};   V_{k,t+1/2} = A(X_{t+1/2}) + U_{k,t+1/2};
 *   Y_{t+1} = Y_t - mean_k Vhat_{k,t+1/2};  sum += sum_k ||Vhat_{k,t} - Vhat_{k,t+1/2}||^2;
 *   gamma_{t+1} = K / sqrt(1 + sum);  X_{t+1} = anchor + gamma_{t+1} Y_{t+1};
 *   Xbar += (X_{t+1/2} - Xbar) / t;  t += 1.
 * noise_t, noise_half [dev] float[K][d] or NULL; exchange ids are 2t and 2t+1.  cfg [host] is
 * in/out when refit != 0 (and the call then synchronizes once).  bits [dev] uint64[2][K]
 * (stream bits of the two exchanges), may be NULL. */
qgx_status qgx_eg_step(qgx_ctx *ctx, qgx_eg_state *st, const qgx_operator *op,
                       const float *noise_t, const float *noise_half, qgx_quant_cfg *cfg,
                       int refit, uint64_t *bits);
/* qgx_eg_step with a level table and a code of its own for each exchange (the finer scheme that the footnote
 * of Sec. 3.3 describes: one sequence of adaptive levels for the V_{k,t}, another for the V_{k,t+1/2}).  The first
 * exchange uses cfg_t, the second cfg_half; when refit != 0 each is refitted on its own dual vectors (one more
 * histogram pass).  Both must have the same bucket and sub-block sizes; the seeds may differ.  The squared
 * differences compare vectors dequantized with their own tables. */
qgx_status qgx_eg_step_two_tables(qgx_ctx *ctx, qgx_eg_state *st, const qgx_operator *op,
                                  const float *noise_t, const float *noise_half, qgx_quant_cfg *cfg_t,
                                  qgx_quant_cfg *cfg_half, int refit, uint64_t *bits);
/* The other two members of the family that Sec. 3.1 lists (Eq. Quantized DA, Eq. Quantized OptDA): one
 * oracle call and one exchange per iteration, same state, same step-size rule.
 *   QGX_METHOD_DA:    Vhat_{k,t} = 0, so X_{t+1/2} = X_t;  g_k = Q(A(X_t) + U_k);  Y_{t+1} = Y_t - mean_k g_k;
 *                     sum += sum_k ||g_k||^2.
 *   QGX_METHOD_OPTDA: Vhat_{k,t} = g_{k,t-1/2}, the vectors of the previous iteration (zero in the first):
 *                     X_{t+1/2} = X_t - gamma_t mean_k g_{k,t-1/2};  g_{k,t+1/2} = Q(A(X_{t+1/2}) + U_k);
 *                     Y_{t+1} = Y_t - mean_k g_{k,t+1/2};  sum += sum_k ||g_{k,t-1/2} - g_{k,t+1/2}||^2.
 * Then gamma_{t+1}, X_{t+1}, Xbar and t as in qgx_eg_step.  The exchange id is 2t + 1; a refit uses the
 * iteration's only dual vectors.  noise [dev] float[K][d] or NULL.  mean_prev [dev] float[d] (OPTDA; may be
 * NULL for DA) holds the mean of g_{k,t-1/2} between calls: read at t > 1, overwritten.  The previous vectors
 * themselves stay in the context (symbols, norms and their level table), so between two OPTDA steps of one
 * state no other exchange may run on this context (QGX_ERR_INVALID_ARG if the kept vectors do not fit).
 * bits [dev] uint64[K], may be NULL. */
enum { QGX_METHOD_DE = 0, QGX_METHOD_DA = 1, QGX_METHOD_OPTDA = 2 };
qgx_status qgx_family_step(qgx_ctx *ctx, qgx_eg_state *st, int method, const qgx_operator *op,
                           const float *noise, qgx_quant_cfg *cfg, int refit, float *mean_prev,
                           uint64_t *bits);
/* A(x) alone: out [dev] float[d]. */
qgx_status qgx_apply_operator(qgx_ctx *ctx, const qgx_operator *op, const float *x, float *out);

#ifdef __cplusplus
}
#endif
#endif /* QGX_H_ */
