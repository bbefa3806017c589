/*
 * tq.h -- C ABI of libtq: truncated quantization of heavy-tailed gradients on one GPU.
 *
 * The library implements the per-round hot path of Algorithm 1 (TQSGD) of "Improved
 * Quantization Strategies for Managing Heavy-tailed Gradients in Distributed Learning":
 *
 *   client i :  statistics of g_i  ->  (alpha, codebook)            tq_stats, tq_params
 *               Q_lambda[T_alpha(g_i)], b bits per element, packed   tq_compress
 *   server   :  mean over the N clients of the dequantized codes     tq_decompress_aggregate
 *
 * The N clients ("workers") are N gradient slices resident on one GPU.
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are ordinary
 *     host memory.  The library allocates no device memory and frees nothing.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  The four compute
 *     calls only enqueue work on it; none of them synchronises.
 *   - num_levels L = 2^bits is the number of quantization points; the paper's s = 2^b - 1 is the
 *     number of intervals, s = L - 1 (Section 3.1).  bits is 1, 2, 3 or 4.
 *   - Every call returns a tq_status; nothing throws or aborts, kernels never trap.
 *   - NaN gradients are counted by tq_stats and quantized as -alpha (code 0); +-Inf as +-alpha.
 *
 * Arithmetic that decides a code is fp32 with one rounding per operation (no contraction), and the
 * random bits are a pure function of (seed, worker, element index), so a packed buffer is a
 * deterministic function of its inputs.
 */
#ifndef TQ_H_
#define TQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TQ_MAX_LEVELS 16
#define TQ_MAX_WORKERS 64
#define TQ_STATIC_MAX_WORKERS 16   /* most workers one tq_stats_static call can reduce */
#define TQ_MAX_SEGMENTS 64         /* most layer groups per row in the tq_*_segments calls */

typedef enum {
    TQ_OK = 0,
    TQ_ERR_INVALID_ARG = -1,       /* null pointer, bad enum, N out of range, bits mismatch */
    TQ_ERR_DOMAIN = -2,            /* gamma <= 2, rho outside (0, 0.5), g_min <= 0, alpha <= 0 */
    TQ_ERR_ALIGNMENT = -3,         /* a device pointer or stride misses its stated alignment */
    TQ_ERR_BUFFER_TOO_SMALL = -4,  /* packed stride or workspace smaller than required */
    TQ_ERR_DEGENERATE_LEVELS = -5, /* codebook not strictly increasing in fp32 */
    TQ_ERR_CUDA = -6,              /* a CUDA runtime call failed; see tq_last_cuda_error */
    TQ_ERR_STATIC_LIMIT = -7       /* request exceeds the library's built-in scratch (tq_stats_static) */
} tq_status;

typedef enum { TQ_F32 = 0, TQ_BF16 = 1 } tq_dtype;               /* gradient storage type */
typedef enum {
    TQ_UNIFORM = 0,     /* evenly spaced levels (Section 4.1) */
    TQ_NONUNIFORM = 1,  /* density proportional to p^(1/3) (Section 4.2); also any caller-made codebook */
    TQ_BISCALED = 2     /* two step sizes, inside and outside k* alpha (Appendix, truncated BiScaled) */
} tq_mode;
typedef enum {
    TQ_ALPHA_CLOSED = 0,       /* alpha' : the boxed equation with Q = 1 (text after Theorem 1) */
    TQ_ALPHA_FIXED_POINT = 1,  /* iterate the boxed equation of Section 4.1 / 4.2 */
    TQ_ALPHA_USER = 2,         /* caller supplies alpha */
    TQ_ALPHA_MAXABS = 3        /* alpha = max|g|: no truncation (the QSGD / NQSGD baselines of Section 5) */
} tq_alpha_rule;

enum { TQ_FLAG_ALPHA_CAPPED = 1, TQ_FLAG_ALPHA_AT_GMIN = 2, TQ_FLAG_GAMMA_FROM_MLE = 4,
       TQ_FLAG_INVALID = 8 /* set by tq_params_device when a worker's statistics are outside the domain */ };

/* Statistics of one worker's gradient; 64 bytes, written on the device by tq_stats. */
typedef struct {
    uint64_t d;             /* elements seen */
    uint64_t n_tail;        /* #{ j : |g_j| > g_min }, both signs pooled */
    uint64_t n_nonfinite;   /* NaN / Inf elements, excluded from every sum */
    double sum_abs;         /* sum |g_j| */
    double sum_sq;          /* sum g_j^2 */
    double sum_log_tail;    /* sum over the tail of ln(|g_j| / g_min) */
    float max_abs;          /* max |g_j| over finite elements */
    float g_min;            /* threshold used: the caller's, or kappa * mean|g| */
    uint64_t reserved;
} tq_stats_t;

/* Quantizer of one worker; plain data, produced on the host, passed to the kernels by value. */
typedef struct {
    uint32_t bits;          /* b */
    uint32_t num_levels;    /* L = 2^b */
    uint32_t mode;          /* tq_mode */
    uint32_t flags;         /* TQ_FLAG_* */
    float alpha;            /* truncation threshold, = levels[L-1] */
    float inv_step;         /* uniform mode: (L-1) / (2 alpha), rounded up */
    float gamma;            /* tail exponent used */
    float g_min;
    float rho;              /* one-sided tail mass n_tail / (2 d) */
    int32_t iterations;     /* fixed-point iterations spent on alpha */
    float reserved[2];
    float levels[TQ_MAX_LEVELS];     /* l_0 = -alpha < ... < l_{L-1} = alpha */
    float inv_width[TQ_MAX_LEVELS];  /* 1 / (l_{k+1} - l_k), rounded up, k < L-1 */
} tq_params_t;

/* Words (uint32) of one worker's packed buffer: ceil(d * bits / 32) rounded up to a multiple of 4.
 * Wire format (the paper only says "b bits per element", Section 2): code j occupies bits
 * [j*bits, (j+1)*bits) of an LSB-first stream over little-endian 32-bit words; unused bits are 0. */
size_t tq_packed_words(uint64_t d, uint32_t bits);

/* Bytes of device scratch tq_stats needs for n_workers slices (block partials + tickets). */
size_t tq_stats_workspace_bytes(uint32_t n_workers);

/*
 * Statistics reduction (Section 5: gamma = 1 + n [sum ln(g_j / g_min)]^-1 over g_j > g_min;
 * Section 4.1: rho = tail mass beyond g_min).  One 64-byte record per worker.
 *   grad_dev     [n_workers][grad_stride] elements of `dtype`, 32-byte aligned; worker i's slice is
 *                the first d elements of row i.  grad_stride (elements) must keep rows 32-byte aligned.
 *   g_min        > 0: threshold for the tail (any positive fp32 value, subnormal ones included).
 *                <= 0: each worker uses kappa * mean|g| of its own slice (one extra pass over the data).
 *   stats_dev    [n_workers] tq_stats_t, device memory, 8-byte aligned; valid when the stream reaches
 *                the end of this call's work (copy it back to the host for tq_params).
 *   workspace_dev, ws_bytes   device scratch of at least tq_stats_workspace_bytes(n_workers), 256-byte
 *                aligned; contents need not be initialised and are not meaningful afterwards.  Calls
 *                sharing one workspace must not overlap on the device.
 * Sums are accumulated in fp32 over runs of 16 elements and in fp64 beyond; counts and max are exact.
 * d = 0 is allowed (all-zero records).  Errors: INVALID_ARG, ALIGNMENT, BUFFER_TOO_SMALL, CUDA.
 */
tq_status tq_stats(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride,
                   uint32_t n_workers, float g_min, float kappa, tq_stats_t* stats_dev,
                   void* workspace_dev, size_t ws_bytes, void* stream);

/* What tq_stats_hinted remembers between rounds, one per worker, device memory owned by the caller.
 * Zero-fill it before the first round. */
typedef struct {
    float level;     /* kappa * mean|g| of the last call (0: no hint yet) */
    uint32_t hit;    /* 1: the last call's single pass already held the tail sums; 0: its tail pass had to run */
} tq_gmin_hint_t;

/*
 * Statistics in ONE pass over the gradient, for the automatic threshold.
 * Section 4.1 introduces g_min only as the point from which the power-law behaviour holds and gives no
 * rule for choosing it; this call
 * uses g_min = kappa * mean|g| rounded DOWN to a power of two (0, i.e. no tail, below 2^-126).  A
 * power-of-two threshold can be tried before the mean is known: the pass gathers the tail count and
 * sum ln|g| for the two powers of two nearest to hint->level (the previous round's kappa * mean|g|),
 * and when the finished mean selects one of them the record is complete after reading the data once.
 * When it selects neither (first round; mean moved by more than a factor of about 1.4 to 2) a second
 * kernel, which is always enqueued and otherwise returns at once, redoes the tail sums for the right
 * threshold: the record is the same, bit for bit, either way, and the host never has to look.
 *   hint_dev     [n_workers] tq_gmin_hint_t, device memory, 8-byte aligned, in/out (updated by every call).
 *   kappa        > 0.
 *   other arguments, the record's fields, workspace rules and errors as for tq_stats; stats_dev[i].g_min
 *   is the power of two used.  tq_stats with that g_min passed explicitly gives the same counts (sums
 *   to rounding).
 */
tq_status tq_stats_hinted(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride, uint32_t n_workers,
                          float kappa, tq_gmin_hint_t* hint_dev, tq_stats_t* stats_dev, void* workspace_dev,
                          size_t ws_bytes, void* stream);

/*
 * tq_stats without a scratch argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of tq_stats, same kernels, same results.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework's stream-ordered
 * or pooled allocator callback, in a plugin that is handed device buffers but owns none, or in a
 * latency-critical loop where an allocation would synchronise the device.  Such a caller still passes
 * its gradient and the output records; only the reduction's scratch (block partials + tickets) comes
 * from the library: a fixed 1 MiB + 384 B array that lives in the library's device image, so every GPU
 * that loads libtq holds it until the process exits.
 *
 *   n_workers    at most TQ_STATIC_MAX_WORKERS (16); more returns TQ_ERR_STATIC_LIMIT and does nothing.
 *   all other arguments, results and errors as for tq_stats.
 *
 * The call allocates nothing and frees nothing.  The first call on each device looks up the array's
 * device address (once per device, with that device current); make that first call outside any
 * stream capture.  All calls on a device share the one array and it keeps the previous call's
 * contents: the library clears the ticket counters itself at the start of every call, nothing else
 * needs to start at zero.  Two calls whose kernels overlap on the same GPU (different streams, or
 * different host threads) race on the array and give wrong statistics: serialise them.
 * The looked-up address is remembered per device ordinal for the life of the process.  It does not
 * survive cudaDeviceReset, nor a second CUDA context on the same ordinal: a process that resets a device
 * or switches contexts must not call tq_stats_static on that device afterwards (use tq_stats with its
 * own workspace there).
 */
tq_status tq_stats_static(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride,
                          uint32_t n_workers, float g_min, float kappa, tq_stats_t* stats_dev, void* stream);

/*
 * Parameter design on the host (Section 4), O(L) work in double precision.
 *   stats_host   one record copied back from tq_stats.
 *   gamma        tail exponent of the power-law model; NaN = use the maximum-likelihood estimate.
 *                Must exceed 2.
 *   alpha_rule   CLOSED: alpha' = g_min [2 rho s^2 / (gamma-2)]^(1/(gamma-1)).
 *                FIXED_POINT: the boxed equations alpha = g_min [2 rho s^2 / ((gamma-2) Q(alpha))]^(1/(gamma-1))
 *                with Q = Q_U (uniform, Section 4.1) or Q_N (non-uniform, Section 4.2), evaluated on
 *                the model density (flat below g_min, power law above), iterated from alpha' until the
 *                relative change is <= 1e-12 or 10000 iterations.  Both are clamped to
 *                [g_min, max_abs] (flags ALPHA_AT_GMIN / ALPHA_CAPPED).
 *                USER: alpha_user, unclamped.
 *                MAXABS: alpha = max_abs, so nothing is truncated: with UNIFORM this is the paper's QSGD
 *                baseline, with NONUNIFORM its NQSGD baseline (Section 5).
 *   mode         UNIFORM: l_k = -alpha + k 2 alpha / s.  NONUNIFORM: the boxed density
 *                lambda_s proportional to p^(1/3) (Section 4.2), turned into levels by
 *                integral_{-alpha}^{l_k} lambda_s = k.  BISCALED: the Appendix's two-piece density
 *                (k* = argmin_k Q_B(alpha, k) by a 65-point scan + golden section, alpha from the
 *                boxed BiScaled equation with k* recomputed at every step), levels by the same rule.
 *                To the kernels BISCALED is a table codebook like NONUNIFORM.
 * Errors: INVALID_ARG, DOMAIN, DEGENERATE_LEVELS.  out_host is unspecified on error.
 */
tq_status tq_params(const tq_stats_t* stats_host, uint32_t num_levels, tq_mode mode, double gamma,
                    tq_alpha_rule alpha_rule, double alpha_user, tq_params_t* out_host);

/* tq_params for n workers in one call: stats_host[n] -> out_host[n], same arguments for all.
 * Stops at the first failing worker and returns its status. */
tq_status tq_params_batch(const tq_stats_t* stats_host, uint32_t n_workers, uint32_t num_levels, tq_mode mode,
                          double gamma, tq_alpha_rule alpha_rule, double alpha_user, tq_params_t* out_host);

/* Quantizer for a caller-supplied codebook (any strictly increasing levels with
 * levels[0] = -levels[L-1]; Section 3.1's general codebook).  Fills inv_width / inv_step. */
tq_status tq_params_from_levels(const float* levels_host, uint32_t num_levels, tq_mode mode,
                                tq_params_t* out_host);

/*
 * Client side: truncate (Section 3.1, truncation equation), stochastically round onto the codebook
 * (quantizer equation) and pack, for n_workers slices in one launch.
 *   grad_dev     as for tq_stats.
 *   params_host  [n_workers]; all must have the same bits.  Copied during the call.
 *   seed, first_worker   element j of slice i draws its 16 random bits from Philox4x32-10 with
 *                key = seed and counter = (j >> 3, first_worker + i, 0), slot j & 7.
 *   packed_dev   [n_workers][words_stride] uint32, 16-byte aligned, words_stride a multiple of 4 and
 *                >= tq_packed_words(d, bits).  The first tq_packed_words(d, bits) words of each row
 *                are written (padding as zeros); words beyond are untouched.
 * Decision per element: t = clip(g); interval k and p = (t - l_k) / (l_{k+1} - l_k) in fp32;
 * T = rint(p * 2^16); code = k + [r < T].  The round-up probability is therefore p rounded to a multiple of
 * 2^-16: E[Q(g)] differs from the truncated value by at most about 2^-17 of the interval width, a deviation
 * that is fixed for a given value (it is some 1e-5 of the quantization noise of the workers' mean, and matters
 * only against elements smaller than 2^-17 of the interval, i.e. without truncation on very heavy tails).
 * Errors: INVALID_ARG, ALIGNMENT, BUFFER_TOO_SMALL, CUDA.
 */
tq_status tq_compress(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride,
                      uint32_t n_workers, const tq_params_t* params_host, uint64_t seed,
                      uint32_t first_worker, uint32_t* packed_dev, size_t words_stride, void* stream);

/*
 * Server side (Algorithm 1, aggregation step): out_j = sum_i w_i * levels_i[code_ij].
 *   weights_host NULL: w_i = 1/N (Lemma 2): fp32 adds in worker order, then one division by N.
 *                else [n_workers] fp32: each product is rounded, then added in worker order.
 *   out_dev      [d] fp32, 32-byte aligned (the kernel stores 32 bytes per thread at a time).
 * Errors: INVALID_ARG, ALIGNMENT, BUFFER_TOO_SMALL, CUDA.  TQ_OK means the launch was accepted; it does
 * not cover a bounded wait running out inside the kernel, see tq_wait_expired_count.
 */
tq_status tq_decompress_aggregate(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers,
                                  uint64_t d, const tq_params_t* params_host, const float* weights_host,
                                  float* out_dev, void* stream);

/*
 * The same aggregation with the N packed rows given one by one (Algorithm 1, aggregation step, where
 * worker i's message lives wherever worker i left it): rows_host[i] is the device address of worker
 * i's packed row.  The rows need not be neighbours or share an allocation, and may be in another GPU's
 * memory that the current device can read (peer access enabled, or a mapped symmetric buffer): the
 * kernel then pulls each row's bytes straight over NVLink while it aggregates, with no gather copy
 * first.  Every row: 16-byte aligned, at least tq_packed_words(d, bits) words readable.
 *   rows_host    [n_workers] host array of device pointers; read during the call, not kept.
 *   other arguments, arithmetic, result and errors as for tq_decompress_aggregate.
 */
tq_status tq_decompress_aggregate_rows(const uint32_t* const* rows_host, uint32_t n_workers, uint64_t d,
                                       const tq_params_t* params_host, const float* weights_host, float* out_dev,
                                       void* stream);

/*
 * Server side including the model update (Algorithm 1, last step: theta <- theta - eta * g_bar) with the
 * optimiser of the paper's experiments (Section 5: momentum SGD with weight decay), fused into the
 * aggregation so that g_bar never goes to memory:
 *     g = g_bar_j (as tq_decompress_aggregate);  g += weight_decay * theta_j  (skipped when 0);
 *     m_j = momentum * m_j + g  (when momentum_dev is given; g = m_j);  theta_j -= lr * g.
 * fp32, every operation rounded once.  theta_dev [d] and momentum_dev [d] (may be NULL) are fp32 device
 * arrays, 32-byte aligned, updated in place.  Other arguments and errors as tq_decompress_aggregate.
 * A tile whose bounded wait ran out (see tq_wait_expired_count) is left as it was, so after such a launch
 * theta and the momentum buffer are updated in some tiles and not in others: a caller that cannot
 * tolerate that checks tq_wait_expired_count before and after the step and restores theta from its own
 * copy when the count moved.
 */
tq_status tq_decompress_aggregate_apply(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers, uint64_t d,
                                        const tq_params_t* params_host, const float* weights_host, float* theta_dev,
                                        float* momentum_dev, float lr, float momentum, float weight_decay, void* stream);

/*
 * The same round without a host round trip (the paper takes alpha and lambda_s as given inputs of
 * Algorithm 1; where they come from -- Section 4 -- can equally run on the device).
 *
 * tq_params_device: Section 4 for n_workers records, one device thread per worker, same formulas and
 *   arguments as tq_params, reading stats_dev and writing params_dev (both device memory, 8-byte
 *   aligned).  Nothing is returned to the host: a worker whose statistics are outside the model's
 *   domain gets flags = TQ_FLAG_INVALID, iterations = the tq_status it would have returned, alpha = 0
 *   and an all-zero codebook; tq_compress_device_params then writes an all-zero row for it and the
 *   aggregate receives zeros from it.  Device and host math libraries may differ in the last fp32 bit
 *   of alpha or a level.
 * tq_compress_device_params / tq_decompress_aggregate_device_params: as tq_compress /
 *   tq_decompress_aggregate with params_dev[n_workers] in device memory; bits and mode are not read
 *   from the records but given by the caller (num_levels, mode).
 * All three only enqueue work on `stream`, so a round made of tq_stats_hinted (or tq_stats) and these three can be
 * captured into a CUDA graph and replayed; call each once outside the capture first (the first launch of some kernels
 * sets a function attribute).  Errors: INVALID_ARG, DOMAIN (alpha_user <= 0), ALIGNMENT, BUFFER_TOO_SMALL, CUDA.
 */
tq_status tq_params_device(const tq_stats_t* stats_dev, uint32_t n_workers, uint32_t num_levels, tq_mode mode,
                           double gamma, tq_alpha_rule alpha_rule, double alpha_user, tq_params_t* params_dev,
                           void* stream);
tq_status tq_compress_device_params(const void* grad_dev, tq_dtype dtype, uint64_t d, uint64_t grad_stride,
                                    uint32_t n_workers, const tq_params_t* params_dev, uint32_t num_levels, tq_mode mode,
                                    uint64_t seed, uint32_t first_worker, uint32_t* packed_dev, size_t words_stride,
                                    void* stream);
tq_status tq_decompress_aggregate_device_params(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers,
                                                uint64_t d, const tq_params_t* params_dev, uint32_t num_levels,
                                                const float* weights_host, float* out_dev, void* stream);

/*
 * Layer groups in one launch per step.  Section 5 (experimental setting) quantizes groups of layers --
 * the convolutional and the fully-connected ones -- independently: each group has its own statistics,
 * its own alpha and codebook, and its own packed stream.  A group is a segment [offset, offset + length)
 * of every worker's row, the same for all workers.  These calls do for all (worker, segment) pairs at once
 * what one tq_stats / tq_params_device / tq_compress_device_params / tq_decompress_aggregate_device_params
 * call per group does on the sub-range, with the same results bit for bit:
 *   - records are indexed [worker * n_segments + segment];
 *   - element j of a segment is element j of that group's gradient: the random bits of Section 3.1's
 *     rounding come from (seed, first_worker + worker, j) with j counted from the segment's start;
 *   - segment s of a worker's packed row starts at word sum_{t < s} tq_packed_words(length_t, bits) of the row
 *     (every segment is padded to a multiple of 4 words; tq_segments_packed_words gives the row total).
 *   segments_host  [n_segments] host array, 1 <= n_segments <= TQ_MAX_SEGMENTS, read during the call; every
 *                  length >= 1; offset * element size a multiple of 32 bytes (gradient: 8 fp32 or 16 bf16
 *                  elements; output: 8 elements); segments must not overlap and, for the gradient, must end
 *                  inside grad_stride.
 *   n_workers * n_segments may reach TQ_MAX_WORKERS * TQ_MAX_SEGMENTS; tq_params_device accepts that many
 *                  records.  tq_stats_segments needs tq_stats_workspace_bytes(n_workers * n_segments) of scratch.
 * The parameter records are read from device memory (tq_params_device writes them there), so a round with
 * layer groups needs no host round trip.  A pair whose statistics are outside the model's domain (for
 * instance a one-element group) is marked TQ_FLAG_INVALID by tq_params_device; its packed segment is all
 * zeros and it contributes zeros to the aggregate.
 * Errors: INVALID_ARG (also overlapping or empty segments), ALIGNMENT, BUFFER_TOO_SMALL, CUDA.
 */
typedef struct {
    uint64_t offset;   /* first element of the group in every worker's row */
    uint64_t length;   /* elements */
} tq_segment_t;
size_t tq_segments_packed_words(const tq_segment_t* segments_host, uint32_t n_segments, uint32_t bits);
tq_status tq_stats_segments(const void* grad_dev, tq_dtype dtype, uint64_t grad_stride, uint32_t n_workers,
                            const tq_segment_t* segments_host, uint32_t n_segments, float g_min, float kappa,
                            tq_stats_t* stats_dev, void* workspace_dev, size_t ws_bytes, void* stream);
/* The one-pass statistics of tq_stats_hinted for every (worker, segment) pair: hint_dev holds n_workers * n_segments
 * entries, indexed like the records; everything else as tq_stats_segments and tq_stats_hinted. */
tq_status tq_stats_hinted_segments(const void* grad_dev, tq_dtype dtype, uint64_t grad_stride, uint32_t n_workers,
                                   const tq_segment_t* segments_host, uint32_t n_segments, float kappa,
                                   tq_gmin_hint_t* hint_dev, tq_stats_t* stats_dev, void* workspace_dev, size_t ws_bytes,
                                   void* stream);
tq_status tq_compress_segments(const void* grad_dev, tq_dtype dtype, uint64_t grad_stride, uint32_t n_workers,
                               const tq_segment_t* segments_host, uint32_t n_segments, const tq_params_t* params_dev,
                               uint32_t num_levels, tq_mode mode, uint64_t seed, uint32_t first_worker,
                               uint32_t* packed_dev, size_t words_stride, void* stream);
tq_status tq_decompress_aggregate_segments(const uint32_t* packed_dev, size_t words_stride, uint32_t n_workers,
                                           const tq_segment_t* segments_host, uint32_t n_segments,
                                           const tq_params_t* params_dev, uint32_t num_levels,
                                           const float* weights_host, float* out_dev, void* stream);

const char* tq_strerror(tq_status status);
int tq_last_cuda_error(void);   /* cudaError_t of the last failed runtime call on this thread, else 0 */
uint64_t tq_kernel_launches(void); /* kernels launched by this library in this process so far */

/* Bounded waits.  The large-input decompression kernel stages packed bytes through asynchronous bulk
 * copies and waits for them on shared-memory barriers; every such wait gives up after a fixed number
 * of polls.  While barriers remain in the tile's loop the whole block takes the decision (it stores nothing for
 * the tile and counts itself once); in the last three steps of a tile there is no barrier left, and a thread whose
 * wait runs out there drops its own 32 outputs and counts itself, so a tile can then be partly stored.
 * *count_host receives the number of such give-ups on the current device since the library was loaded
 * (0 in a healthy run: a non-zero value means the outputs of the affected launch are incomplete).
 * Synchronises the device.  Returns TQ_ERR_INVALID_ARG for a null pointer, TQ_ERR_CUDA if the read fails.
 * (The paper has no counterpart; this is a health check of the implementation.) */
tq_status tq_wait_expired_count(uint32_t* count_host);

#ifdef __cplusplus
}
#endif
#endif /* TQ_H_ */
