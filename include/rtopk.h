/*
 * rtopk.h -- C ABI of the rTop-k sparsification / aggregation library for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel hot path of
 *   Barnes, Inan, Isik, Ozgur, "rTop-k: A Statistical Estimation Approach to Distributed SGD":
 * for W workers whose gradient vectors are held as the rows of one matrix on one GPU,
 *
 *   node body   (Algorithm 1):  a = g + m ;  ghat = rTop_k(a) ;  m' = a - ghat ;  send ghat
 *   rTop_k      (Definition 3): keep a uniformly random k-subset U of the r largest-magnitude
 *                               coordinates (Definition 1, top-r), zero the rest
 *   master      (Algorithm 1):  ghat = (1/n) sum_i ghat_i          (n = W here)
 *
 * Conventions fixed where the paper is silent:
 *   - magnitudes are ordered by the binary32 bit pattern with the sign cleared; ties go to the
 *     lower index ("pi is a permutation" in Definition 1 leaves this open);
 *   - U is drawn with Floyd's subset algorithm over positions 0..r-1 of the top-r set listed by
 *     ascending index; iteration j (j = r-k .. r-1) draws t_j = floor(u64 * (j+1) / 2^64) with
 *     u64 = (x1 << 32) | x0 and (x0..x3) = Philox4x32-10(counter = (j, worker, segment, step),
 *     key = (seed low word, seed high word)); t_j joins U's positions unless already there, in
 *     which case j does;
 *   - a, m, message values and the dense update are binary32; g may be binary32 or bfloat16
 *     (widened exactly); the add is one round-to-nearest add, and a NaN sum is stored as the
 *     default quiet NaN 0x7FC00000 (IEEE 754 leaves NaN payloads to the implementation);
 *   - a message is k (index, value) pairs in ascending index order; m' is a bit copy of a
 *     outside U and +0.0f on U.
 *
 * Pointers are DEVICE pointers owned by the caller unless a parameter is documented as host
 * memory.  Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 * and return without synchronising unless stated.  Every function returns an rtopk_status; on a
 * non-zero status detected on the host nothing has been enqueued and no buffer was written.
 * Conditions only the device can detect (an internal bounded wait that gave up) are reported by
 * rtopk_poll_status.  A context serialises its scratch memory: calls that share a context must be
 * ordered on one stream (or otherwise not overlap on the GPU).
 *
 * A call that only enqueues work may be captured into a CUDA graph (it forks onto a stream of the
 * context and joins again, which capture follows).  The context keeps the table of the call's
 * slices on the device and re-sends it only when the shape of the call changes (d, W, segments,
 * r, k, leading dimensions, worker-independent); a captured graph holds either no such copy or one
 * from a buffer of the context.  So between the capture and the last replay of the graph make no
 * call of another shape on that context, or capture again after it.
 */
#ifndef RTOPK_H_
#define RTOPK_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rtopk_ctx rtopk_ctx;

typedef enum {
  RTOPK_OK = 0,
  RTOPK_ERR_INVALID_ARG = 1, /* null/misaligned pointer, size out of range, k > r, r > d, ... */
  RTOPK_ERR_ALLOC = 2,       /* device or host allocation failed */
  RTOPK_ERR_CUDA = 3,        /* a CUDA runtime call failed; see rtopk_last_cuda_error */
  RTOPK_ERR_UNSUPPORTED = 4, /* valid request the build does not cover */
  RTOPK_ERR_INTERNAL = 5     /* device-side bounded wait expired or an internal invariant broke */
} rtopk_status;

/* gradient element type; residual, message values and the update are always binary32 */
enum { RTOPK_F32 = 0, RTOPK_BF16 = 1 };

/* Scaling of the aggregated update (S_i = sum over the workers that sent coordinate i, in double):
 *   MEAN      S_i / W                 Algorithm 1's master step;
 *   SUM       S_i;
 *   UNBIASED  S_i * r / (W * k)       the estimator in the proof of Theorem 1, (1/n) sum_w X_w / S with
 *                                     subsampling fraction S = k / r (needs r: rtopk_step, rtopk_step_apply,
 *                                     rtopk_aggregate_unbiased; the segmented step returns UNSUPPORTED);
 *   COUNT     S_i / c_i               c_i = number of workers that sent i (the average over the updates a
 *                                     coordinate received, a second reading of the master step; W <= 65535).
 * All four are rounded to binary32 once. */
enum { RTOPK_SCALE_MEAN = 0, RTOPK_SCALE_SUM = 1, RTOPK_SCALE_UNBIASED = 2, RTOPK_SCALE_COUNT = 3 };

/* rtopk_set_option keys */
enum {
  RTOPK_OPT_SELECT_PATH = 0, /* where the first bracket of the r-th largest magnitude comes from (the result
                                is the same): 0 = from a sample of the slice, or from the slice's last
                                thresholds with RTOPK_OPT_REUSE_THRESHOLD (a bracket that misses is repaired
                                exactly); 1 = from an exact histogram of the 11 leading bits of every
                                magnitude, one more pass that reads g and m: no sample, no statistics */
  RTOPK_OPT_PROFILE = 1,     /* 1 = record CUDA events between the phases of each call on the
                                caller's stream (read with rtopk_get_phase_times); 0 = off */
  RTOPK_OPT_REUSE_THRESHOLD = 2, /* 1 = consecutive calls of one shape on one residual buffer predict the
                                first threshold from the exact thresholds of the last two calls instead
                                of sampling, once those two are within 25 % of each other (a = g + m
                                drifts slowly from round to round); a prediction that misses is
                                repaired by the exact path and the next two calls sample again.
                                Results never depend on it.  0 = off (default) */
  RTOPK_OPT_THRESHOLD_SIGNS = 3, /* what rtopk_sparsify_threshold sends for a kept coordinate: 0 (default) its
                                value a_i; 1 = sign(a_i) * M with M = 2 theta, the quantised observation of
                                Section II (after the pre-processing step a coordinate is 0 or +-M, so one bit
                                per kept coordinate describes it); the node then keeps a_i - sign(a_i) * M in
                                that residual slot (one binary32 subtraction), m' = a - ghat as before */
  RTOPK_OPT_DEVICE_STEP = 4,    /* 1 = the round number t that enters the Philox counter is kept in a word on
                                the device: the sparsify / step calls (plain, segmented, threshold) ignore
                                their `step` argument, read the word, and add one to it at their end (set it
                                with rtopk_set_device_step; it starts at 0).  A caller that captures one round
                                in a CUDA graph can then replay the graph round after round and still draw a
                                fresh subset each time.  0 = off (default): `step` is the argument */
  RTOPK_OPT_FINISH_PATH = 5,    /* how the candidates of the streaming pass become messages (the result is the
                                same): 0 (default) or 2 = three grid-wide launches over all slices that walk
                                the candidate list as the streaming pass left it (a histogram over the
                                bracket, a count, the emission; the k-of-r subset is drawn beside the first
                                two), with the cluster kernel behind them for what they leave (a missed
                                bracket, heavy ties); 1 = the cluster kernel alone: one thread-block cluster
                                per slice, which lays the candidate runs out in index order first (the subset
                                is then drawn beside the start of the streaming pass) */
  RTOPK_OPT_TEST_STREAM_GIVEUP = 6 /* for tests of the give-up path only: 1 = every block of the streaming pass
                                behaves as if its first bounded wait had run out (consumers at once, the
                                producer after a short wait for them).  The call still returns, all copies in
                                flight are waited for, nothing outside the caller's buffers is written, the
                                messages of that call are meaningless, and rtopk_poll_status reports
                                RTOPK_ERR_INTERNAL.  0 = off (default) */
};

/* Phases of one call, in stream order.  STREAM is the single pass over the full vectors that
 * performs a = g + m, writes it back and gathers the coordinates above the threshold. */
enum {
  RTOPK_PHASE_SUBSET = 0,    /* scratch clearing; the k-of-r subset itself runs on a stream of the context, beside
                                the kernels that follow the stream pass */
  RTOPK_PHASE_THRESHOLD = 1, /* first bracket of the r-th largest magnitude (sample, history or histogram pass) */
  RTOPK_PHASE_STREAM = 2,    /* the one kernel over W x d elements: add, write-back, candidate gathering */
  RTOPK_PHASE_ORDER = 3,     /* candidate runs laid out in index order; count check */
  RTOPK_PHASE_EXACT = 4,     /* empty (kept so that the phase numbers stay what they were) */
  RTOPK_PHASE_FINISH = 5,    /* exact threshold among the candidates (over the whole slice where the first
                                threshold missed), messages, residual zeroing */
  RTOPK_PHASE_AGGREGATE = 6, /* master average (step calls only) */
  RTOPK_N_PHASES = 7
};

/* Per-slice facts of the last sparsify call (one slice = one worker row, or one tensor of one
 * worker row in the segmented calls). */
typedef struct {
  uint32_t tau_key;     /* bit pattern (sign cleared) of the r-th largest magnitude */
  uint32_t tie_quota;   /* how many coordinates with exactly that magnitude are inside the top-r set */
  uint32_t n_greater;   /* coordinates with a strictly larger magnitude */
  uint32_t n_candidates;/* coordinates that survived the first threshold */
  uint32_t used_fallback; /* 1 if the first bracket missed and the slice was selected over all its coordinates */
  uint32_t bracket_predicted; /* 1 if the first threshold came from the slice's history, not from a sample */
  uint32_t reserved[2];
} rtopk_stats;

int rtopk_version(void);
const char* rtopk_status_string(int status);
/* cudaError_t (as int) of the last failing runtime call seen by this context, 0 if none. */
int rtopk_last_cuda_error(const rtopk_ctx* ctx);

/*
 * Creates a context on `device` with scratch sized for calls up to the given maxima:
 * vectors of at most d_max elements, W_max rows, r_max / k_max per slice summed over a row's
 * slices (for the plain calls: r and k), segments_max slices per row (1 for the plain calls).
 * The context owns its scratch (cudaMalloc) until rtopk_destroy.  d_max < 2^31.
 * A context with r_max = d_max whose candidate lists would take 2^30 entries or more (W_max * d_max, about)
 * is taken to be made for Definition 2's r = d (random-k), which needs no lists: it also serves calls
 * with r < d, but only up to about r = d_max / 32 per row (a call beyond what the lists hold returns
 * INVALID_ARG, as every call beyond the context's maxima does).
 * Errors: INVALID_ARG, ALLOC, CUDA.
 */
int rtopk_create(rtopk_ctx** out, int device, int64_t d_max, int32_t W_max, int64_t r_max,
                 int64_t k_max, int32_t segments_max);
int rtopk_destroy(rtopk_ctx* ctx);
int rtopk_set_option(rtopk_ctx* ctx, int option, int64_t value);

/*
 * Algorithm 1, node body, for W workers at once (add residual, Definition 3, residual update).
 *   grad      [in]      W x ld_g elements of grad_dtype, row-major; row w is worker worker_base+w;
 *                       never written.
 *   residual  [in/out]  W x ld_m binary32; on entry m (zero before the first step), on return m'.
 *   d                   vector length, 1 <= k <= r <= d < 2^31 (Definition 3's 1 <= k <= r <= d).
 *   ld_g, ld_m          row strides in elements, >= d, multiples of 4 (binary32) / 8 (bfloat16);
 *                       base pointers 16-byte aligned.  Padding columns are neither read nor written.
 *   worker_base         global id of row 0; enters the Philox counter so that a run sharded over
 *                       several GPUs draws the same subsets as the single-GPU run.
 *   seed, step          RNG key and the training step t; the caller advances step every round.
 *   msg_idx, msg_val [out]  W x k: row w holds worker w's k (index, value) pairs, ascending index.
 * Errors: INVALID_ARG (also when a size exceeds the context's maxima), CUDA.
 */
int rtopk_sparsify(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                   int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k,
                   uint64_t seed, uint32_t step, uint32_t* msg_idx, float* msg_val, void* stream);

/*
 * Algorithm 1, master step: out_i = scale * sum_w [i in U_w] val_{w,i}; scale_mode MEAN, SUM or
 * COUNT (UNBIASED: rtopk_aggregate_unbiased).
 * Sums run in double precision in worker order and are rounded once, so the result does not depend
 * on scheduling.  msg_idx rows must be ascending (as rtopk_sparsify writes them) with entries < d.
 *   msg_idx, msg_val [in]  W x k;   out [out]  d binary32, fully overwritten.
 * Errors: INVALID_ARG, CUDA.
 */
int rtopk_aggregate(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d,
                    int32_t W, int64_t k, int scale_mode, float* out, void* stream);

/*
 * rtopk_sparsify and rtopk_aggregate with the messages as one array of 8-byte (index, value) pairs: entry
 * j of worker w is the 64-bit word msg_pairs[w * k + j], low half the index, high half the bit pattern of
 * the binary32 value (ascending index, as always).  This is what a node sends in Algorithm 1 ("send
 * ghat_i"): one contiguous buffer of k pairs per worker, so that a run sharded over several GPUs moves its
 * messages with a single all-gather of W * k * 8 bytes and aggregates the gathered buffer in place.
 * msg_pairs is 8-byte aligned; everything else as in rtopk_sparsify / rtopk_aggregate (MEAN, SUM, COUNT;
 * UNBIASED needs r: scale the SUM by r / (W k)).
 */
int rtopk_sparsify_pairs(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                         int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k,
                         uint64_t seed, uint32_t step, uint64_t* msg_pairs, void* stream);
int rtopk_aggregate_pairs(rtopk_ctx* ctx, const uint64_t* msg_pairs, int64_t d, int32_t W, int64_t k,
                          int scale_mode, float* out, void* stream);

/* rtopk_aggregate with the UNBIASED scaling, which needs the r the messages were drawn from
 * (k <= r <= d).  Errors: INVALID_ARG, CUDA. */
int rtopk_aggregate_unbiased(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d,
                             int32_t W, int64_t k, int64_t r, float* out, void* stream);

/*
 * Sizes for round `step` under the schedule of Section IV: the sparsity grows exponentially over
 * the warm-up period and k / r = 1 / n throughout.  Host only, no GPU work.
 *   density(step) = initial * (final / initial)^(step / warmup_steps) for step < warmup_steps,
 *                   final afterwards;   k = clamp(floor(density * d), 1, d);   r = min(d, n * k).
 *   0 < final_density <= initial_density <= 1.   *r, *k [out] host.   Errors: INVALID_ARG.
 */
int rtopk_warmup_sizes(int64_t d, int32_t n_workers, double initial_density, double final_density,
                       int64_t warmup_steps, int64_t step, int64_t* r, int64_t* k);

/*
 * Packed message format.  Section III counts log d bits per index and a constant number of bits per
 * value; this format spends exactly b = ceil(log2 d) bits (at least 1) per index and 16 per value:
 *   packed_idx  W rows of ld_words 32-bit words: entry j of a row occupies bits [j b, (j + 1) b) of
 *               the row's bit stream, bit p of the stream being bit (p mod 32) of word p / 32;
 *   packed_val  W rows of ld_halves bfloat16 values (binary32 rounded to nearest, ties to even,
 *               upper 16 bits; NaN -> 0x7FC0).
 * rtopk_packed_layout (host only, no GPU work) returns b and the smallest accepted row strides
 * (ld_words a multiple of 4, ld_halves a multiple of 8); any of the three outputs may be null.
 * Errors: INVALID_ARG (d < 1, d >= 2^32, k < 1 or k > d).
 */
int rtopk_packed_layout(int64_t d, int64_t k, int32_t* index_bits, int64_t* ld_words, int64_t* ld_halves);

/*
 * Encodes W rows of k (index, value) pairs (as rtopk_sparsify writes them) into the packed format.
 * Algorithm 1 keeps m = a - ghat with ghat what is sent: when `residual` (W x ld_m, the buffer the
 * sparsify call updated) is not null, the slot of every sent coordinate receives the rounding error
 * a - widen(bfloat16(a)) (one binary32 subtraction; +0.0f when the rounded value is not finite).
 * Row padding of the outputs is written as zero.  All pointers are device pointers; packed_idx and
 * packed_val 16-byte aligned.  Errors: INVALID_ARG, CUDA.
 */
int rtopk_encode(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W,
                 int64_t k, float* residual, int64_t ld_m, uint32_t* packed_idx, int64_t ld_words,
                 uint16_t* packed_val, int64_t ld_halves, void* stream);

/* rtopk_aggregate reading the packed format directly (the decoder is fused into the aggregation
 * kernels).  scale_mode MEAN, SUM or COUNT.  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int rtopk_aggregate_packed(rtopk_ctx* ctx, const uint32_t* packed_idx, int64_t ld_words,
                           const uint16_t* packed_val, int64_t ld_halves, int64_t d, int32_t W,
                           int64_t k, int scale_mode, float* out, void* stream);

/*
 * Span-table message format, for rows in ascending index order (every message of this library is).
 * Section III's log d bits are what an index costs on its own; a sorted row can state the high bits of
 * its indices once per stretch.  The coordinates are cut into spans of 16384; per row
 *   span_tab   spans + 1 32-bit words, spans = ceil(d / 16384): span_tab[t] = how many of the row's
 *              entries have an index below t * 16384 (span_tab[0] = 0, span_tab[spans] = k); rows follow
 *              one another without padding (row stride spans + 1);
 *   low_idx    W rows of ld_low 16-bit words: index mod 16384 of every entry;
 *   packed_val W rows of ld_halves bfloat16 values, as in the packed format.
 * 32 (spans + 1) + 32 k bits per row (4.2 bytes per entry at d = 25.6 M, k = d / 1000; the packed format
 * takes 5.1, plain pairs 8), and the table is also what the aggregation needs to find every worker's
 * entries of an output tile, so rtopk_aggregate_tiled searches nothing.
 * rtopk_tiled_layout (host only, no GPU work) returns spans and the smallest accepted row strides
 * (multiples of 8); any output may be null.  Errors: INVALID_ARG (d < 1, d >= 2^32, k < 1 or k > d).
 */
int rtopk_tiled_layout(int64_t d, int64_t k, int64_t* spans, int64_t* ld_low, int64_t* ld_halves);

/*
 * Encodes W rows of k (index, value) pairs in strictly ascending index order (as rtopk_sparsify writes
 * them) into the span-table format; `residual` as in rtopk_encode (the rounding error of the values is
 * fed back).  Row padding of low_idx and packed_val is written as zero.  Device pointers; span_tab
 * 4-byte, low_idx and packed_val 16-byte aligned.  Rows that are not ascending give a table that does
 * not describe them (nothing is written out of bounds).  Errors: INVALID_ARG, CUDA.
 */
int rtopk_encode_tiled(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W,
                       int64_t k, float* residual, int64_t ld_m, uint32_t* span_tab, uint16_t* low_idx,
                       int64_t ld_low, uint16_t* packed_val, int64_t ld_halves, void* stream);

/* rtopk_aggregate reading the span-table format directly (decoder fused into the aggregation kernels;
 * table entries beyond k are read as k).  scale_mode MEAN, SUM or COUNT.  Errors: INVALID_ARG,
 * UNSUPPORTED, CUDA. */
int rtopk_aggregate_tiled(rtopk_ctx* ctx, const uint32_t* span_tab, const uint16_t* low_idx, int64_t ld_low,
                          const uint16_t* packed_val, int64_t ld_halves, int64_t d, int32_t W, int64_t k,
                          int scale_mode, float* out, void* stream);

/*
 * Algorithm 1, master update w <- w - eta * ghat applied straight from the messages: ghat is the
 * binary32 result rtopk_aggregate would write, and every coordinate that some worker sent receives
 * fp32(double(w_i) - double(eta) * double(ghat_i)) (one rounding); all other weights are not touched
 * (ghat_i = 0 there), so no dense vector is written.
 *   weights [in/out]  d binary32, 16-byte aligned;   eta  finite, >= 0.
 * Errors: INVALID_ARG (also for a negative or non-finite eta), CUDA.
 */
int rtopk_apply_update(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d,
                       int32_t W, int64_t k, int scale_mode, float eta, float* weights, void* stream);

/* rtopk_sparsify followed by rtopk_apply_update of the W messages it produced: one round of
 * Algorithm 1 including the master's update of the model.  Arguments as in the two calls. */
int rtopk_step_apply(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                     int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k,
                     uint64_t seed, uint32_t step, int scale_mode, float eta, uint32_t* msg_idx,
                     float* msg_val, float* weights, void* stream);

/*
 * The master update with momentum.  Section IV trains with momentum SGD and prints no formula; this is
 * the heavy-ball form applied to Algorithm 1's average ghat (the binary32 result rtopk_aggregate would
 * write), for EVERY coordinate i, sent or not:
 *     v_i <- fp32(double(mu) * double(v_i) + double(ghat_i));   w_i <- fp32(double(w_i) - double(eta) * double(v_i))
 * (one rounding per line; with mu = 0 the weights receive what rtopk_apply_update gives them).
 *   velocity, weights [in/out]  d binary32 each, 16-byte aligned, not overlapping;
 *   eta  finite, >= 0;   0 <= mu < 1;   r  only read with RTOPK_SCALE_UNBIASED (k <= r <= d).
 * Errors: INVALID_ARG, UNSUPPORTED (COUNT with more than 65535 workers), CUDA.
 */
int rtopk_apply_momentum(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val, int64_t d, int32_t W,
                         int64_t k, int scale_mode, int64_t r, float eta, float mu, float* velocity,
                         float* weights, void* stream);

/* rtopk_sparsify followed by rtopk_apply_momentum of the W messages it produced.  Arguments as in the
 * two calls. */
int rtopk_step_momentum(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                        int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k,
                        uint64_t seed, uint32_t step, int scale_mode, float eta, float mu, uint32_t* msg_idx,
                        float* msg_val, float* velocity, float* weights, void* stream);

/* One round of Algorithm 1's communication path: rtopk_sparsify followed by rtopk_aggregate of
 * the W messages it produced.  Arguments as in the two calls. */
int rtopk_step(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
               int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, int64_t r, int64_t k,
               uint64_t seed, uint32_t step, int scale_mode, uint32_t* msg_idx, float* msg_val,
               float* out, void* stream);

/*
 * Per-tensor variant: every row is cut into S slices at seg_off[0..S] (HOST array, seg_off[0] = 0,
 * seg_off[S] = d) and Definition 3 is applied to each slice with its own (seg_r[s], seg_k[s])
 * (HOST arrays), the slice number entering the Philox counter.  A row's message has
 * K = sum_s seg_k[s] pairs: slice 0's first; indices are positions in the whole vector, so the
 * row is still ascending and rtopk_aggregate applies unchanged with k = K.
 * The host arrays are read before the call returns.
 */
int rtopk_sparsify_segmented(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g,
                             float* residual, int64_t ld_m, int64_t d, int32_t W,
                             int32_t worker_base, int32_t S, const int64_t* seg_off,
                             const int64_t* seg_r, const int64_t* seg_k, uint64_t seed,
                             uint32_t step, uint32_t* msg_idx, float* msg_val, void* stream);
int rtopk_step_segmented(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g,
                         float* residual, int64_t ld_m, int64_t d, int32_t W, int32_t worker_base,
                         int32_t S, const int64_t* seg_off, const int64_t* seg_r,
                         const int64_t* seg_k, uint64_t seed, uint32_t step, int scale_mode,
                         uint32_t* msg_idx, float* msg_val, float* out, void* stream);

/*
 * Threshold-then-subsample encoder: the scheme in the proof of Theorem 1 (Section V), applied to
 * real-valued vectors the way Section II describes it for continuous observations: a coordinate of
 * a = g + m is marked ("1") when its magnitude exceeds theta, ||X_w||_1 = ones_w of worker w's
 * coordinates are; if ones_w > k, k of them are kept uniformly at random (Floyd / Philox as in
 * rtopk_sparsify, over the marked coordinates listed by ascending index, segment 0), otherwise all.
 * The message carries ones_w, count_w = min(ones_w, k) and the kept (index, value = a_i) pairs,
 * ascending; the node keeps m' = a - ghat (Algorithm 1).  "Exceeds" compares the magnitude bit
 * patterns strictly, so a NaN sum counts as marked.
 *   theta               finite, >= 0 (2 theta finite too with RTOPK_OPT_THRESHOLD_SIGNS).
 *   k                   message capacity (the proof's k'), 1 <= k <= min(d, the context's k_max).
 *   msg_idx, msg_val [out]  W x k; row w: count_w pairs, then padding (index 0xFFFFFFFF, value +0.0f).
 *   msg_count, msg_ones [out]  W 32-bit words each (device).
 * The scratch holds at most min(d, the context's r_max) marked coordinates per worker.  A worker
 * that marks more sends nothing in this call (count_w = 0, ones_w still reported, all of a stays in
 * its residual) and rtopk_poll_status reports RTOPK_ERR_INTERNAL: raise theta or create the context
 * with a larger r_max.
 * Errors: INVALID_ARG, UNSUPPORTED (RTOPK_OPT_SELECT_PATH = 1), CUDA.
 */
int rtopk_sparsify_threshold(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                             int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, float theta, int64_t k,
                             uint64_t seed, uint32_t step, uint32_t* msg_idx, float* msg_val, uint32_t* msg_count,
                             uint32_t* msg_ones, void* stream);

/*
 * The estimator of the same proof: out_i = (1/W) sum_w [i kept by w] val_{w,i} / S_w with the
 * subsampling fraction S_w = count_w / ones_w.  One term is double(val) * (double(ones_w) /
 * double(count_w)); terms are summed in double in worker order, divided by W and rounded once.
 *   msg_* [in] as rtopk_sparsify_threshold writes them (rows of several GPUs may be concatenated);
 *   out [out] d binary32, fully overwritten.
 * Errors: INVALID_ARG, CUDA.
 */
int rtopk_aggregate_threshold(rtopk_ctx* ctx, const uint32_t* msg_idx, const float* msg_val,
                              const uint32_t* msg_count, const uint32_t* msg_ones, int64_t d, int32_t W, int64_t k,
                              float* out, void* stream);

/* rtopk_sparsify_threshold followed by rtopk_aggregate_threshold of the messages it produced. */
int rtopk_step_threshold(rtopk_ctx* ctx, const void* grad, int grad_dtype, int64_t ld_g, float* residual,
                         int64_t ld_m, int64_t d, int32_t W, int32_t worker_base, float theta, int64_t k,
                         uint64_t seed, uint32_t step, uint32_t* msg_idx, float* msg_val, uint32_t* msg_count,
                         uint32_t* msg_ones, float* out, void* stream);

/*
 * rtopk_step with HOST gradient and HOST results.  h_grad (W x ld_g, ideally pinned, and complete when
 * the call is made) is copied to one of two device staging buffers owned by the context (allocated
 * on first use), the step runs on `stream` against the DEVICE residual, and the messages and the
 * dense update are copied back to h_msg_idx, h_msg_val (W x k) and h_out (d).  The copies run on two
 * streams of the context's own: the upload does not wait for `stream`, so in a sequence of calls it
 * overlaps the previous call's step and download; `stream` waits for the download, so work enqueued on
 * it afterwards, or a synchronisation of it, sees the results.  The call itself returns without
 * waiting.  h_grad must stay unchanged until the step that reads it has started (synchronise `stream`,
 * or make two further calls), the result buffers until `stream` has passed this call.
 * A call whose shape (W, ld_g, k or grad_dtype) differs from the previous host call's waits on the host
 * for the work of the earlier calls (`stream` and both copy streams) before it re-divides the staging
 * buffers, and a call that needs larger buffers than any before it also reallocates them (cudaFree /
 * cudaMalloc): keep the shape fixed inside a loop that must not stall.
 */
int rtopk_step_host(rtopk_ctx* ctx, const void* h_grad, int grad_dtype, int64_t ld_g,
                    float* residual, int64_t ld_m, int64_t d, int32_t W, int32_t worker_base,
                    int64_t r, int64_t k, uint64_t seed, uint32_t step, int scale_mode,
                    uint32_t* h_msg_idx, float* h_msg_val, float* h_out, void* stream);

/*
 * The k-of-r subset alone (Definition 3's U as positions in the top-r list): writes the k chosen
 * positions of (seed, step, worker, segment), ascending, to pos (device, k entries).
 */
int rtopk_sample_positions(rtopk_ctx* ctx, int64_t r, int64_t k, uint64_t seed, uint32_t step,
                           uint32_t worker, uint32_t segment, uint32_t* pos, void* stream);

/*
 * rtopk_sample_positions without a context and without any allocation.  (The paper has no
 * counterpart: this exists for the sake of callers, not of the method.)
 *
 * Who needs it: code that must not call cudaMalloc / cudaFree while it runs -- a training process
 * whose framework has already claimed the device memory for its own caching allocator, so that a
 * late cudaMalloc may fail or fragment it; a latency-critical loop with other streams in flight,
 * where the device-wide synchronisation hidden in cudaMalloc / cudaFree stalls everything; a host
 * program whose rules forbid allocation after start-up.  rtopk_create allocates its scratch, so
 * such callers cannot use a context; this call needs none.
 *
 * Its scratch (draw buffer, first-occurrence table, position bitmap and prefix: about 8.7 MB) is a
 * fixed array inside the library's device image.  Every GPU that loads the library holds that
 * array until the process exits, whether or not this call is ever made.
 *
 *   r, k      1 <= k <= r <= RTOPK_STATIC_MAX_R; a larger r returns RTOPK_ERR_UNSUPPORTED and
 *             nothing is enqueued (use a context for larger sets).
 *   pos [out] device, k entries: the chosen positions, ascending; same values as
 *             rtopk_sample_positions for the same (r, k, seed, step, worker, segment).
 * Works on the current device.  The first call on a device looks up the array's device address
 * (once per device); make that first call outside any stream capture.
 * All calls on a device share the one array, which still holds the previous call's contents: the
 * parts that must start clean are cleared at the start of every call, in stream order.  Two calls
 * whose work overlaps on the GPU (different streams, no ordering between them) race on the array
 * and give undefined positions; order them.
 * Calls no cudaMalloc, cudaFree or other allocating routine.
 * Errors: INVALID_ARG (null pos, k < 1, k > r), UNSUPPORTED (r too large), CUDA.
 */
#define RTOPK_STATIC_MAX_R (1 << 20)
int rtopk_sample_positions_static(int64_t r, int64_t k, uint64_t seed, uint32_t step, uint32_t worker,
                                  uint32_t segment, uint32_t* pos, void* stream);

/* Sets the context's round counter (RTOPK_OPT_DEVICE_STEP) to `step`, in stream order.  A bookkeeping
 * call with no counterpart in the paper beyond Algorithm 1's loop variable t.  Errors: INVALID_ARG, CUDA. */
int rtopk_set_device_step(rtopk_ctx* ctx, uint32_t step, void* stream);

/* Waits for `stream` and returns RTOPK_ERR_INTERNAL if any kernel of this context has raised the
 * device-side error flag since the last poll (the flag is then cleared), else RTOPK_OK. */
int rtopk_poll_status(rtopk_ctx* ctx, void* stream);

/* Waits for `stream`, then writes the duration in milliseconds of each phase of the last call
 * made with RTOPK_OPT_PROFILE on into ms[0..RTOPK_N_PHASES) (host); -1 where not recorded. */
int rtopk_get_phase_times(rtopk_ctx* ctx, float* ms, void* stream);

/* Waits for `stream` and copies the statistics of slice `slice` (row-major over rows x segments)
 * of the last sparsify call into *out (host). */
int rtopk_get_stats(rtopk_ctx* ctx, int32_t slice, rtopk_stats* out, void* stream);

/* Number of kernels this context has launched since rtopk_create (memsets and copies are not
 * counted; neither are the launches of rtopk_sample_positions_static, which has no context).
 * A bookkeeping call with no counterpart in the paper.  *out is host memory.  Errors: INVALID_ARG. */
int rtopk_get_launch_count(const rtopk_ctx* ctx, uint64_t* out);

#ifdef __cplusplus
}
#endif
#endif /* RTOPK_H_ */
