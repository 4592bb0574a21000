/* windq -- scoring and fitting hot path of WINDQuant-style mixed-precision allocation,
 * CUDA (sm_100a) library with a C ABI.
 *
 * The paper's PPO controller gives every column-chunk *unit* of every linear weight matrix one
 * of seven actions (Eq. 3, "Action Space"): skip (keep fp16) or quantize at 8, 4, 3, 2, 1.58 or
 * 1 bit.  This library computes what the controller needs in order to score units and actions:
 * calibration statistics, per-unit state features (Table 1), per-group quantizer fits under all
 * six bit-widths with their reconstruction errors (Sec. 3.5 "Quantization Engine and Bit
 * Accounting", App. "Per-unit Scale Optimization"), the application of a chosen plan, and
 * effective-bit accounting (Eq. 6).  The policy, the perplexity proxy and the model forward
 * are consumers and stay outside.
 *
 * Conventions (all calls)
 *   - A linear weight is W[R][C], fp16 (IEEE binary16), row-major with leading dimension ldw
 *     (elements): R = out features, C = in features.  Unit u = columns [u*G, (u+1)*G) of all R
 *     rows; U = C / G.  A *group* (r, u) is the G contiguous values of row r in unit u; it
 *     carries one scale (and one zero point).
 *   - Action codes follow Eq. 3: 0 = skip(16)  1 = 8  2 = 4  3 = 3  4 = 2  5 = 1.58  6 = 1.
 *     Per-bit-width tables have six columns in the order [8, 4, 3, 2, 1.58, 1].
 *   - Every data pointer is a DEVICE pointer owned by the caller, unless it says "host".
 *     Nothing is retained after a call.  `stream` is a cudaStream_t passed as void* (NULL = the
 *     legacy default stream).  Calls only enqueue work on `stream`; outputs are valid once the
 *     stream has reached that point.  The library allocates no outputs.  It owns a scratch
 *     buffer inside the context, grown (cudaMalloc, which synchronises) only when a call needs
 *     more than it has; windq_reserve sizes it ahead of time.
 *   - Errors: every argument check happens on the host before anything is launched; a failing
 *     call launches nothing and returns a status, and windq_last_error gives the reason.  There
 *     are no exceptions, aborts or device traps.  Inputs must be finite; NaN / Inf give
 *     unspecified values, never a fault.  A context must not be used from two threads at once.
 *   - Ordering.  Every call on a context works in that context's one scratch buffer, from its
 *     first byte (the item counter and partial sums of the fits, the histograms of the feature
 *     and selection passes, the row counts of protected packing, the allocator's tables).  Two
 *     calls on the same context must therefore not overlap on the GPU: issue them on one stream,
 *     or order the streams with events (the later call's stream waits for an event recorded
 *     after the earlier call), or give every stream a context of its own.  Calls on one context
 *     from unordered streams corrupt each other's results silently.
 *   - Pointers to fp16 / fp32 / int64 arrays must be 16-byte aligned (any cudaMalloc or torch
 *     allocation is); ldw and ldx must be multiples of 8.
 *   - G must be one of 32, 64, 128, 256, 512; C a multiple of G; 1 <= K <= 64; clip ratios in
 *     [1/64, 1].
 */
#ifndef WINDQ_H_
#define WINDQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct windq_ctx windq_ctx; /* opaque: device id, SM count, scratch, last error */

typedef enum {
  WINDQ_OK = 0,
  WINDQ_ERR_NULL = 1,        /* a required pointer is NULL */
  WINDQ_ERR_SHAPE = 2,       /* a size is <= 0, C % G != 0, ld < C, ... */
  WINDQ_ERR_ALIGN = 3,       /* a pointer or leading dimension is misaligned */
  WINDQ_ERR_ARG = 4,         /* G, K, a clip ratio or a bit count is out of range */
  WINDQ_ERR_SCRATCH = 5,     /* the scratch buffer could not be grown */
  WINDQ_ERR_CUDA = 6,        /* a CUDA runtime call or a launch failed */
  WINDQ_ERR_UNSUPPORTED = 7  /* the device is not an sm_100 GPU */
} windq_status;

#define WINDQ_N_BITWIDTHS 6
#define WINDQ_N_FEATURES 8

/* Creates a context on CUDA device `device` (the caller's current device is left unchanged).
 * *out receives the context (host memory, freed by windq_destroy). */
windq_status windq_create(windq_ctx** out, int device);
void windq_destroy(windq_ctx* ctx);

/* Reason of the last failing call on this context (or of the last failing windq_create when ctx
 * is NULL).  The string is owned by the library and stays valid until the next call. */
const char* windq_last_error(const windq_ctx* ctx);

/* Checks, on the device, an arithmetic shortcut the fits rely on: the reciprocal of a stored scale is formed by
 * the hardware approximation and one Newton step instead of a full IEEE division; for every positive finite fp16
 * value (all a stored scale can be) the two must agree bit for bit.  n_failures_out (i64 [1], device) receives
 * the number of values for which they do not: 0 on every GPU this library supports. */
windq_status windq_selfcheck(windq_ctx* ctx, int64_t* n_failures_out, void* stream);

/* How much of the clip search the fits skipped (the paper has no counterpart; a measurement aid).  The eight-bit
 * search of windq_fit_eval and its variants leaves out candidates that provably cannot win (the error of a group
 * is at least the error term of any one of its weights; see windq_fit_eval), so the work of a fit depends on the
 * data.  Every fit kernel of the context adds to two counters: the clip candidates of its searches, counted once
 * per warp pass (a pass covers the 1024 weights a warp holds), and those of them it evaluated in full.
 *   evaluated_out, searched_out: HOST pointers to one int64 each; reset != 0 puts both counters back to zero.
 * Synchronises the device (a blocking copy). */
windq_status windq_fit_work(windq_ctx* ctx, int64_t* evaluated_out, int64_t* searched_out, int reset);

/* Grows the context's scratch buffer to at least `bytes` now (synchronises the device), so that
 * later calls do not allocate.  windq_scratch_bytes_* tell how much a call will need. */
windq_status windq_reserve(windq_ctx* ctx, int64_t bytes);
int64_t windq_scratch_bytes_act_stats(int64_t T, int64_t C);
int64_t windq_scratch_bytes_unit_features(int64_t R, int64_t C, int G);
int64_t windq_scratch_bytes_fit_eval(int64_t R, int64_t C, int G);

/* a1 -- activation statistics of one calibration input (App. "Salient Weight Protection":
 * per-channel activation scale estimated during a calibration forward pass; Table 1 dims 9-11).
 *   s_out[j] = (1/T) * sum_t X[t][j]^2,  j < C.
 * X: fp16 [T][ldx] (T tokens, C channels, ldx >= C); s_out: fp32 [C].  C % 8 == 0. */
windq_status windq_act_stats(windq_ctx* ctx, const void* X, int64_t T, int64_t C, int64_t ldx,
                             float* s_out, void* stream);

/* windq_act_stats for several calibration inputs in one launch (the paper has no counterpart: a decoder block has
 * a handful of distinct inputs of a few tens of megabytes, each too short a read to amortise a launch of its own).
 * Every job is one windq_act_stats call -- X, T, C, ldx, s_out as there -- and gives the same bits.
 *   jobs: HOST array of n_jobs descriptors (1 <= n_jobs <= WINDQ_MAX_ACT_JOBS), read during the call only.
 * The channels of all jobs together may number at most 4 194 304.
 * Scratch: windq_scratch_bytes_act_stats_batch (the sum of the jobs' windq_scratch_bytes_act_stats). */
#define WINDQ_MAX_ACT_JOBS 16
typedef struct {
  const void* X;  /* fp16 [T][ldx] */
  int64_t T, C, ldx;
  float* s_out;   /* fp32 [C] */
} windq_act_job;
int64_t windq_scratch_bytes_act_stats_batch(const windq_act_job* jobs, int n_jobs);
windq_status windq_act_stats_batch(windq_ctx* ctx, const windq_act_job* jobs, int n_jobs, void* stream);

/* Variant of windq_act_stats that allocates nothing.  (The paper has no counterpart: this entry
 * point exists for the sake of callers, not of the method.)
 *
 * windq_act_stats keeps its per-slice partial sums in the context's scratch buffer, which it
 * grows with cudaMalloc when a call needs more than is there.  Some hosts cannot afford that: a
 * process whose device memory has been handed out completely to its own pool, so that a fresh
 * cudaMalloc fails; a latency-bound loop that must not take the device-wide synchronisation
 * cudaMalloc and cudaFree imply; code that runs where only kernel launches are allowed.  For them
 * this call keeps the partial sums in an array of WINDQ_NOALLOC_SCRATCH_BYTES that is built into
 * the library image.  Every device that loads the library's device code holds that array until
 * the process exits, whether or not this entry point is ever called.
 *
 * Arguments, layout, result and argument errors are those of windq_act_stats.  In addition:
 *   - the call needs 4 * C * ceil(T / 64) bytes of the array (windq_scratch_bytes_act_stats
 *     gives the figure); a larger request is refused with WINDQ_ERR_SCRATCH before anything is
 *     launched -- use windq_act_stats, or call once per block of tokens and combine the means;
 *   - this entry point calls no cudaMalloc, cudaFree or other allocating routine, on any path;
 *   - the first call on a device asks the runtime for the array's device address (one
 *     cudaGetSymbolAddress, kept per device afterwards).  With the CUDA runtime's default lazy
 *     loading that request, or the first kernel launch of the library, is also the moment the
 *     driver loads the library's device code on that device and reserves the array: the driver
 *     itself takes device memory then (the array and the code), and may synchronise.  So make
 *     the first call per device at start-up -- before the process hands its device memory to a
 *     pool of its own, and outside any stream capture; every later call finds the address kept
 *     and only launches;
 *   - all calls on a device share the one array, and it keeps whatever the last call left.  That
 *     is harmless from call to call, because every partial sum that is read has been written by
 *     the same call first; but two calls whose kernels can overlap on the GPU (different streams
 *     with no ordering between them, or two contexts on one device) race on it and give wrong
 *     results.  Order such calls on one stream or with events.
 *   - at most 64 devices (device index below 64). */
#define WINDQ_NOALLOC_SCRATCH_BYTES (4 * 1024 * 1024)
windq_status windq_act_stats_noalloc(windq_ctx* ctx, const void* X, int64_t T, int64_t C, int64_t ldx,
                                     float* s_out, void* stream);

/* a2 -- state features of every unit (Table 1, dims 0-4 and 9-11).
 *   feat_out[u] = { mean, std, abs_mean, sparsity, outlier_frac, mean(s), std(s), max(s) }
 * over the R*G weights of unit u and the G statistics s[u*G .. (u+1)*G).  std is the population
 * standard deviation; sparsity = #{|w| < 1e-6} / n; outlier_frac = #{|w| > 0.5 * P99} / n with
 * P99 the ceil(0.99 n)-th smallest |w| (nearest rank).  Both counts are exact.
 * W: fp16 [R][ldw]; s: fp32 [C]; feat_out: fp32 [U][8]. */
windq_status windq_unit_features(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                 int G, const float* s, float* feat_out, void* stream);

/* a3 -- fit every group under all six bit-widths and score each fit by its s-weighted squared
 * reconstruction error  e = sum_j s_j (w_j - w^_j)^2  (Sec. 3.5: local scale fitting per unit,
 * judged by reconstruction error; App.: group size = chunk size).
 *   8/4/3/2 bit: asymmetric uniform grid over [p*mn, p*mx] (mn = min(0, min w), mx = max(0, max
 *     w)), scale rounded to fp16, integer zero point; every clip ratio p = clip_grid[k] is tried
 *     and the smallest k with the least error kept.
 *   1.58 bit: threshold 0.7 * mean|w|, one fp16 scale = s-weighted mean |w| on the support.
 *   1 bit: sign(w) times one fp16 scale = s-weighted mean |w|.
 * Outputs:
 *   err_out      fp32 [U][6]     sum over rows of the best error, per bit-width
 *   energy_out   fp32 [U]        sum_r sum_j s_j w_rj^2 (error of "quantize to zero"); nullable
 *   clip_idx_out u8   [4][U][R]  best clip index for 8, 4, 3, 2 bit; nullable
 *   group_err_out fp32 [6][U][R] best error of every group; nullable
 * clip_grid: fp32 [K] (device).  Group-level results (clip indices, group errors) are
 * bit-reproducible: every operation is a fixed IEEE binary32 sequence.
 * s must be >= 0 (it is a mean of squares).  The eight-bit search relies on it: every term s_j d_j^2 of an error is
 * then >= 0 and rounding is monotone, so the error of a candidate is at least the term of any single weight, and
 * a candidate for which the term of a group's least or greatest weight already exceeds the least error found is
 * skipped without changing any result (windq_fit_work tells how many were).  With negative s the results are
 * unspecified, like those of non-finite input. */
windq_status windq_fit_eval(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                            const float* s, const float* clip_grid, int K, float* err_out,
                            float* energy_out, uint8_t* clip_idx_out, float* group_err_out,
                            void* stream);

/* a5 -- effective bits of a plan for one matrix (Eq. 6 with no protected weights, extended by
 * the per-group scale / zero-point overhead), in integer centibits (1 bit = 100), and the byte
 * offsets of the packed code blocks that windq_apply_plan writes.  With n = R*G:
 *   skip: 1600 n;  b in {8,4,3,2}: 100 b n + 100 R (scale_bits + zero_bits);
 *   1.58: 158 n + 100 R scale_bits;  1: 100 n + 100 R scale_bits.
 * Bytes of one packed group: skip 2G, 8-bit G, 4-bit G/2, 3-bit 3G/8, 2-bit G/4, 1.58-bit
 * ceil(G/5), 1-bit G/8.  A unit's block holds its R groups in row order; every block starts on a
 * 16-byte boundary.
 *   actions               u8  [U]    action code per unit (device)
 *   unit_centibits_out    i64 [U]    nullable
 *   code_offsets_out      i64 [U+1]  byte offset of every block, [U] = total code bytes; nullable
 *   total_centibits_out   i64 [1]    sum over units; average bits = total / (100 * U * R * G)
 *   total_packed_bytes_out i64 [1]   code bytes + 2 bytes per stored scale and zero point; nullable
 * An action code above 6 makes both totals -1 (the per-unit entry is -1, its block empty).
 * scale_bits and zero_bits must be in [0, 64]. */
windq_status windq_effective_bits(windq_ctx* ctx, const uint8_t* actions, int64_t U, int64_t R, int G,
                                  int scale_bits, int zero_bits, int64_t* unit_centibits_out,
                                  int64_t* code_offsets_out, int64_t* total_centibits_out,
                                  int64_t* total_packed_bytes_out, void* stream);

/* windq_unit_features for several matrices in one pass (no counterpart in the paper; same reason as
 * windq_fit_eval_batch below).  Every job is one windq_unit_features call: W, R, C, ldw, s, feat_out as there;
 * all jobs share G.  The features that come from the histogram (std, abs_mean, sparsity, outlier_frac) and
 * those of s are those of the separate calls bit for bit; the mean is a sum of block sums whose blocks fall
 * differently, so its last bits can differ (within 1e-6 relative).
 *   jobs: HOST array of n_jobs descriptors (1 <= n_jobs <= 16), read during the call only.
 * Scratch: windq_scratch_bytes_unit_features_batch (128 KB per unit of all jobs). */
typedef struct {
  const void* W;    /* fp16 [R][ldw] */
  int64_t R, C, ldw;
  const float* s;   /* fp32 [C] */
  float* feat_out;  /* fp32 [U][8] */
} windq_feat_job;
int64_t windq_scratch_bytes_unit_features_batch(const windq_feat_job* jobs, int n_jobs, int G);
windq_status windq_unit_features_batch(windq_ctx* ctx, const windq_feat_job* jobs, int n_jobs, int G, void* stream);

/* windq_unit_features_batch at TWO chunk widths, G and 2 G, from one pass over the weights (the paper has no
 * counterpart; its chunk-size ablation scores the same model at nested chunk sizes).  A unit of width 2 G is the union
 * of two neighbouring units of width G, and the histogram of a union is the sum of the histograms, so the wider units'
 * features come from the histograms the pass has built anyway -- the same values as a windq_unit_features_batch
 * call at 2 G (histogram features and those of s bit for bit; the mean within 1e-6 relative).
 *   feat_out_2G: HOST array of n_jobs device pointers, fp32 [C / (2 G)][8] each, or NULL for a job that wants
 *   width G only; with any non-NULL entry every job's C must be a multiple of 2 G.  G <= 256.
 * Everything else as windq_unit_features_batch, including the scratch size. */
windq_status windq_unit_features_batch2(windq_ctx* ctx, const windq_feat_job* jobs, float* const* feat_out_2G, int n_jobs,
                                        int G, void* stream);

/* windq_fit_eval for several matrices in one launch (the paper has no counterpart: the consumer loops
 * over the seven projections of every block, and matrices that are small against the GPU -- a few million
 * weights -- neither fill it nor amortise the fixed cost of a call on their own).  All jobs share G, the
 * clip grid and K; every job is one windq_fit_eval: W, R, C, ldw, s and the four outputs with the meanings,
 * layouts and nullability given there.  Results are those of the separate calls (group errors and clip
 * indices bit for bit; unit sums to the last bit too, being added in the same order).
 *   jobs: HOST array of n_jobs descriptors (1 <= n_jobs <= 16), read during the call only; the pointers
 *   inside are device pointers.  Scratch: windq_scratch_bytes_fit_eval_batch. */
typedef struct {
  const void* W;          /* fp16 [R][ldw] */
  int64_t R, C, ldw;
  const float* s;         /* fp32 [C] */
  float* err_out;         /* fp32 [U][6] */
  float* energy_out;      /* fp32 [U], nullable */
  uint8_t* clip_idx_out;  /* u8 [4][U][R], nullable */
  float* group_err_out;   /* fp32 [6][U][R], nullable */
  void* lowbit_out;       /* fp16 [3][U][R], nullable: per group the 1.58-bit scale, the 1-bit scale and the 1.58-bit
                             threshold 0.7 * mean|w| rounded towards zero to fp16 -- what windq_apply_plan_multi can
                             take in place of forming the low-bit sums again (as it takes the clip indices) */
} windq_fit_job;
int64_t windq_scratch_bytes_fit_eval_batch(const windq_fit_job* jobs, int n_jobs, int G);
windq_status windq_fit_eval_batch(windq_ctx* ctx, const windq_fit_job* jobs, int n_jobs, int G, const float* clip_grid,
                                  int K, void* stream);

/* windq_unit_features_batch and windq_fit_eval_batch in ONE pass over the weights (the paper has no counterpart: its
 * state features, Table 1, and its engine's fits, Sec. 3.5, are computed on the same chunk).  The fit pass holds every
 * weight in registers anyway; it also counts it in its unit's histogram of |w| bit patterns and adds it to the unit's
 * sum, so that the features need no second read of the matrix and no pass of their own.  Every job is one
 * windq_fit_eval call plus one windq_unit_features call on the same W and s: the fit outputs are those of
 * windq_fit_eval_batch bit for bit, the features those of windq_unit_features (the histogram features and those of s
 * bit for bit; the mean is a sum of block sums whose blocks fall differently: within 1e-6 relative).
 * Measured on B200 this call is SLOWER than the two it replaces (5.05 against 4.07 ms for a 7B-shaped block at chunk
 * width 128): the histogram updates are atomics in global memory, and the fit's own shared-memory loads queue behind
 * them.  It saves the second read of the weights, which matters only where memory traffic, not time, is the constraint.
 *   jobs: HOST array of n_jobs descriptors (1 <= n_jobs <= 16), read during the call only.
 * Scratch: windq_scratch_bytes_features_fit_batch (the fit's partial sums + 128 KB per unit of all jobs). */
typedef struct {
  const void* W;          /* fp16 [R][ldw] */
  int64_t R, C, ldw;
  const float* s;         /* fp32 [C] */
  float* feat_out;        /* fp32 [U][8] */
  float* err_out;         /* fp32 [U][6] */
  float* energy_out;      /* fp32 [U], nullable */
  uint8_t* clip_idx_out;  /* u8 [4][U][R], nullable */
  float* group_err_out;   /* fp32 [6][U][R], nullable */
  void* lowbit_out;       /* fp16 [3][U][R], nullable (see windq_fit_job) */
} windq_featfit_job;
int64_t windq_scratch_bytes_features_fit_batch(const windq_featfit_job* jobs, int n_jobs, int G);
windq_status windq_features_fit_batch(windq_ctx* ctx, const windq_featfit_job* jobs, int n_jobs, int G,
                                      const float* clip_grid, int K, void* stream);

/* windq_effective_bits for several plans in one launch (plans of different matrices may differ in U and R;
 * G, scale_bits and zero_bits are shared).  Every job is one windq_effective_bits call with the same meanings,
 * nullability and results.  Two jobs must not share an output array.
 *   jobs: HOST array of n_jobs descriptors (1 <= n_jobs <= 32), read during the call only. */
typedef struct {
  const uint8_t* actions;           /* u8 [U] */
  int64_t U, R;
  int64_t* unit_centibits_out;      /* i64 [U], nullable */
  int64_t* code_offsets_out;        /* i64 [U+1], nullable */
  int64_t* total_centibits_out;     /* i64 [1] */
  int64_t* total_packed_bytes_out;  /* i64 [1], nullable */
} windq_bits_job;
windq_status windq_effective_bits_batch(windq_ctx* ctx, const windq_bits_job* jobs, int n_jobs, int G, int scale_bits,
                                        int zero_bits, void* stream);

/* a4 -- apply a plan to one matrix ("Transition and Discount": after the policy has chosen, the
 * environment quantizes the current unit with the chosen operator): integer codes packed as
 * described above, the fp16 scale and zero point of every group, and optionally the
 * fake-quantised weights for the consumer's forward pass.
 *   actions      u8  [U]          action per unit
 *   clip_idx     u8  [4][U][R]    clip indices from windq_fit_eval, or NULL: the clip search is
 *                                 repeated for the chosen bit-width (same result, more work).
 *                                 An index >= K is treated as K-1.
 *   code_offsets i64 [U+1]        from windq_effective_bits for the same actions, R and G
 *   codes_out    u8  [code_offsets[U]]  every byte is written (padding = 0)
 *   scales_out   fp16 [U][R]      scale (alpha for 1.58 / 1 bit, 0 for skip)
 *   zeros_out    fp16 [U][R]      integer zero point (0 for 1.58 / 1 bit and skip)
 *   Wq_out       fp16 [R][ldw]    fake-quantised weights, nullable; must not alias W
 * Packing inside a group, little-endian within a byte: 8-bit byte j = q_j; 4-bit byte i = q_2i |
 * q_2i+1 << 4; 3-bit: a bit stream, code j at bits [3j, 3j+3); 2-bit byte i = sum q_4i+m << 2m;
 * 1.58-bit byte i = sum_{m<5} t_5i+m 3^m with trits t = 1 + sign(w) on the support, 1 elsewhere;
 * 1-bit byte i = sum bit_8i+m << m with bit = !(w < 0); skip: the raw fp16 bytes.
 * Action codes live on the device, so they cannot be checked before the launch: a unit whose code
 * is above 6 is skipped -- its codes, scales, zero points and fake-quantised weights keep whatever
 * the output arrays held -- and the call still returns WINDQ_OK.  windq_effective_bits reports such
 * a plan (totals of -1); check its total before applying a plan that was not produced by trusted
 * code.  The same holds for every windq_apply_plan* variant.  codes_out must be 16-byte aligned. */
windq_status windq_apply_plan(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                              const float* s, const float* clip_grid, int K, const uint8_t* actions,
                              const uint8_t* clip_idx, const int64_t* code_offsets, uint8_t* codes_out,
                              void* scales_out, void* zeros_out, void* Wq_out, void* stream);

/* Several plans of ONE matrix in one pass over its weights (the paper has no counterpart; a consumer that
 * compares candidate plans, or keeps plans for several bit budgets, packs them together): every weight is read
 * from memory once and quantised under each plan in turn.  Every plan is one windq_apply_plan call with clip
 * indices (clip_idx u8 [4][U][R] is required and shared by the plans): same meanings, layouts and results, bit
 * for bit.  Plans must not share output arrays; Wq_out may be NULL in any of them.
 *   lowbit: fp16 [3][U][R] (device) or NULL: lowbit_out of windq_fit_eval_batch for the same W, s and G.  With it the
 *           1.58- and 1-bit units take their scale (and threshold) from the table instead of forming the sums of the
 *           fit again: same results, about a third less time on plans that are mostly low-bit.
 *   plans: HOST array of n_plans descriptors (1 <= n_plans <= 4), read during the call only. */
typedef struct {
  const uint8_t* actions;       /* u8 [U] */
  const int64_t* code_offsets;  /* i64 [U+1] */
  uint8_t* codes_out;
  void* scales_out;             /* fp16 [U][R] */
  void* zeros_out;              /* fp16 [U][R] */
  void* Wq_out;                 /* fp16 [R][ldw], nullable */
} windq_plan_out;
windq_status windq_apply_plan_multi(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                    const float* s, const float* clip_grid, int K, const uint8_t* clip_idx,
                                    const void* lowbit, const windq_plan_out* plans, int n_plans, void* stream);

/* windq_apply_plan for several (matrix, plan) pairs in one launch.  Every job is one windq_apply_plan call with
 * clip indices (clip_idx is required here): same meanings, layouts and results, bit for bit.  All jobs share G,
 * the clip grid and K.  Jobs must not share output arrays (two plans of one matrix need two Wq_out, or NULL).
 *   jobs: HOST array of n_jobs descriptors (1 <= n_jobs <= 24), read during the call only. */
typedef struct {
  const void* W;                /* fp16 [R][ldw] */
  int64_t R, C, ldw;
  const float* s;               /* fp32 [C] */
  const uint8_t* actions;       /* u8 [U] */
  const uint8_t* clip_idx;      /* u8 [4][U][R] */
  const int64_t* code_offsets;  /* i64 [U+1] */
  uint8_t* codes_out;
  void* scales_out;             /* fp16 [U][R] */
  void* zeros_out;              /* fp16 [U][R] */
  void* Wq_out;                 /* fp16 [R][ldw], nullable */
} windq_apply_job;
windq_status windq_apply_plan_batch(windq_ctx* ctx, const windq_apply_job* jobs, int n_jobs, int G,
                                    const float* clip_grid, int K, void* stream);

/* ---- beyond the five calls: salient-weight protection (App. "Salient Weight Protection") ---------
 *
 * The paper keeps, in every unit, the top-r fraction of the weights by saliency -- weight magnitude
 * times the activation scale of the weight's input channel -- in INT8 and counts them at 8 bits in
 * Eq. 6.  windq_salient_select finds that set exactly; windq_effective_bits_protected is Eq. 6 with
 * it; windq_fit_eval_protected scores the fits with those weights left out; windq_apply_plan_protected
 * packs a plan with the INT8 side storage for them.
 *
 *   key(r, j)  = |W[r][j]| * sqrt(s[j])            two binary32 operations (sqrt, then product)
 *   n_p        = floor(rate_ppm * R * G / 10^6)     weights asked for per unit (rate in parts per million)
 *   thresh_out fp32 [U]   the n_p-th largest key of the unit; +infinity when n_p = 0
 *   count_out  i64  [U]   number of keys >= thresh: keys equal to the threshold are all protected, so
 *                         the count can exceed n_p; it is the n^(p) of Eq. 6
 *   mask_out   u8   [R][C/8], nullable   bit (j % 8) of byte [r][j / 8] is set for a protected weight
 * R * G must be below 2^32.  Scratch: windq_scratch_bytes_salient_select. */
int64_t windq_scratch_bytes_salient_select(int64_t R, int64_t C, int G);
windq_status windq_salient_select(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                  const float* s, int64_t rate_ppm, float* thresh_out, int64_t* count_out,
                                  uint8_t* mask_out, void* stream);

/* windq_fit_eval with the protected weights taken out of the fits: a weight whose key reaches
 * thresh[u] (fp32 [U], device, from windq_salient_select with the same W, s and G) counts, inside its
 * group, as a zero weight with zero activation weight -- it leaves the range, every sum and every
 * error, while its position and the group size stay.  The error of its INT8 copy is not part of the
 * outputs.  With every threshold +infinity the results are those of windq_fit_eval, bit for bit.
 * Outputs and the other arguments as windq_fit_eval; scratch: windq_scratch_bytes_fit_eval_protected. */
int64_t windq_scratch_bytes_fit_eval_protected(int64_t R, int64_t C, int G);
windq_status windq_fit_eval_protected(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                      const float* s, const float* clip_grid, int K, const float* thresh,
                                      float* err_out, float* energy_out, uint8_t* clip_idx_out, float* group_err_out,
                                      void* stream);

/* windq_apply_plan with salient-weight protection.  In every unit that is not skipped, a weight whose
 * key reaches thresh[u] is protected: inside its group it counts as a zero weight with zero activation
 * weight (as in windq_fit_eval_protected, whose clip indices this call takes), so scales, zero points
 * and the codes of the other weights are those of the masked group, and its own slot in the packed
 * stream holds the code of the value 0 (a reader skips it by the mask of windq_salient_select).  The
 * protected weights of a unit share one symmetric INT8 grid (the paper says no more than that they are kept in INT8):
 *   prot_scale_out   fp16 [U]     sigma_u = fp16(max |w| over the unit's protected weights / 127), 1 if that
 *                                 is zero; 0 for a skipped unit, which protects nothing
 *   prot_offsets_out i64  [U+1]   start of every unit's INT8 codes in prot_q_out; [U] = their number
 *   prot_q_out       i8   [prot_q_capacity]  codes clamp(rne(w / sigma_u), -127, 127), per unit in row-major
 *                                 order (rows, then columns).  Nothing is written at or beyond prot_q_capacity:
 *                                 size it from the counts of windq_salient_select, or compare prot_offsets_out[U]
 *   Wq_out                        fp16(code * sigma_u) at the protected positions
 * Everything else as windq_apply_plan.  Scratch: windq_scratch_bytes_apply_plan_protected. */
int64_t windq_scratch_bytes_apply_plan_protected(int64_t R, int64_t C, int G);
windq_status windq_apply_plan_protected(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                        const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                        const uint8_t* clip_idx, const int64_t* code_offsets, const float* thresh,
                                        uint8_t* codes_out, void* scales_out, void* zeros_out, void* Wq_out,
                                        void* prot_scale_out, int64_t* prot_offsets_out, int8_t* prot_q_out,
                                        int64_t prot_q_capacity, void* stream);

/* Eq. 6 in full, in centibits: 1600 n for a skipped unit (nothing of it is protected), otherwise
 * 100 b (n - n_p) + 800 n_p, plus 100 R (scale_bits [+ zero_bits for 8/4/3/2 bit]) for the groups'
 * parameters as in windq_effective_bits.  n_protected: i64 [U] (device), e.g. count_out above.
 * An action code above 6 or a count outside [0, R * G] makes the total -1 (that unit's entry -1).
 *   unit_centibits_out i64 [U], nullable;  total_centibits_out i64 [1] */
windq_status windq_effective_bits_protected(windq_ctx* ctx, const uint8_t* actions, const int64_t* n_protected,
                                            int64_t U, int64_t R, int G, int scale_bits, int zero_bits,
                                            int64_t* unit_centibits_out, int64_t* total_centibits_out, void* stream);

/* Saliency score of every unit ("Comparison with Heuristic Sensitivity Allocator": the mean product of
 * activation scale and weight magnitude), the quantity the paper's heuristic allocator ranks units by:
 *   sal_out[u] = (1 / (R G)) * sum over the unit of sqrt(s[j]) * |W[r][j]|        fp32 [U]
 * (double accumulation; the order of the block sums is not fixed, so the last bits can differ from run
 * to run; within 1e-6 relative of the exact value). */
windq_status windq_unit_saliency(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                 const float* s, float* sal_out, void* stream);

/* Iterative refinement of the step sizes (App. "Per-unit Scale Optimization": the selected operator fits
 * its scale by a small local optimisation, typically 10 Adam steps, on the reconstruction loss of the
 * chunk; the 3/4/8-bit operators learn step sizes with straight-through estimation of the rounding).
 * The paper prints no formulas; this call does the following for the four uniform bit-widths (8, 4, 3,
 * 2), per group, in binary32:
 *   warm start  the clip-grid fit that clip_idx names: Delta_0 = its fp16 scale, its zero point z stays
 *   iterate t   Delta_h = fp16(Delta_t);  c_j = clamp(rne(w_j / Delta_h), -z, qmax - z);
 *               d_j = c_j Delta_h - w_j;  loss e_t = sum s_j d_j^2  (the operations of windq_fit_eval)
 *               psi_j = rne(w_j / Delta_h) - w_j / Delta_h in range, c_j where clipped;  g_t = sum s_j d_j psi_j
 *   Adam        beta1 0.9, beta2 0.999, eps 1e-8, bias-corrected, learning rate lr * Delta_0
 *   result      the iterate of least loss among t = 0..n_steps (the first on ties), so no error exceeds
 *               that of windq_fit_eval; a group stops early when fp16(Delta) is not positive and finite
 * Arguments as windq_fit_eval, and
 *   clip_idx      u8   [4][U][R]  from windq_fit_eval for the same W, s, G and grid (an index >= K is K-1)
 *   n_steps       0..32 (host);  lr in [0, 1] (host): step of the first update relative to Delta_0
 *   err_out       fp32 [U][4]     unit sums of the refined group errors (double accumulation)
 *   scale_out     fp16 [4][U][R]  refined scales
 *   group_err_out fp32 [4][U][R]  nullable
 * With n_steps = 0 scales and group errors are those of the clip-grid fit, bit for bit.  Scratch:
 * windq_scratch_bytes_fit_refine. */
int64_t windq_scratch_bytes_fit_refine(int64_t R, int64_t C, int G);
windq_status windq_fit_refine(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                              const float* clip_grid, int K, const uint8_t* clip_idx, int n_steps, float lr,
                              float* err_out, void* scale_out, float* group_err_out, void* stream);

/* windq_fit_refine with the salient weights taken out of the groups, as in windq_fit_eval_protected:
 * thresh fp32 [U] from windq_salient_select, clip_idx from windq_fit_eval_protected with the same thresholds.
 * With every threshold +infinity the results are those of windq_fit_refine, bit for bit.  Same scratch size. */
windq_status windq_fit_refine_protected(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                        const float* s, const float* clip_grid, int K, const uint8_t* clip_idx,
                                        const float* thresh, int n_steps, float lr, float* err_out, void* scale_out,
                                        float* group_err_out, void* stream);

/* windq_apply_plan with the refined step sizes: the scale of every 8/4/3/2-bit group is scale_in
 * (fp16 [4][U][R], device, from windq_fit_refine); its zero point is that of the clip-grid fit clip_idx
 * names (required here).  Everything else as windq_apply_plan; scales_out repeats the scales used. */
windq_status windq_apply_plan_refined(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                      const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                      const uint8_t* clip_idx, const void* scale_in, const int64_t* code_offsets,
                                      uint8_t* codes_out, void* scales_out, void* zeros_out, void* Wq_out, void* stream);

/* windq_apply_plan_protected with the refined step sizes of windq_fit_refine_protected (scale_in fp16
 * [4][U][R], device; clip_idx required).  Everything else as windq_apply_plan_protected. */
windq_status windq_apply_plan_protected_refined(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                                const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                                const uint8_t* clip_idx, const void* scale_in, const int64_t* code_offsets,
                                                const float* thresh, uint8_t* codes_out, void* scales_out, void* zeros_out,
                                                void* Wq_out, void* prot_scale_out, int64_t* prot_offsets_out,
                                                int8_t* prot_q_out, int64_t prot_q_capacity, void* stream);

/* Search over the ternary assignment (App. "Per-unit Scale Optimization" and Sec. 3.5 name fitted low-bit
 * operators -- soft assignments with a scale per group at 1.58 bit, elastic binarization at 1 bit -- without
 * formulas).  What this call does: for a fixed scale alpha the best ternary code of w_j is sign(w_j) when
 * |w_j| > alpha / 2 and 0 otherwise, whatever s_j is, so the best support is a threshold set; and for a fixed
 * support the best scale is the s-weighted mean of |w| on it.  The call tries thr_K thresholds
 *   tau_k = thr_grid[k] * mean|w|          (ratios supplied by the caller, like the clip ratios),
 * fits every one exactly as windq_fit_eval fits its single threshold 0.7 * mean|w| (support {|w| > tau_k}, scale
 * = fp16 of the s-weighted mean of |w| on it, the unweighted mean if that support carries no activation weight, 0
 * if it is empty), scores it by the s-weighted squared error and keeps the smallest k with the least error.
 * With thr_grid = {0.7} the results are the 1.58-bit column of windq_fit_eval, bit for bit.  (The 1-bit operator
 * needs no search: with levels +-alpha the code sign(w_j) is the best one for every alpha > 0, and alpha has
 * the closed form windq_fit_eval uses.)
 *   thr_grid      fp32 [thr_K] (device), 1 <= thr_K <= 64, ratios in (0, 64]
 *   thresh        fp32 [U] or NULL: salient-weight thresholds of windq_salient_select; protected weights leave the
 *                 groups as in windq_fit_eval_protected
 *   err_out       fp32 [U]      sum over rows of the best error (double accumulation)
 *   thr_idx_out   u8   [U][R]   the chosen index
 *   alpha_out     fp16 [U][R]   the scale of the chosen fit
 *   group_err_out fp32 [U][R]   nullable
 * Group-level results are bit-reproducible.  Scratch: windq_scratch_bytes_fit_ternary_search. */
int64_t windq_scratch_bytes_fit_ternary_search(int64_t R, int64_t C, int G);
windq_status windq_fit_ternary_search(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                      const float* s, const float* thr_grid, int thr_K, const float* thresh,
                                      float* err_out, uint8_t* thr_idx_out, void* alpha_out, float* group_err_out,
                                      void* stream);

/* windq_apply_plan with the thresholds that windq_fit_ternary_search chose: a 1.58-bit unit is packed with
 * tau = thr_grid[thr_idx[u][r]] * mean|w| in place of 0.7 * mean|w| (an index >= thr_K means thr_K - 1).
 * clip_idx, thr_grid and thr_idx (u8 [U][R]) are required; everything else as windq_apply_plan. */
windq_status windq_apply_plan_searched(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                       const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                       const uint8_t* clip_idx, const float* thr_grid, int thr_K, const uint8_t* thr_idx,
                                       const int64_t* code_offsets, uint8_t* codes_out, void* scales_out, void* zeros_out,
                                       void* Wq_out, void* stream);

/* The deterministic rule of the paper's heuristic allocator ("Comparison with Heuristic Sensitivity
 * Allocator": units ranked by saliency; all start at 2 bit; the least sensitive are pushed to 1.58 or
 * 1 bit to free budget; the most sensitive are promoted to 3 or 4 bit if budget permits).  The paper
 * fixes neither the order of the moves nor how much is freed; this call does the following, over the
 * U units of any number of matrices:
 *   cost(u, a) = 100 b_a (n_u - p_u) + 800 p_u + 100 g_u (scale_bits [+ zero_bits for 4/3/2 bit])   Eq. 6, centibits
 *   budget = target_cb * N,  floor = budget - headroom_cb * N,  N = sum of n_u
 *   rank: saliency descending in the total order of the binary32 bit patterns (-0 below +0), equal
 *         scores by ascending unit index
 *   1. every unit takes 2 bit; total = sum of the costs
 *   2. two sweeps from the least sensitive unit upwards, the first to 1.58 bit, the second to 1 bit: a
 *      unit moves while total > floor; the first unit met with total <= floor ends the step
 *   3. one pass from the most sensitive unit downwards over the units still at 2 bit: 4 bit if the total
 *      stays <= budget, else 3 bit if it stays <= budget, else no change
 * Arguments (device unless said otherwise):
 *   saliency fp32 [U] (e.g. windq_unit_saliency, matrix after matrix);  n_weights, n_groups i64 [U]
 *   (R G and R of the unit's matrix);  n_protected i64 [U], nullable = none (count_out of
 *   windq_salient_select);  target_cb, headroom_cb in [0, 1600] (host values)
 *   actions_out u8 [U];  order_out i64 [U], nullable: unit indices, most sensitive first;
 *   total_centibits_out i64 [1]: the final total, or -1 if a count is negative or p_u > n_u (actions
 *   are then meaningless)
 * U <= WINDQ_MAX_ALLOC_UNITS.  All arithmetic is int64: results are exact.  Scratch:
 * windq_scratch_bytes_greedy_allocate. */
#define WINDQ_MAX_ALLOC_UNITS (1 << 20)
int64_t windq_scratch_bytes_greedy_allocate(int64_t U);
windq_status windq_greedy_allocate(windq_ctx* ctx, const float* saliency, const int64_t* n_weights,
                                   const int64_t* n_protected, const int64_t* n_groups, int64_t U, int64_t target_cb,
                                   int64_t headroom_cb, int scale_bits, int zero_bits, uint8_t* actions_out,
                                   int64_t* order_out, int64_t* total_centibits_out, void* stream);

/* Fallback to higher precision (Sec. 3.5: an operator whose reconstruction error turns out too large
 * is replaced by one of higher precision).  The paper gives neither the measure nor the threshold;
 * here the error of unit u under action a is excessive when
 *   err[u][a] > theta * energy[u]     (binary32 on both sides; err and energy from windq_fit_eval)
 * and the unit moves one step at a time towards higher precision (1 -> 1.58 -> 2 -> 3 -> 4 -> 8 ->
 * skip) until the test passes; skip always passes.
 *   err fp32 [U][6], energy fp32 [U], actions u8 [U] (device); theta >= 0 (host value)
 *   actions_out u8 [U] (may be `actions` itself);  n_changed_out i64 [1], nullable
 * Action codes above 6 are copied unchanged. */
windq_status windq_fallback(windq_ctx* ctx, const float* err, const float* energy, const uint8_t* actions, int64_t U,
                            float theta, uint8_t* actions_out, int64_t* n_changed_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* WINDQ_H_ */
