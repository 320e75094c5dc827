/* libqasg - the per-iteration hot path of QCMD adagrad / QRDA adagrad on one GPU.
 *
 * Paper: "Quantized Adaptive Subgradient Algorithms and Their Applications"
 * (arXiv 2208.05631).  One iteration of its Algorithm 1, with the M workers simulated on
 * one device: every worker's fp32 gradient is quantized to ternary codes and a scale,
 * the codes are decoded and averaged (Eq. SynQ_t), the diagonal AdaGrad accumulator
 * H_t = delta*I + diag(c_t) is updated from the quantized gradient, and the closed-form
 * L1-proximal update is applied (Eq. QCMD or Eq. QRDA).  The averaged gradient is not
 * re-quantized (the one-way variant marked with a dagger in Section 5).
 *
 * Conventions for every entry point
 *   - "device pointer": memory of the context's device, owned by the caller, at least
 *     16-byte aligned unless stated, not overlapping any other argument.  "host
 *     pointer": ordinary or pinned host memory.
 *   - Calls validate their arguments on the host, enqueue their kernels on `stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream) and return without
 *     waiting.  An argument error returns a status other than QASG_OK and enqueues
 *     nothing.  Conditions found on the device (a non-finite gradient, an invalid
 *     code) are reported later by qasg_last_async_status.
 *   - One context must not be used from two streams at the same time: its workspace
 *     (per-worker statistics, partial sums, code scratch) is shared by all calls.
 *   - Step index t is 1-based.  1 <= M <= 64.  1 <= d <= 2^34.
 *   - There is no CPU implementation behind this interface.
 */
#ifndef QASG_H_
#define QASG_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qasg_ctx qasg_ctx; /* opaque; owns only its workspace */

typedef enum {
  QASG_OK = 0,
  QASG_ERR_INVALID_ARG = 1, /* NULL pointer, size or parameter out of range           */
  QASG_ERR_ALIGNMENT = 2,   /* pointer or leading dimension not aligned as required   */
  QASG_ERR_WORKSPACE = 3,   /* d or M beyond what the context was created for         */
  QASG_ERR_CUDA = 4,        /* a CUDA runtime call failed                             */
  QASG_ERR_TIMEOUT = 5,     /* (async) a bounded device-side wait ran out             */
  QASG_ERR_NONFINITE = 6,   /* (async) a gradient held NaN or Inf                     */
  QASG_ERR_BAD_CODE = 7,    /* (async) a packed code word held the unused value 3     */
  QASG_ERR_BAD_INDEX = 8    /* (async) a row or column index of sparse data out of range */
} qasg_status;

/* The quantization function Q(.) applied to each worker's gradient. */
typedef enum {
  /* Q_Delta of Section 3.4 with the threshold of Section 3.5:
   * Delta = thr_coef/d * sum|v_i|; code +1 if v > Delta, -1 if v < -Delta, 0 if
   * |v| <= Delta; scale s = mean of |v_i| over the non-zero codes.  Deterministic. */
  QASG_Q_THRESHOLD = 0,
  /* The unbiased ternary quantizer the paper compares with (Section 3.4, first
   * paragraph): scale s = max|v_i|; code sign(v_i) with probability |v_i|/s, else 0.
   * Randomness: Philox4x32-10 (Salmon et al., SC'11), key (seed lo, seed hi), counter
   * (i>>2, m, t lo, t hi), coordinate i uses output word i&3, u = (word>>8) * 2^-24,
   * non-zero iff u < |v_i|/s in fp32. */
  QASG_Q_TERNARY_STOCH = 1,
  /* No quantization: the 32-bit CMD adagrad / RDA adagrad the paper compares with
   * (Section 5.1 "Baselines"; Eq. CMD adagrad, Eq. RDA adagrad).  Accepted by qasg_step
   * and qasg_step_host only: q_t is the plain mean of the M fp32 gradients. */
  QASG_Q_NONE = 2
} qasg_quantizer;

typedef enum {
  QASG_RULE_CMD = 0, /* Eq. QCMD: soft-threshold composite mirror descent           */
  QASG_RULE_RDA = 1  /* Eq. QRDA: dual averaging with closed-form truncation        */
} qasg_rule;

typedef struct {
  uint32_t struct_size; /* sizeof(qasg_params), checked                              */
  uint32_t quantizer;   /* qasg_quantizer                                            */
  float thr_coef;       /* 0.75 in Section 3.5; > 0                                  */
  float lambda;         /* L1 coefficient, >= 0                                      */
  float eta;            /* learning rate, > 0                                        */
  float delta;          /* the delta of H_t = delta*I + diag(c_t), > 0               */
  uint64_t seed;        /* Philox key (stochastic quantizer only)                    */
} qasg_params;

/* Flags of qasg_create. */
#define QASG_CREATE_NO_CODE_SCRATCH 1u /* qasg_step will always be given codes_out   */
/* By default the kernels of a step are launched as programmatic dependents of one another: a
 * kernel's CTAs are placed, and in pass B request their first gradient tile, while the kernel
 * before it drains; each waits for that kernel's completion before it touches what it wrote.
 * With this flag every kernel starts only after the one before it has completed.  Same bits. */
#define QASG_CREATE_SERIAL_LAUNCHES 2u

/* Creates a context on CUDA device `device` able to serve calls with d <= d_max and
 * M <= M_max.  Allocates the whole workspace here (a few hundred KB of statistics, and,
 * unless QASG_CREATE_NO_CODE_SCRATCH, (M_max + 1) * qasg_code_words(d_max) * 4 bytes of code
 * scratch and 4 * d_max bytes for the averaged gradient of the double-quantized step); no
 * other call allocates device memory.  On error *out is NULL. */
qasg_status qasg_create(qasg_ctx** out, int device, uint64_t d_max, uint32_t M_max,
                        uint32_t flags);
/* Frees the workspace.  The caller must have synchronized the streams it used. */
qasg_status qasg_destroy(qasg_ctx* ctx);

/* Options of a context (qasg_set_option).
 *
 * qasg_quantize_pack and qasg_step read every gradient row twice: once for the threshold of
 * Section 3.5 (a sum over the whole row), once to cut the codes; by default in two launches (all
 * sums, then all codes).
 *
 * QASG_OPT_STREAM_ROW_BYTES > 0 selects, for rows of at most that many bytes (4*d), ONE cooperative
 * launch that codes a row QASG_OPT_STREAM_LAG rows after it was summed, while the row is still in L2:
 * the gradients then cross device memory once.  Its CTAs wait for one another through words in the
 * context's workspace, every wait bounded by QASG_OPT_WAIT_POLLS polls (about 0.2 us each), after
 * which the call gives up and qasg_last_async_status reports QASG_ERR_TIMEOUT (the outputs of that
 * call are then incomplete, and further calls do nothing until the status has been read).  It is off
 * by default: on a B200 it moves half the bytes but measured slower than the two launches.
 *
 * QASG_OPT_ONE_LAUNCH_STEP_BYTES: qasg_step on at most that many bytes of gradients (4*d*M) runs its
 * three passes as the phases of ONE launch (cooperative when it has more than one CTA) whose CTAs meet
 * twice, with the same bounded waits and the same time-out behaviour: at such sizes a launch costs
 * more than a pass (measured on a B200: 5 to 20 % faster up to 8 MB, level to 32 MB, slower beyond).
 *
 * Every setting gives the same bits. */
typedef enum {
  QASG_OPT_STREAM_ROW_BYTES = 0,     /* 0 = never (default)                                          */
  QASG_OPT_STREAM_LAG = 1,           /* 0, 1, 2, ...; 0xFFFFFFFF = chosen from the row size (default) */
  QASG_OPT_WAIT_POLLS = 2,           /* 1 .. 2^31; default 2^22 (about a second)                      */
  QASG_OPT_ONE_LAUNCH_STEP_BYTES = 3 /* 0 = never; default 16 MiB (faster or level there on a B200)   */
} qasg_option;
qasg_status qasg_set_option(qasg_ctx* ctx, qasg_option option, uint64_t value);

/* Runs the bounded device-side wait on a word that nothing sets, with a bound of max_polls polls:
 * the kernel returns by itself and the next qasg_last_async_status reports QASG_ERR_TIMEOUT.  This
 * is how the give-up path of the waits is exercised without hanging anything. */
qasg_status qasg_wait_selftest(qasg_ctx* ctx, uint32_t max_polls, void* stream);

/* Number of 32-bit code words one worker's d codes occupy: ceil(d/16)
 * (Section 3.5 "Encode": 2 bits per coordinate). */
uint64_t qasg_code_words(uint64_t d);

/* Workers' side of Algorithm 1 ("Quantize ... the gradients", with the selection S
 * keeping every coordinate): quantizes each of the M gradients and packs the codes.
 *   g          device, fp32 [M][ld_g] row-major, row m = gradient of worker m; ld_g >= d,
 *              ld_g a multiple of 4 (so every row is 16-byte aligned).
 *   codes      device, uint32 [M][qasg_code_words(d)]; coordinate i of worker m is in
 *              word i>>4 at bits 2*(i&15), 2*(i&15)+1: 0 -> 0, 1 -> +1, 2 -> -1; unused
 *              tail bits are written as 0.
 *   scales     device, fp32 [M]: s_m.
 *   thresholds device, fp32 [M] or NULL: Delta_m (0 for the stochastic quantizer).
 *   counts     device, uint64 [M] or NULL: number of non-zero codes of worker m.
 * Delta_m and s_m come from sums taken in a fixed order (4096-coordinate tiles, fp64,
 * pairwise), so they do not depend on the launch shape. */
qasg_status qasg_quantize_pack(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g,
                               uint32_t M, uint64_t t, const qasg_params* params,
                               uint32_t* codes, float* scales, float* thresholds,
                               uint64_t* counts, void* stream);

/* Server's side of Algorithm 1 ("Decode", "Average the quantized gradients",
 * Eq. SynQ_t): gbar_i = (1/M) * sum_m scales[m] * code_{m,i}.
 *   codes, scales  device, as written by qasg_quantize_pack.
 *   gbar           device, fp32 [d]. */
qasg_status qasg_decode_average(qasg_ctx* ctx, const uint32_t* codes, const float* scales,
                                uint64_t d, uint32_t M, float* gbar, void* stream);

/* Workers' update of Algorithm 1 for QCMD adagrad (Eq. H_t, Eq. QCMD), from a dense
 * quantized gradient q (device, fp32 [d]):
 *   h_i += q_i^2;  H = delta + sqrt(h_i);  u = x_i - (eta/H) q_i;
 *   x_i = sign(u) * max(|u| - lambda*eta/H, 0), zeros written as +0.0.
 *   x, h  device, fp32 [d], updated in place (h holds the sum of squares, not its root). */
qasg_status qasg_cmd_step(qasg_ctx* ctx, const float* q, float* x, float* h, uint64_t d,
                          uint64_t t, const qasg_params* params, void* stream);

/* Same for QRDA adagrad (Eq. H_t, Eq. QRDA):
 *   h_i += q_i^2;  z_i += q_i;  H = delta + sqrt(h_i);
 *   x_i = -sign(z_i) * (t*eta/H) * max(|z_i|/t - lambda, 0), zeros written as +0.0.
 *   x is written only (its old value is not read); h, z updated in place. */
qasg_status qasg_rda_step(qasg_ctx* ctx, const float* q, float* x, float* h, float* z,
                          uint64_t d, uint64_t t, const qasg_params* params, void* stream);

/* The whole iteration, fused: quantize_pack, then decode + average + accumulator +
 * update in one pass that keeps the averaged gradient in registers, so that per
 * coordinate the M gradients are read twice (threshold statistics, then codes), the
 * M/4 code bytes are written and read once, and h, x (z) cross memory once.
 *   rule        QASG_RULE_CMD (z may be NULL) or QASG_RULE_RDA (z required).
 *   codes_out   device uint32 [M][code_words(d)] or NULL to use the context's scratch.
 *   scales_out  device fp32 [M] or NULL.
 * With params->quantizer = QASG_Q_NONE nothing is quantized: one pass reads the M gradients
 * of a coordinate once, sums them in fp64 in worker order, q_i = fp32(sum * (1/M)), and applies
 * the same accumulator and update (4M + 16 or 20 bytes per coordinate); codes_out and
 * scales_out are not touched, thr_coef and seed are not used.  A non-finite mean is reported
 * as QASG_ERR_NONFINITE and still enters the state, as it would in plain AdaGrad.
 * Three launches (sums, codes, decode + update), or one launch with the same three phases for up to
 * QASG_OPT_ONE_LAUNCH_STEP_BYTES of gradients; the results have the same bits either way. */
qasg_status qasg_step(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g,
                      uint32_t M, uint64_t t, const qasg_params* params, float* x, float* h,
                      float* z, uint32_t* codes_out, float* scales_out, void* stream);

/* Server's side of Algorithm 1 with double quantization ("Quantize the aggregated gradient",
 * Eq. q_t = Q(SynQ_t)): decodes and averages the workers' codes as qasg_decode_average does, rounds
 * the average to fp32, and applies the same Q to it as to a worker's gradient, without ever
 * storing the average.
 *   codes, scales  device, the workers' messages as written by qasg_quantize_pack.
 *   qcodes         device, uint32 [qasg_code_words(d)]: the codes of q_t, same layout as one worker row.
 *   qscale         device, fp32 [1]: the scale of q_t.
 *   qthreshold     device, fp32 [1] or NULL: its threshold (0 for the stochastic quantizer).
 *   qcount         device, uint64 [1] or NULL: its number of non-zero codes.
 * The stochastic quantizer draws from the Philox stream with counter word 1 = 1<<16 (a stream of
 * its own: the workers use 0 .. M-1 there).  The workers then recover q_t with
 * qasg_decode_average(qcodes, qscale, d, 1, ...) and update with qasg_cmd_step / qasg_rda_step. */
qasg_status qasg_requantize(qasg_ctx* ctx, const uint32_t* codes, const float* scales, uint64_t d,
                            uint32_t M, uint64_t t, const qasg_params* params, uint32_t* qcodes,
                            float* qscale, float* qthreshold, uint64_t* qcount, void* stream);

/* The whole iteration of Algorithm 1 as printed, with both quantizations: qasg_quantize_pack,
 * qasg_requantize, then decode of q_t + accumulator + update in one pass.  Arguments as for
 * qasg_step, plus
 *   qcodes_out  device uint32 [code_words(d)] or NULL to use the context's scratch.
 *   qscale_out  device fp32 [1] or NULL. */
qasg_status qasg_step_double(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g,
                             uint32_t M, uint64_t t, const qasg_params* params, float* x, float* h,
                             float* z, uint32_t* codes_out, float* scales_out, uint32_t* qcodes_out,
                             float* qscale_out, void* stream);

/* Workers' side of Algorithm 1 with the sparse selection of Section 3.2: "Compute the indicator
 * function", "Quantize the selected elements of the gradients" Q(S(g, I)).
 * Worker m's indicator marks coordinate i when x_i != 0 or when the worker's local trial update,
 * taken with its own full-precision gradient and H_hat = delta + sqrt(h + g^2), leaves it non-zero.
 * Where x_i != 0 the bit is set whatever the trial gives; where x_i = 0 the closed form of the
 * trial update is non-zero iff (fp32, every operation rounded on its own)
 *   QCMD: |g| > lambda   (H_hat > 0 scales both sides and drops out)      QRDA: |z + g| > lambda*t
 * Only marked coordinates are quantized: Delta_m = thr_coef/k_m * sum over them of |g| (k_m of
 * them), the scale is the mean kept magnitude (stochastic quantizer: the maximum over them);
 * unmarked coordinates code 0.
 *   x, h, z     device, fp32 [d]: the current state (read only).  z is read by QRDA only and may
 *               be NULL for QCMD; h is read by neither test and may be NULL.
 *   indicators  device, uint32 [M][ceil(d/32)]: bit i&31 of word i>>5 of row m; unused bits 0.
 *   selected    device, uint64 [M] or NULL: k_m.  A worker's message is then 32 + d + 2*k_m bits
 *               (Section 3.5 "Encode").
 *   other arguments as for qasg_quantize_pack.
 * The comparisons are "greater or unordered": a NaN component (QRDA: a NaN z + g) is marked like an
 * infinite one, enters the sums and is reported as QASG_ERR_NONFINITE; outputs are then unspecified. */
qasg_status qasg_select_quantize_pack(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d,
                                      uint64_t ld_g, uint32_t M, uint64_t t, const qasg_params* params,
                                      const float* x, const float* h, const float* z, uint32_t* codes,
                                      float* scales, float* thresholds, uint64_t* counts,
                                      uint32_t* indicators, uint64_t* selected, void* stream);

/* Server's side: "Compute the synchronous indicator", the bitwise OR of the M indicators.
 *   isyn  device, uint32 [ceil(d/32)].   ksyn  device, uint64 [1]: its number of set bits. */
qasg_status qasg_indicator_or(qasg_ctx* ctx, const uint32_t* indicators, uint64_t d, uint32_t M,
                              uint32_t* isyn, uint64_t* ksyn, void* stream);

/* The whole iteration with sparse selection, fused like qasg_step (double_quant = 0) or like
 * qasg_step_double (double_quant != 0: the server quantizes the average over the coordinates of
 * the synchronous indicator only, Delta' = thr_coef/k_syn * sum|avg|).
 *   indicators_out, selected_out, isyn_out, ksyn_out   device, as above, each may be NULL
 *   (NULL indicators use the context's scratch).  Other arguments as for qasg_step. */
qasg_status qasg_step_select(qasg_ctx* ctx, qasg_rule rule, int double_quant, const float* g, uint64_t d,
                             uint64_t ld_g, uint32_t M, uint64_t t, const qasg_params* params, float* x,
                             float* h, float* z, uint32_t* codes_out, float* scales_out,
                             uint32_t* indicators_out, uint64_t* selected_out, uint32_t* isyn_out,
                             uint64_t* ksyn_out, void* stream);

/* qasg_step for callers whose data lives in host memory.  Copies g (M rows of d floats,
 * row stride ld_g) and the state from the host buffers into the caller's device staging
 * buffers, runs qasg_step there, and copies the new state back, all on `stream`; returns
 * without waiting (synchronize the stream before reading the host buffers).
 *   g_host, x_host, h_host, z_host   host pointers (pinned memory for asynchronous
 *                                    copies); z_host NULL for QASG_RULE_CMD.  For
 *                                    QASG_RULE_RDA x_host is output only.
 *   g_dev [M][ld_g], x_dev, h_dev, z_dev [d]   device staging, as for qasg_step. */
qasg_status qasg_step_host(qasg_ctx* ctx, qasg_rule rule, const float* g_host, uint64_t d,
                           uint64_t ld_g, uint32_t M, uint64_t t, const qasg_params* params,
                           float* x_host, float* h_host, float* z_host, float* g_dev,
                           float* x_dev, float* h_dev, float* z_dev, void* stream);

/* Per-worker minibatch gradient of logistic regression, the linear-model workload of
 * Section 5.1 (Eq. of Section 3.1: the minibatch average of per-sample gradients):
 *   g_m = (1/B) sum_{j in batch m} -y_j * sigmoid(-y_j <a_j, x>) * a_j ,  y_j in {-1,+1}.
 * The L1 term is left to the proximal update.
 *   X          device, fp32 [n_rows][d] row-major, d a multiple of 4.
 *   y          device, fp32 [n_rows].
 *   shard_row0 host, uint64 [M+1]: worker m owns rows [shard_row0[m], shard_row0[m+1]).
 *   batch_rows device, uint32 [M][B] global row ids, or NULL for the default minibatch:
 *              B consecutive rows of the shard starting at ((t-1)*B) mod shard size,
 *              wrapping inside the shard.
 *   x          device, fp32 [d].
 *   g          device, fp32 [M][ld_g], rows fully overwritten (first d entries). */
qasg_status qasg_logreg_grad_dense(qasg_ctx* ctx, const float* X, const float* y,
                                   uint64_t n_rows, uint64_t d, uint32_t M,
                                   const uint64_t* shard_row0, const uint32_t* batch_rows,
                                   uint32_t B, uint64_t t, const float* x, float* g,
                                   uint64_t ld_g, void* stream);

/* Same for a CSR matrix: rowptr device int64 [n_rows+1] (rowptr[n_rows] = nnz), colidx device
 * int32 [nnz] (0 <= colidx < d), vals device fp32 [nnz].  g rows are zeroed, then accumulated
 * with atomic adds: the summation order inside one coordinate is not fixed, so the last bits of
 * g, and with them the codes of coordinates that sit within rounding of Delta_m, can differ from
 * run to run.  The indices are checked on the device: a minibatch row id >= n_rows, a row whose
 * rowptr pair is not 0 <= lo <= hi <= rowptr[n_rows], or an entry with a column outside [0, d)
 * is skipped (it adds nothing and no memory outside the arguments is touched) and
 * qasg_last_async_status reports QASG_ERR_BAD_INDEX.  The dense entry point checks batch_rows
 * the same way. */
qasg_status qasg_logreg_grad_csr(qasg_ctx* ctx, const int64_t* rowptr, const int32_t* colidx,
                                 const float* vals, const float* y, uint64_t n_rows,
                                 uint64_t d, uint32_t M, const uint64_t* shard_row0,
                                 const uint32_t* batch_rows, uint32_t B, uint64_t t,
                                 const float* x, float* g, uint64_t ld_g, void* stream);

/* Gradients held in sparse form (the text data sets of Section 5.1, Table 1, have a few dozen
 * non-zeros per row, so a minibatch gradient touches a small part of the d coordinates, and "a zero
 * entry lies inside [-Delta, Delta] and codes 0", Section 3.4).  The rows of g keep their dense
 * layout [M][ld_g], but only the entries marked in
 *   touched   device, uint32 [M][ceil(d/32)], 16-byte aligned: bit i&31 of word i>>5 of row m; bits at
 *             or past d are ignored
 * are stored: every other entry IS +0.0, its memory is never read and may hold anything.  Results are
 * bit for bit those of the dense entry points on the row with +0.0 in the unmarked places (Delta_m
 * still divides by the full d); the memory traffic shrinks to the touched sectors plus d/8 bytes of
 * bits per worker.
 *
 * qasg_logreg_grad_csr_touched: the CSR gradient in this form.  g and touched carry state from call
 * to call: on entry the bits must mark every entry of g[.., 0..d) that is not +0.0 (before the first
 * call: g and touched all zero, once).  The call zeroes the marked entries and the bits, then
 * accumulates the minibatch with atomic adds and sets the bit of every entry it adds to (a touched
 * entry may still sum to 0).  Nothing else of g is written or read. */
qasg_status qasg_logreg_grad_csr_touched(qasg_ctx* ctx, const int64_t* rowptr, const int32_t* colidx,
                                         const float* vals, const float* y, uint64_t n_rows,
                                         uint64_t d, uint32_t M, const uint64_t* shard_row0,
                                         const uint32_t* batch_rows, uint32_t B, uint64_t t,
                                         const float* x, float* g, uint64_t ld_g, uint32_t* touched,
                                         void* stream);

/* qasg_quantize_pack and qasg_step on gradients held in sparse form (see above).  Arguments as
 * for the dense entry points, plus touched (read only). */
qasg_status qasg_quantize_pack_touched(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g,
                                       uint32_t M, uint64_t t, const qasg_params* params,
                                       const uint32_t* touched, uint32_t* codes, float* scales,
                                       float* thresholds, uint64_t* counts, void* stream);
qasg_status qasg_step_touched(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g,
                              uint32_t M, uint64_t t, const qasg_params* params, const uint32_t* touched,
                              float* x, float* h, float* z, uint32_t* codes_out, float* scales_out,
                              void* stream);

/* The threshold quantizer at the exact optimal threshold of Section 3.4 instead of the 0.75 * mean|g|
 * rule of Section 3.5: per worker, the magnitudes are ranked (radix sort), every component is taken as
 * the candidate threshold, and the one that maximises (sum_{I_Delta} |g_i|)^2 / |I_Delta| is kept
 * (candidates are the strict drops of the ranked magnitudes, equal maxima resolve to the smaller set,
 * Delta* is the largest component outside the chosen set, 0 if everything non-zero is kept).  Codes,
 * scales (mean kept magnitude) and counts (|I_Delta*|) then as for qasg_quantize_pack.  O(d log d) work
 * and 12 passes over the row: an accuracy reference for the rule, not a per-step path.
 *   params        quantizer must be QASG_Q_THRESHOLD; thr_coef is not used.
 *   scratch       device, 256-byte aligned, at least qasg_optimal_scratch_bytes(d) bytes (about 8.3 d),
 *                 used for one worker after the other; contents undefined afterwards.
 *   d             below 2^31 (qasg_optimal_scratch_bytes returns 0 beyond).
 * Non-finite gradients: status NONFINITE, outputs unspecified. */
uint64_t qasg_optimal_scratch_bytes(uint64_t d);
qasg_status qasg_quantize_pack_optimal(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                                       const qasg_params* params, uint32_t* codes, float* scales,
                                       float* thresholds, uint64_t* counts, void* scratch,
                                       uint64_t scratch_bytes, void* stream);

/* The threshold quantizer of qasg_quantize_pack for callers that cannot allocate device
 * memory.  (The paper has no counterpart: this entry point exists for the sake of its
 * callers, not of the method.)
 *
 * Some code that wants to quantize gradients runs where cudaMalloc is off limits: inside a
 * framework that has already handed all device memory to its own pool, so that a raw
 * allocation fails or fragments it; or inside a latency-critical loop that cannot accept the
 * device-wide synchronisation an allocation implies.  Such callers cannot create a qasg_ctx,
 * whose workspace is allocated in qasg_create.  This call needs no context and allocates
 * nothing, on the host or on the device: its scratch (per-chunk partial sums and counts,
 * per-worker statistics, a completion counter) is a fixed array of
 * QASG_STATIC_SCRATCH_BYTES bytes built into the library, which every GPU that loads the
 * library holds until the process exits.
 *
 *   device      CUDA device ordinal (0 <= device < 64); made current by the call.
 *   g, d, ld_g, codes, scales, thresholds, counts, stream   as for qasg_quantize_pack;
 *               the quantizer is QASG_Q_THRESHOLD with coefficient thr_coef (0.75 in
 *               Section 3.5).  Results are bit-identical to qasg_quantize_pack's.
 *   M           1 <= M <= QASG_STATIC_MAX_WORKERS; more workers than the scratch holds is
 *               refused with QASG_ERR_WORKSPACE and nothing is enqueued.  d may be as large
 *               as for any other call (1 <= d <= 2^34): the scratch does not grow with d.
 *
 * The first call on a device looks up the device address of the built-in array; make that
 * first call before any stream capture begins.  All calls on a device share the one array
 * and it keeps the previous call's contents: each call clears the counter it needs at zero
 * on `stream` before its kernels, so calls issued one after another on one stream are safe,
 * but two calls that may overlap on the GPU (different streams, no dependency between them)
 * race on the array and give undefined results.  A non-finite gradient gives all-zero codes
 * and a zero scale for that worker, as in qasg_quantize_pack, but is not reported. */
#define QASG_STATIC_MAX_WORKERS 16u
#define QASG_STATIC_SCRATCH_BYTES (336u * 1024u)
qasg_status qasg_quantize_pack_static(int device, const float* g, uint64_t d, uint64_t ld_g,
                                      uint32_t M, float thr_coef, uint32_t* codes, float* scales,
                                      float* thresholds, uint64_t* counts, void* stream);

/* Waits for `stream`, then returns and clears the conditions kernels recorded since
 * the last call: QASG_ERR_TIMEOUT, QASG_ERR_NONFINITE, QASG_ERR_BAD_CODE, QASG_ERR_BAD_INDEX,
 * QASG_ERR_CUDA, else QASG_OK (the first of these that applies). */
qasg_status qasg_last_async_status(qasg_ctx* ctx, void* stream);

/* Number of kernels this context has launched since it was created. */
uint64_t qasg_launch_count(const qasg_ctx* ctx);

/* Per-kernel device timing, for benchmarks.  Between qasg_profile_begin and
 * qasg_profile_end every kernel the context launches is bracketed by a pair of CUDA events
 * recorded on the stream it is launched on.  qasg_profile_end waits for those events and
 * adds up, per kernel id (0 <= id < QASG_KERNEL_COUNT, names from qasg_kernel_name), the
 * elapsed milliseconds into ms[id] and the number of launches into launches[id] (both host
 * arrays of QASG_KERNEL_COUNT entries), then stops recording. */
#define QASG_KERNEL_COUNT 26
qasg_status qasg_profile_begin(qasg_ctx* ctx);
qasg_status qasg_profile_end(qasg_ctx* ctx, double* ms, uint64_t* launches);
const char* qasg_kernel_name(int id);

const char* qasg_status_string(qasg_status s);

#ifdef __cplusplus
}
#endif
#endif /* QASG_H_ */
