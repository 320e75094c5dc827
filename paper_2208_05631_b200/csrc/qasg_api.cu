// C-ABI layer of libqasg: context, argument validation, sequencing of the passes.
#include "../../include/qasg.h"

#include <new>
#include <vector>

#include "qasg_internal.h"

using namespace qasg;

struct qasg_ctx {
  int device;
  uint64_t d_max;
  uint32_t M_max;
  LaunchShape shape;
  Workspace ws;
  Workspace wsq;            // server row (the re-quantized average): kRowChunks partial slots, 1 statistic
  Workspace wss;            // selection statistics, pass B of the one-launch step: [M_max][kRowChunks] partial slots, the statistics of ws
  uint32_t* code_scratch;   // [M_max][code_words(d_max)] or NULL
  uint32_t* qcode_scratch;  // [code_words(d_max)] or NULL
  float* gbar_scratch;      // [d_max rounded up to 4] or NULL: the averaged gradient of the server row
  uint32_t* ind_scratch;    // [M_max + 1][ceil(d_max/32)] or NULL: workers' indicators, then their OR
  unsigned long long* ksyn; // [1] number of bits of the synchronous indicator
  float* logreg_ws;         // kLogregEntries coefficients followed by as many row ids
  StreamSync* sync;         // words the CTAs of the one-launch quantizer wait on
  StreamSlots slots;        // and the slots their chunk partials travel through
  uint64_t stream_row_bytes;  // rows up to this size are quantized by the one-launch kernel (0: never)
  uint32_t stream_lag;      // kAutoLag: chosen from the row size
  uint32_t wait_polls;
  uint64_t launches;
  uint64_t one_launch_step_bytes;  // qasg_step runs as one launch up to this many bytes of gradients
  bool cooperative;                // the device can run cooperative launches (else the one-launch paths stay off)
  bool ticket_dirty;        // a launch failed since the completion counter was last known to be zero
  bool profiling;
  std::vector<cudaEvent_t> events;  // pairs (start, stop), reused between profiles
  std::vector<int> event_kernel;    // kernel id of each recorded pair
};

namespace {

enum KernelId {
  kAbsSum = 0, kAbsMax, kThresholdCodes, kStochasticCodes, kDecodeUpdateCmd, kDecodeUpdateRda,
  kDecodeAverage, kDenseUpdateCmd, kDenseUpdateRda, kLogregDense, kLogregCsr, kAvgAbsSum, kAvgAbsMax,
  kAvgThresholdCodes, kAvgStochasticCodes, kSelectStats, kIndicatorOr, kTouchedClear, kLogregCsrTouched,
  kOptimalThreshold, kMeanUpdateCmd, kMeanUpdateRda, kStreamThreshold, kStreamStochastic, kFusedStepCmd,
  kFusedStepRda, kKernelIdCount
};
static_assert(kKernelIdCount <= QASG_KERNEL_COUNT, "kernel id table");

// Counts the launches of one launcher call and, while profiling, brackets them with events.
struct Launch {
  qasg_ctx* ctx;
  cudaStream_t stream;
  bool timed;
  size_t slot;
  Launch(qasg_ctx* c, int kernel, cudaStream_t s) : ctx(c), stream(s), timed(c->profiling), slot(0) {
    if (!timed) return;
    slot = ctx->event_kernel.size();
    while (ctx->events.size() < 2 * (slot + 1)) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreate(&e) != cudaSuccess) {
        timed = false;
        return;
      }
      ctx->events.push_back(e);
    }
    ctx->event_kernel.push_back(kernel);
    cudaEventRecord(ctx->events[2 * slot], stream);
  }
  void operator+=(int n) { ctx->launches += n; }
  ~Launch() {
    if (timed) cudaEventRecord(ctx->events[2 * slot + 1], stream);
  }
};

constexpr uint64_t kMaxD = 1ull << 34;
constexpr uint32_t kAutoLag = 0xFFFFFFFFu;
constexpr uint64_t kDefaultStreamRowBytes = 0;         // the one-launch kernel is opt-in
// Up to 16 MB of gradients the one-launch step measured faster than three chained launches or level with them
// (single cold steps: 5 to 20 % up to 2^18 coordinates x 32 workers, level at 2^20 x 2 and 2^20 x 8; replayed
// from a graph d = 10,000, M = 4: 9.6 against 11.9 us); beyond that its two meetings cost more than two launches.
constexpr uint64_t kDefaultOneLaunchStepBytes = 16ull << 20;
// A row is coded `lag` rows after it was summed; in between the rows summed and coded meanwhile pass
// through L2.  One row of lag hides the wait for a worker's threshold; it is taken while three rows fit.
constexpr uint64_t kLagOneRowBytes = 24ull << 20;
// Code rows small enough to stay in L2 until pass C reads them are written with ordinary stores.
constexpr uint64_t kKeepCodesBytes = 32ull << 20;
constexpr uint64_t kLogregEntries = 1ull << 20;  // M * B of one gradient call

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

qasg_status check_params_update(const qasg_params* p) {
  if (!(p->lambda >= 0.f) || !isfinite(p->lambda)) return QASG_ERR_INVALID_ARG;
  if (!(p->eta > 0.f) || !isfinite(p->eta)) return QASG_ERR_INVALID_ARG;
  if (!(p->delta > 0.f) || !isfinite(p->delta)) return QASG_ERR_INVALID_ARG;
  return QASG_OK;
}

qasg_status check_params(const qasg_params* p, bool need_update, bool allow_none = false) {
  if (!p || p->struct_size != sizeof(qasg_params)) return QASG_ERR_INVALID_ARG;
  if (p->quantizer == QASG_Q_NONE) return allow_none && need_update ? check_params_update(p) : QASG_ERR_INVALID_ARG;
  if (p->quantizer != QASG_Q_THRESHOLD && p->quantizer != QASG_Q_TERNARY_STOCH) return QASG_ERR_INVALID_ARG;
  if (!(p->thr_coef > 0.f) || !isfinite(p->thr_coef)) return QASG_ERR_INVALID_ARG;
  return need_update ? check_params_update(p) : QASG_OK;
}

qasg_status check_shape(const qasg_ctx* ctx, uint64_t d, uint32_t M) {
  if (!ctx) return QASG_ERR_INVALID_ARG;
  if (d < 1 || d > kMaxD || M < 1 || M > static_cast<uint32_t>(kMaxWorkers)) return QASG_ERR_INVALID_ARG;
  if (d > ctx->d_max || M > ctx->M_max) return QASG_ERR_WORKSPACE;
  return QASG_OK;
}

qasg_status enter(const qasg_ctx* ctx) {
  return cudaSetDevice(ctx->device) == cudaSuccess ? QASG_OK : QASG_ERR_CUDA;
}

// A launch that failed may have left the grid-completion counter of the reduction kernels non-zero (its
// last CTA puts it back to zero): the next call that uses it clears it first.
qasg_status leave(qasg_ctx* ctx) {
  if (cudaGetLastError() == cudaSuccess) return QASG_OK;
  ctx->ticket_dirty = true;
  return QASG_ERR_CUDA;
}

void clear_ticket_if_dirty(qasg_ctx* ctx, cudaStream_t stream) {
  if (!ctx->ticket_dirty) return;
  cudaMemsetAsync(ctx->ws.ticket, 0, sizeof(unsigned int), stream);
  ctx->ticket_dirty = false;
}

// About four rounds of resident CTAs: enough items to balance the launch.
uint32_t target_items(const qasg_ctx* ctx) {
  return static_cast<uint32_t>(ctx->shape.sm_count * ctx->shape.reduce_ctas_per_sm * 4);
}

StepScalars scalars(const qasg_params* p, uint64_t t) {
  StepScalars sc;
  sc.lambda = p->lambda;
  sc.eta = p->eta;
  sc.delta = p->delta;
  sc.t = static_cast<float>(t);
  sc.inv_t = 1.0f / sc.t;
  return sc;
}

// Passes A and B on validated arguments.
void quantize_pack(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g, uint32_t M, uint64_t t,
                   const qasg_params* p, uint32_t* codes, float* scales, float* thresholds,
                   uint64_t* counts, cudaStream_t stream, const uint32_t* touched = nullptr) {
  const Geometry geo = make_geometry(d, ld_g, M, kMaxChunks, target_items(ctx));
  unsigned long long* counts_out = reinterpret_cast<unsigned long long*>(counts);
  clear_ticket_if_dirty(ctx, stream);
  if (touched) {  // rows held in sparse form: one warp per tile
    const bool stochastic = p->quantizer != QASG_Q_THRESHOLD;
    if (!stochastic) {
      Launch l(ctx, kAbsSum, stream);
      l += launch_touched_abs_sum(g, geo, p->thr_coef, ctx->ws, thresholds, touched, ctx->shape, stream);
    } else {
      Launch l(ctx, kAbsMax, stream);
      l += launch_touched_abs_max(g, geo, ctx->ws, touched, ctx->shape, stream);
    }
    {
      Launch l(ctx, stochastic ? kStochasticCodes : kThresholdCodes, stream);
      l += launch_touched_codes(stochastic, g, geo, p->seed, t, ctx->ws, codes, scales, counts_out, touched, ctx->shape,
                                stream);
    }
    if (stochastic && thresholds) cudaMemsetAsync(thresholds, 0, M * sizeof(float), stream);
    return;
  }
  // One launch, each row coded out of L2: items of a worker's row are dealt to the resident CTAs one row
  // after the other, so a row is cut into about as many chunks as there are CTAs.
  const Geometry sgeo = make_geometry(d, ld_g, M, static_cast<uint32_t>(ctx->shape.sm_count * ctx->shape.reduce_ctas_per_sm));
  if (ctx->cooperative && d * sizeof(float) <= ctx->stream_row_bytes && sgeo.group <= kStreamMaxGroup) {
    const bool stochastic = p->quantizer != QASG_Q_THRESHOLD;
    StreamParams sp;
    sp.coef = p->thr_coef;
    sp.lag = ctx->stream_lag != kAutoLag ? ctx->stream_lag : (d * sizeof(float) <= kLagOneRowBytes ? 1u : 0u);
    if (sp.lag > M) sp.lag = M;
    sp.max_polls = ctx->wait_polls;
    sp.stream_base = 0u;
    sp.seed = p->seed;
    sp.t = t;
    const bool keep_codes = static_cast<uint64_t>(M) * qasg_code_words(d) * 4 <= kKeepCodesBytes;
    Launch l(ctx, stochastic ? kStreamStochastic : kStreamThreshold, stream);
    l += launch_quantize_stream(stochastic, keep_codes, g, sgeo, sp, ctx->ws, ctx->slots, ctx->sync, codes, scales, thresholds,
                                counts_out, ctx->shape, stream);
    return;
  }
  if (p->quantizer == QASG_Q_THRESHOLD) {
    { Launch l(ctx, kAbsSum, stream); l += launch_abs_sum(g, geo, p->thr_coef, ctx->ws, thresholds, ctx->shape, stream); }
    { Launch l(ctx, kThresholdCodes, stream); l += launch_threshold_codes(g, geo, ctx->ws, codes, scales, counts_out, ctx->shape, stream); }
  } else {
    { Launch l(ctx, kAbsMax, stream); l += launch_abs_max(g, geo, ctx->ws, ctx->shape, stream); }
    { Launch l(ctx, kStochasticCodes, stream); l += launch_stochastic_codes(g, geo, p->seed, t, 0u, ctx->ws, codes, scales, counts_out,
                                             ctx->shape, stream); }
    if (thresholds) cudaMemsetAsync(thresholds, 0, M * sizeof(float), stream);
  }
}

// Server row on validated arguments: q = Q(average of the decoded workers).
// With scratch, the average is written once as an fp32 row (fast per-lane-table decode) and the
// workers' own two quantization kernels run on that row; without, two kernels rebuild the average
// from the code bytes and nothing is stored.  Both give the same bits.
// denom (device, [1]): number of coordinates of the synchronous indicator when Q runs over those only.
void requantize(qasg_ctx* ctx, const uint32_t* codes, const float* scales, uint64_t d, uint32_t M, uint64_t t,
                const qasg_params* p, uint32_t* qcodes, float* qscale, float* qthreshold, uint64_t* qcount,
                cudaStream_t stream, const unsigned long long* denom = nullptr) {
  const bool stochastic = p->quantizer == QASG_Q_TERNARY_STOCH;
  unsigned long long* count_out = reinterpret_cast<unsigned long long*>(qcount);
  clear_ticket_if_dirty(ctx, stream);
  if (ctx->gbar_scratch) {
    float* gbar = ctx->gbar_scratch;
    const uint64_t ld = ((d + 3) / 4) * 4;
    {
      Launch l(ctx, kDecodeAverage, stream);
      l += launch_decode_average(codes, scales, d, M, gbar, ctx->ws.status, ctx->shape, stream);
    }
    const Geometry row = make_geometry(d, ld, 1, kMaxChunks, target_items(ctx));
    if (!stochastic) {
      { Launch l(ctx, kAbsSum, stream); l += launch_abs_sum(gbar, row, p->thr_coef, ctx->wsq, qthreshold, ctx->shape, stream, denom); }
      { Launch l(ctx, kThresholdCodes, stream); l += launch_threshold_codes(gbar, row, ctx->wsq, qcodes, qscale, count_out, ctx->shape, stream); }
    } else {
      { Launch l(ctx, kAbsMax, stream); l += launch_abs_max(gbar, row, ctx->wsq, ctx->shape, stream); }
      { Launch l(ctx, kStochasticCodes, stream); l += launch_stochastic_codes(gbar, row, p->seed, t, 1u << 16, ctx->wsq, qcodes, qscale, count_out, ctx->shape, stream); }
    }
  } else {
    const Geometry row = make_geometry(d, d, 1, kRowChunks);
    {
      Launch l(ctx, stochastic ? kAvgAbsMax : kAvgAbsSum, stream);
      l += launch_avg_stats(stochastic, codes, scales, M, row, p->thr_coef, ctx->wsq, qthreshold, ctx->shape, stream, denom);
    }
    {
      Launch l(ctx, stochastic ? kAvgStochasticCodes : kAvgThresholdCodes, stream);
      l += launch_avg_codes(stochastic, codes, scales, M, row, p->seed, t, ctx->wsq, qcodes, qscale, count_out,
                            ctx->shape, stream);
    }
  }
  if (stochastic && qthreshold) cudaMemsetAsync(qthreshold, 0, sizeof(float), stream);
}

// Workers' side with sparse selection on validated arguments: indicators, then Q(S(g, I)).
void select_quantize_pack(qasg_ctx* ctx, int rule, const float* g, uint64_t d, uint64_t ld_g, uint32_t M, uint64_t t,
                          const qasg_params* p, const float* x, const float* h, const float* z, uint32_t* codes,
                          float* scales, float* thresholds, uint64_t* counts, uint32_t* indicators,
                          uint64_t* selected, cudaStream_t stream) {
  // The selection kernel's items are chunks (each for all M workers), not (worker, chunk) pairs: it takes
  // shorter chunks (up to kRowChunks of them, about sixteen rounds of its resident CTAs) so that the launch
  // still balances; its partials have their own slots.
  const Geometry geo_sel =
      make_geometry(d, ld_g, M, kRowChunks, static_cast<uint32_t>(ctx->shape.sm_count) * kSelectCtasPerSm * 16u * M);
  const Geometry geo = make_geometry(d, ld_g, M, kMaxChunks, target_items(ctx));
  const bool stochastic = p->quantizer == QASG_Q_TERNARY_STOCH;
  SelectScalars sc;
  sc.lambda = p->lambda;
  sc.lambda_t = p->lambda * static_cast<float>(t);
  unsigned long long* counts_out = reinterpret_cast<unsigned long long*>(counts);
  clear_ticket_if_dirty(ctx, stream);
  {
    Launch l(ctx, kSelectStats, stream);
    l += launch_select_stats(rule, stochastic, g, geo_sel, x, rule == QASG_RULE_CMD ? h : z, sc, p->thr_coef, ctx->wss,
                             indicators, thresholds, reinterpret_cast<unsigned long long*>(selected), ctx->shape,
                             stream);
  }
  if (!stochastic) {
    Launch l(ctx, kThresholdCodes, stream);
    l += launch_threshold_codes(g, geo, ctx->ws, codes, scales, counts_out, ctx->shape, stream, indicators);
  } else {
    Launch l(ctx, kStochasticCodes, stream);
    l += launch_stochastic_codes(g, geo, p->seed, t, 0u, ctx->ws, codes, scales, counts_out, ctx->shape, stream,
                                 indicators);
  }
}

qasg_status check_gradient(const float* g, uint64_t d, uint64_t ld_g) {
  if (!g) return QASG_ERR_INVALID_ARG;
  if (ld_g < d) return QASG_ERR_INVALID_ARG;
  if ((ld_g & 3u) || !aligned16(g)) return QASG_ERR_ALIGNMENT;
  return QASG_OK;
}

// Everything qasg_step checks before it enqueues anything (shared with qasg_step_host, which must not
// start a copy for a call that will be refused).
qasg_status check_step(const qasg_ctx* ctx, int rule, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                       uint64_t t, const qasg_params* params, const float* x, const float* h, const float* z,
                       const uint32_t* codes_out) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, true, true);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (rule != QASG_RULE_CMD && rule != QASG_RULE_RDA) return QASG_ERR_INVALID_ARG;
  if (!x || !h || t < 1 || (rule == QASG_RULE_RDA && !z)) return QASG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(h) || (z && !aligned16(z)) || (codes_out && !aligned16(codes_out)))
    return QASG_ERR_ALIGNMENT;
  if (params->quantizer != QASG_Q_NONE && !codes_out && !ctx->code_scratch) return QASG_ERR_WORKSPACE;
  return QASG_OK;
}

}  // namespace

extern "C" {

qasg_status qasg_create(qasg_ctx** out, int device, uint64_t d_max, uint32_t M_max, uint32_t flags) {
  if (!out) return QASG_ERR_INVALID_ARG;
  *out = nullptr;
  if (d_max < 1 || d_max > kMaxD || M_max < 1 || M_max > static_cast<uint32_t>(kMaxWorkers))
    return QASG_ERR_INVALID_ARG;
  if (cudaSetDevice(device) != cudaSuccess) return QASG_ERR_CUDA;
  qasg_ctx* ctx = new (std::nothrow) qasg_ctx();
  if (!ctx) return QASG_ERR_CUDA;
  ctx->device = device;
  ctx->d_max = d_max;
  ctx->M_max = M_max;
  ctx->launches = 0;
  ctx->ticket_dirty = false;
  ctx->profiling = false;
  ctx->stream_row_bytes = kDefaultStreamRowBytes;
  ctx->stream_lag = kAutoLag;
  ctx->wait_polls = 1u << 22;
  ctx->one_launch_step_bytes = kDefaultOneLaunchStepBytes;
  int cooperative = 0;  // the one-launch paths need all their CTAs resident together
  cudaDeviceGetAttribute(&cooperative, cudaDevAttrCooperativeLaunch, device);
  ctx->cooperative = cooperative != 0;
  query_launch_shape(&ctx->shape);
  ctx->shape.chained = !(flags & QASG_CREATE_SERIAL_LAUNCHES);
  const size_t slots = static_cast<size_t>(M_max) * kMaxChunks;
  bool ok = true;
  ok &= cudaMalloc(&ctx->ws.part_sum, slots * sizeof(double)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.part_max, slots * sizeof(uint32_t)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.part_cnt, slots * sizeof(unsigned long long)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.thresholds, kMaxWorkers * sizeof(float)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.scales, kMaxWorkers * sizeof(float)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.counts, kMaxWorkers * sizeof(unsigned long long)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.selected, kMaxWorkers * sizeof(unsigned long long)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ksyn, 64) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.ticket, 64) == cudaSuccess;
  ok &= cudaMalloc(&ctx->ws.status, 64) == cudaSuccess;
  ok &= cudaMalloc(&ctx->logreg_ws, kLogregEntries * 2 * sizeof(float)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->sync, sizeof(StreamSync)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->slots.sum_a, 3 * slots * sizeof(unsigned long long)) == cudaSuccess;
  ctx->slots.sum_b = ctx->slots.sum_a ? ctx->slots.sum_a + slots : nullptr;
  ctx->slots.cnt_b = ctx->slots.sum_a ? ctx->slots.sum_a + 2 * slots : nullptr;
  ok &= cudaMalloc(&ctx->wsq.part_sum, kRowChunks * sizeof(double)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wsq.part_max, kRowChunks * sizeof(uint32_t)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wsq.part_cnt, kRowChunks * sizeof(unsigned long long)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wsq.thresholds, 64) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wsq.scales, 64) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wsq.counts, 64) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wsq.selected, 64) == cudaSuccess;
  ctx->wsq.ticket = ctx->ws.ticket;
  ctx->wsq.status = ctx->ws.status;
  ctx->wss = ctx->ws;
  const size_t sel_slots = static_cast<size_t>(M_max) * kRowChunks;
  ctx->wss.part_sum = nullptr, ctx->wss.part_max = nullptr, ctx->wss.part_cnt = nullptr;
  ok &= cudaMalloc(&ctx->wss.part_sum, sel_slots * sizeof(double)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wss.part_max, sel_slots * sizeof(uint32_t)) == cudaSuccess;
  ok &= cudaMalloc(&ctx->wss.part_cnt, sel_slots * sizeof(unsigned long long)) == cudaSuccess;
  if (ok && !(flags & QASG_CREATE_NO_CODE_SCRATCH)) {
    ok &= cudaMalloc(&ctx->code_scratch, static_cast<size_t>(M_max) * qasg_code_words(d_max) * 4) == cudaSuccess;
    ok &= cudaMalloc(&ctx->qcode_scratch, qasg_code_words(d_max) * 4) == cudaSuccess;
    ok &= cudaMalloc(&ctx->gbar_scratch, ((d_max + 3) / 4) * 4 * sizeof(float)) == cudaSuccess;
    ok &= cudaMalloc(&ctx->ind_scratch, static_cast<size_t>(M_max + 1) * ((d_max + 31) / 32) * 4) == cudaSuccess;
  }
  if (ok) {
    ok &= cudaMemset(ctx->ws.ticket, 0, 64) == cudaSuccess;
    ok &= cudaMemset(ctx->ws.status, 0, 64) == cudaSuccess;
    ok &= cudaMemset(ctx->sync, 0, sizeof(StreamSync)) == cudaSuccess;
    ok &= cudaMemset(ctx->slots.sum_a, 0xFF, 3 * slots * sizeof(unsigned long long)) == cudaSuccess;
    ok &= cudaMemset(ctx->ws.thresholds, 0, kMaxWorkers * sizeof(float)) == cudaSuccess;
    ok &= cudaMemset(ctx->ws.scales, 0, kMaxWorkers * sizeof(float)) == cudaSuccess;
    ok &= cudaMemset(ctx->wsq.thresholds, 0, 64) == cudaSuccess;
    ok &= cudaMemset(ctx->wsq.scales, 0, 64) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    qasg_destroy(ctx);
    return QASG_ERR_CUDA;
  }
  *out = ctx;
  return QASG_OK;
}

qasg_status qasg_destroy(qasg_ctx* ctx) {
  if (!ctx) return QASG_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaFree(ctx->ws.part_sum);
  cudaFree(ctx->ws.part_max);
  cudaFree(ctx->ws.part_cnt);
  cudaFree(ctx->ws.thresholds);
  cudaFree(ctx->ws.scales);
  cudaFree(ctx->ws.counts);
  cudaFree(ctx->ws.ticket);
  cudaFree(ctx->ws.status);
  cudaFree(ctx->logreg_ws);
  cudaFree(ctx->sync);
  cudaFree(ctx->slots.sum_a);
  cudaFree(ctx->code_scratch);
  cudaFree(ctx->qcode_scratch);
  cudaFree(ctx->gbar_scratch);
  cudaFree(ctx->ind_scratch);
  cudaFree(ctx->ksyn);
  cudaFree(ctx->ws.selected);
  cudaFree(ctx->wsq.selected);
  cudaFree(ctx->wss.part_sum);
  cudaFree(ctx->wss.part_max);
  cudaFree(ctx->wss.part_cnt);
  cudaFree(ctx->wsq.part_sum);
  cudaFree(ctx->wsq.part_max);
  cudaFree(ctx->wsq.part_cnt);
  cudaFree(ctx->wsq.thresholds);
  cudaFree(ctx->wsq.scales);
  cudaFree(ctx->wsq.counts);
  for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
  delete ctx;
  return QASG_OK;
}

uint64_t qasg_code_words(uint64_t d) { return (d + 15) >> 4; }

qasg_status qasg_set_option(qasg_ctx* ctx, qasg_option option, uint64_t value) {
  if (!ctx) return QASG_ERR_INVALID_ARG;
  switch (option) {
    case QASG_OPT_STREAM_ROW_BYTES:
      ctx->stream_row_bytes = value;
      return QASG_OK;
    case QASG_OPT_STREAM_LAG:
      if (value != kAutoLag && value > static_cast<uint64_t>(kMaxWorkers)) return QASG_ERR_INVALID_ARG;
      ctx->stream_lag = static_cast<uint32_t>(value);
      return QASG_OK;
    case QASG_OPT_WAIT_POLLS:
      if (value < 1 || value > (1ull << 31)) return QASG_ERR_INVALID_ARG;
      ctx->wait_polls = static_cast<uint32_t>(value);
      return QASG_OK;
    case QASG_OPT_ONE_LAUNCH_STEP_BYTES:
      ctx->one_launch_step_bytes = value;
      return QASG_OK;
  }
  return QASG_ERR_INVALID_ARG;
}

qasg_status qasg_wait_selftest(qasg_ctx* ctx, uint32_t max_polls, void* stream) {
  if (!ctx || max_polls < 1 || max_polls > (1u << 24)) return QASG_ERR_INVALID_ARG;
  qasg_status st = enter(ctx);
  if (st != QASG_OK) return st;
  ctx->launches += launch_wait_selftest(ctx->sync, ctx->ws.status, max_polls, static_cast<cudaStream_t>(stream));
  return leave(ctx);
}

qasg_status qasg_quantize_pack(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                               uint64_t t, const qasg_params* params, uint32_t* codes, float* scales,
                               float* thresholds, uint64_t* counts, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, false);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (!codes || !scales || t < 1) return QASG_ERR_INVALID_ARG;
  if (!aligned16(codes)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  quantize_pack(ctx, g, d, ld_g, M, t, params, codes, scales, thresholds, counts,
                static_cast<cudaStream_t>(stream));
  return leave(ctx);
}

qasg_status qasg_decode_average(qasg_ctx* ctx, const uint32_t* codes, const float* scales, uint64_t d,
                                uint32_t M, float* gbar, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st != QASG_OK) return st;
  if (!codes || !scales || !gbar) return QASG_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(gbar)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  { Launch l(ctx, kDecodeAverage, static_cast<cudaStream_t>(stream)); l += launch_decode_average(codes, scales, d, M, gbar, ctx->ws.status, ctx->shape,
                                         static_cast<cudaStream_t>(stream)); }
  return leave(ctx);
}

qasg_status qasg_cmd_step(qasg_ctx* ctx, const float* q, float* x, float* h, uint64_t d, uint64_t t,
                          const qasg_params* params, void* stream) {
  qasg_status st = check_shape(ctx, d, 1);
  if (st == QASG_OK) st = check_params(params, true);
  if (st != QASG_OK) return st;
  if (!q || !x || !h || t < 1) return QASG_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(x) || !aligned16(h)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  { Launch l(ctx, kDenseUpdateCmd, static_cast<cudaStream_t>(stream)); l += launch_dense_update(QASG_RULE_CMD, q, d, x, h, nullptr, scalars(params, t), ctx->shape,
                                       static_cast<cudaStream_t>(stream)); }
  return leave(ctx);
}

qasg_status qasg_rda_step(qasg_ctx* ctx, const float* q, float* x, float* h, float* z, uint64_t d,
                          uint64_t t, const qasg_params* params, void* stream) {
  qasg_status st = check_shape(ctx, d, 1);
  if (st == QASG_OK) st = check_params(params, true);
  if (st != QASG_OK) return st;
  if (!q || !x || !h || !z || t < 1) return QASG_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(x) || !aligned16(h) || !aligned16(z)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  { Launch l(ctx, kDenseUpdateRda, static_cast<cudaStream_t>(stream)); l += launch_dense_update(QASG_RULE_RDA, q, d, x, h, z, scalars(params, t), ctx->shape,
                                       static_cast<cudaStream_t>(stream)); }
  return leave(ctx);
}

qasg_status qasg_step(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                      uint64_t t, const qasg_params* params, float* x, float* h, float* z,
                      uint32_t* codes_out, float* scales_out, void* stream) {
  qasg_status st = check_step(ctx, rule, g, d, ld_g, M, t, params, x, h, z, codes_out);
  if (st != QASG_OK) return st;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (params->quantizer == QASG_Q_NONE) {
    Launch l(ctx, rule == QASG_RULE_CMD ? kMeanUpdateCmd : kMeanUpdateRda, s);
    l += launch_mean_update(rule, g, d, ld_g, M, x, h, z, scalars(params, t), ctx->ws.status, ctx->shape, s);
    return leave(ctx);
  }
  uint32_t* codes = codes_out ? codes_out : ctx->code_scratch;
  if (ctx->cooperative && static_cast<uint64_t>(M) * d * 4 <= ctx->one_launch_step_bytes) {  // small: the three passes as one launch
    const Geometry geo = make_geometry(d, ld_g, M, kMaxChunks, target_items(ctx));
    Launch l(ctx, rule == QASG_RULE_CMD ? kFusedStepCmd : kFusedStepRda, s);
    l += launch_fused_step(rule, params->quantizer == QASG_Q_TERNARY_STOCH, g, geo, params->thr_coef, params->seed, t,
                           0u, ctx->wait_polls, ctx->ws, ctx->wss, ctx->sync, codes, scales_out, x, h, z, scalars(params, t),
                           ctx->shape, s);
    return leave(ctx);
  }
  quantize_pack(ctx, g, d, ld_g, M, t, params, codes, scales_out, nullptr, nullptr, s);
  { Launch l(ctx, rule == QASG_RULE_CMD ? kDecodeUpdateCmd : kDecodeUpdateRda, s); l += launch_decode_update(rule, codes, ctx->ws.scales, d, M, x, h, z, scalars(params, t),
                                        ctx->ws.status, ctx->shape, s); }
  return leave(ctx);
}

qasg_status qasg_quantize_pack_touched(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                                       uint64_t t, const qasg_params* params, const uint32_t* touched,
                                       uint32_t* codes, float* scales, float* thresholds, uint64_t* counts,
                                       void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, false);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (!touched || !codes || !scales || t < 1) return QASG_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(touched)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  quantize_pack(ctx, g, d, ld_g, M, t, params, codes, scales, thresholds, counts, static_cast<cudaStream_t>(stream),
                touched);
  return leave(ctx);
}

qasg_status qasg_step_touched(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                              uint64_t t, const qasg_params* params, const uint32_t* touched, float* x, float* h,
                              float* z, uint32_t* codes_out, float* scales_out, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, true);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (rule != QASG_RULE_CMD && rule != QASG_RULE_RDA) return QASG_ERR_INVALID_ARG;
  if (!touched || !x || !h || t < 1 || (rule == QASG_RULE_RDA && !z)) return QASG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(h) || (z && !aligned16(z)) || (codes_out && !aligned16(codes_out)) ||
      !aligned16(touched))
    return QASG_ERR_ALIGNMENT;
  uint32_t* codes = codes_out ? codes_out : ctx->code_scratch;
  if (!codes) return QASG_ERR_WORKSPACE;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  quantize_pack(ctx, g, d, ld_g, M, t, params, codes, scales_out, nullptr, nullptr, s, touched);
  {
    Launch l(ctx, rule == QASG_RULE_CMD ? kDecodeUpdateCmd : kDecodeUpdateRda, s);
    l += launch_decode_update(rule, codes, ctx->ws.scales, d, M, x, h, z, scalars(params, t), ctx->ws.status,
                              ctx->shape, s);
  }
  return leave(ctx);
}

uint64_t qasg_optimal_scratch_bytes(uint64_t d) { return (d >= 1 && d < (1ull << 31)) ? optimal_scratch_bytes(d) : 0; }

qasg_status qasg_quantize_pack_optimal(qasg_ctx* ctx, const float* g, uint64_t d, uint64_t ld_g, uint32_t M,
                                       const qasg_params* params, uint32_t* codes, float* scales,
                                       float* thresholds, uint64_t* counts, void* scratch, uint64_t scratch_bytes,
                                       void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, false);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (!codes || !scales || !scratch || params->quantizer != QASG_Q_THRESHOLD || d >= (1ull << 31))
    return QASG_ERR_INVALID_ARG;
  if (!aligned16(codes) || (reinterpret_cast<uintptr_t>(scratch) & 255u)) return QASG_ERR_ALIGNMENT;
  if (scratch_bytes < optimal_scratch_bytes(d)) return QASG_ERR_WORKSPACE;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  clear_ticket_if_dirty(ctx, s);
  for (uint32_t m = 0; m < M; ++m) {  // one row after the other through the same scratch
    Launch l(ctx, kOptimalThreshold, s);
    l += launch_optimal_threshold(g + static_cast<uint64_t>(m) * ld_g, d, scratch, ctx->ws.thresholds + m,
                                  thresholds ? thresholds + m : nullptr, nullptr, ctx->ws.status, s);
  }
  const Geometry geo = make_geometry(d, ld_g, M, kMaxChunks, target_items(ctx));
  {
    Launch l(ctx, kThresholdCodes, s);
    l += launch_threshold_codes(g, geo, ctx->ws, codes, scales, reinterpret_cast<unsigned long long*>(counts),
                                ctx->shape, s);
  }
  return leave(ctx);
}

qasg_status qasg_requantize(qasg_ctx* ctx, const uint32_t* codes, const float* scales, uint64_t d, uint32_t M,
                            uint64_t t, const qasg_params* params, uint32_t* qcodes, float* qscale,
                            float* qthreshold, uint64_t* qcount, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, false);
  if (st != QASG_OK) return st;
  if (!codes || !scales || !qcodes || !qscale || t < 1) return QASG_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(qcodes)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  requantize(ctx, codes, scales, d, M, t, params, qcodes, qscale, qthreshold, qcount,
             static_cast<cudaStream_t>(stream));
  return leave(ctx);
}

qasg_status qasg_step_double(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g,
                             uint32_t M, uint64_t t, const qasg_params* params, float* x, float* h, float* z,
                             uint32_t* codes_out, float* scales_out, uint32_t* qcodes_out, float* qscale_out,
                             void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, true);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (rule != QASG_RULE_CMD && rule != QASG_RULE_RDA) return QASG_ERR_INVALID_ARG;
  if (!x || !h || t < 1 || (rule == QASG_RULE_RDA && !z)) return QASG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(h) || (z && !aligned16(z)) || (codes_out && !aligned16(codes_out)) ||
      (qcodes_out && !aligned16(qcodes_out)))
    return QASG_ERR_ALIGNMENT;
  uint32_t* codes = codes_out ? codes_out : ctx->code_scratch;
  uint32_t* qcodes = qcodes_out ? qcodes_out : ctx->qcode_scratch;
  if (!codes || !qcodes) return QASG_ERR_WORKSPACE;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  quantize_pack(ctx, g, d, ld_g, M, t, params, codes, scales_out, nullptr, nullptr, s);
  requantize(ctx, codes, ctx->ws.scales, d, M, t, params, qcodes, qscale_out, nullptr, nullptr, s);
  {
    // the workers decode q_t (one code row, one scale) and update
    Launch l(ctx, rule == QASG_RULE_CMD ? kDecodeUpdateCmd : kDecodeUpdateRda, s);
    l += launch_decode_update(rule, qcodes, ctx->wsq.scales, d, 1, x, h, z, scalars(params, t), ctx->ws.status,
                              ctx->shape, s);
  }
  return leave(ctx);
}

qasg_status qasg_select_quantize_pack(qasg_ctx* ctx, qasg_rule rule, const float* g, uint64_t d, uint64_t ld_g,
                                      uint32_t M, uint64_t t, const qasg_params* params, const float* x,
                                      const float* h, const float* z, uint32_t* codes, float* scales,
                                      float* thresholds, uint64_t* counts, uint32_t* indicators,
                                      uint64_t* selected, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, true);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (rule != QASG_RULE_CMD && rule != QASG_RULE_RDA) return QASG_ERR_INVALID_ARG;
  if (!x || !codes || !scales || !indicators || t < 1) return QASG_ERR_INVALID_ARG;
  if (rule == QASG_RULE_RDA && !z) return QASG_ERR_INVALID_ARG;  // neither test reads h
  if (!aligned16(x) || (h && !aligned16(h)) || (z && !aligned16(z)) || !aligned16(codes) || !aligned16(indicators))
    return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  select_quantize_pack(ctx, rule, g, d, ld_g, M, t, params, x, h, z, codes, scales, thresholds, counts, indicators,
                       selected, static_cast<cudaStream_t>(stream));
  return leave(ctx);
}

qasg_status qasg_indicator_or(qasg_ctx* ctx, const uint32_t* indicators, uint64_t d, uint32_t M, uint32_t* isyn,
                              uint64_t* ksyn, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st != QASG_OK) return st;
  if (!indicators || !isyn || !ksyn) return QASG_ERR_INVALID_ARG;
  if ((st = enter(ctx)) != QASG_OK) return st;
  {
    Launch l(ctx, kIndicatorOr, static_cast<cudaStream_t>(stream));
    l += launch_indicator_or(indicators, d, M, isyn, reinterpret_cast<unsigned long long*>(ksyn), ctx->shape,
                             static_cast<cudaStream_t>(stream));
  }
  return leave(ctx);
}

qasg_status qasg_step_select(qasg_ctx* ctx, qasg_rule rule, int double_quant, const float* g, uint64_t d,
                             uint64_t ld_g, uint32_t M, uint64_t t, const qasg_params* params, float* x, float* h,
                             float* z, uint32_t* codes_out, float* scales_out, uint32_t* indicators_out,
                             uint64_t* selected_out, uint32_t* isyn_out, uint64_t* ksyn_out, void* stream) {
  qasg_status st = check_shape(ctx, d, M);
  if (st == QASG_OK) st = check_params(params, true);
  if (st == QASG_OK) st = check_gradient(g, d, ld_g);
  if (st != QASG_OK) return st;
  if (rule != QASG_RULE_CMD && rule != QASG_RULE_RDA) return QASG_ERR_INVALID_ARG;
  if (!x || !h || t < 1 || (rule == QASG_RULE_RDA && !z)) return QASG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(h) || (z && !aligned16(z)) || (codes_out && !aligned16(codes_out)) ||
      (indicators_out && !aligned16(indicators_out)))
    return QASG_ERR_ALIGNMENT;
  uint32_t* codes = codes_out ? codes_out : ctx->code_scratch;
  uint32_t* indicators = indicators_out ? indicators_out : ctx->ind_scratch;
  uint32_t* isyn = isyn_out;  // else the row after the M_max indicator rows of the scratch
  if (!isyn && ctx->ind_scratch) isyn = ctx->ind_scratch + static_cast<size_t>(ctx->M_max) * ((ctx->d_max + 31) / 32);
  const bool need_or = double_quant || isyn_out || ksyn_out;
  if (!codes || !indicators || (need_or && !isyn) || (double_quant && !ctx->qcode_scratch)) return QASG_ERR_WORKSPACE;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  select_quantize_pack(ctx, rule, g, d, ld_g, M, t, params, x, h, z, codes, scales_out, nullptr, nullptr, indicators,
                       selected_out, s);
  unsigned long long* ksyn = ksyn_out ? reinterpret_cast<unsigned long long*>(ksyn_out) : ctx->ksyn;
  if (need_or) {
    Launch l(ctx, kIndicatorOr, s);
    l += launch_indicator_or(indicators, d, M, isyn, ksyn, ctx->shape, s);
  }
  if (double_quant) {
    requantize(ctx, codes, ctx->ws.scales, d, M, t, params, ctx->qcode_scratch, nullptr, nullptr, nullptr, s, ksyn);
    Launch l(ctx, rule == QASG_RULE_CMD ? kDecodeUpdateCmd : kDecodeUpdateRda, s);
    l += launch_decode_update(rule, ctx->qcode_scratch, ctx->wsq.scales, d, 1, x, h, z, scalars(params, t),
                              ctx->ws.status, ctx->shape, s);
  } else {
    Launch l(ctx, rule == QASG_RULE_CMD ? kDecodeUpdateCmd : kDecodeUpdateRda, s);
    l += launch_decode_update(rule, codes, ctx->ws.scales, d, M, x, h, z, scalars(params, t), ctx->ws.status,
                              ctx->shape, s);
  }
  return leave(ctx);
}

qasg_status qasg_step_host(qasg_ctx* ctx, qasg_rule rule, const float* g_host, uint64_t d, uint64_t ld_g,
                           uint32_t M, uint64_t t, const qasg_params* params, float* x_host, float* h_host,
                           float* z_host, float* g_dev, float* x_dev, float* h_dev, float* z_dev,
                           void* stream) {
  // every check of qasg_step on the staging buffers comes first: a refused call copies nothing
  qasg_status st = check_step(ctx, rule, g_dev, d, ld_g, M, t, params, x_dev, h_dev, z_dev, nullptr);
  if (st != QASG_OK) return st;
  if (!g_host || !x_host || !h_host || (rule == QASG_RULE_RDA && !z_host)) return QASG_ERR_INVALID_ARG;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t vec = d * sizeof(float);
  bool ok = true;
  ok &= cudaMemcpy2DAsync(g_dev, ld_g * sizeof(float), g_host, ld_g * sizeof(float), vec, M,
                          cudaMemcpyHostToDevice, s) == cudaSuccess;
  if (rule == QASG_RULE_CMD) ok &= cudaMemcpyAsync(x_dev, x_host, vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok &= cudaMemcpyAsync(h_dev, h_host, vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
  if (rule == QASG_RULE_RDA) ok &= cudaMemcpyAsync(z_dev, z_host, vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return QASG_ERR_CUDA;
  }
  st = qasg_step(ctx, rule, g_dev, d, ld_g, M, t, params, x_dev, h_dev, z_dev, nullptr, nullptr, stream);
  if (st != QASG_OK) return st;
  ok &= cudaMemcpyAsync(x_host, x_dev, vec, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  ok &= cudaMemcpyAsync(h_host, h_dev, vec, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (rule == QASG_RULE_RDA) ok &= cudaMemcpyAsync(z_host, z_dev, vec, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return QASG_ERR_CUDA;
  }
  return QASG_OK;
}

static qasg_status check_logreg(qasg_ctx* ctx, const float* y, uint64_t n_rows, uint64_t d, uint32_t M,
                                const uint64_t* shard_row0, uint32_t B, uint64_t t, const float* x,
                                const float* g, uint64_t ld_g) {
  qasg_status st = check_shape(ctx, d, M);
  if (st != QASG_OK) return st;
  if (!y || !shard_row0 || !x || !g || B < 1 || t < 1 || n_rows < 1) return QASG_ERR_INVALID_ARG;
  if (ld_g < d) return QASG_ERR_INVALID_ARG;
  if ((ld_g & 3u) || !aligned16(g) || !aligned16(x)) return QASG_ERR_ALIGNMENT;
  if (static_cast<uint64_t>(M) * B > kLogregEntries) return QASG_ERR_WORKSPACE;
  for (uint32_t m = 0; m < M; ++m)
    if (shard_row0[m + 1] <= shard_row0[m] || shard_row0[m + 1] > n_rows) return QASG_ERR_INVALID_ARG;
  if (n_rows > 0xffffffffull) return QASG_ERR_INVALID_ARG;
  return QASG_OK;
}

qasg_status qasg_logreg_grad_dense(qasg_ctx* ctx, const float* X, const float* y, uint64_t n_rows, uint64_t d,
                                   uint32_t M, const uint64_t* shard_row0, const uint32_t* batch_rows,
                                   uint32_t B, uint64_t t, const float* x, float* g, uint64_t ld_g,
                                   void* stream) {
  qasg_status st = check_logreg(ctx, y, n_rows, d, M, shard_row0, B, t, x, g, ld_g);
  if (st != QASG_OK) return st;
  if (!X) return QASG_ERR_INVALID_ARG;
  if ((d & 3u) || !aligned16(X)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  { Launch l(ctx, kLogregDense, static_cast<cudaStream_t>(stream)); l += launch_logreg_dense(X, y, n_rows, d, M, shard_row0, batch_rows, B, t, x, g, ld_g, ctx->logreg_ws,
                                       ctx->ws.status, ctx->shape, static_cast<cudaStream_t>(stream)); }
  return leave(ctx);
}

qasg_status qasg_logreg_grad_csr(qasg_ctx* ctx, const int64_t* rowptr, const int32_t* colidx,
                                 const float* vals, const float* y, uint64_t n_rows, uint64_t d, uint32_t M,
                                 const uint64_t* shard_row0, const uint32_t* batch_rows, uint32_t B,
                                 uint64_t t, const float* x, float* g, uint64_t ld_g, void* stream) {
  qasg_status st = check_logreg(ctx, y, n_rows, d, M, shard_row0, B, t, x, g, ld_g);
  if (st != QASG_OK) return st;
  if (!rowptr || !colidx || !vals) return QASG_ERR_INVALID_ARG;
  if ((st = enter(ctx)) != QASG_OK) return st;
  { Launch l(ctx, kLogregCsr, static_cast<cudaStream_t>(stream)); l += launch_logreg_csr(rowptr, colidx, vals, y, n_rows, d, M, shard_row0, batch_rows, B, t, x, g, ld_g,
                                     ctx->ws.status, ctx->shape, static_cast<cudaStream_t>(stream)); }
  return leave(ctx);
}

qasg_status qasg_logreg_grad_csr_touched(qasg_ctx* ctx, const int64_t* rowptr, const int32_t* colidx,
                                         const float* vals, const float* y, uint64_t n_rows, uint64_t d,
                                         uint32_t M, const uint64_t* shard_row0, const uint32_t* batch_rows,
                                         uint32_t B, uint64_t t, const float* x, float* g, uint64_t ld_g,
                                         uint32_t* touched, void* stream) {
  qasg_status st = check_logreg(ctx, y, n_rows, d, M, shard_row0, B, t, x, g, ld_g);
  if (st != QASG_OK) return st;
  if (!rowptr || !colidx || !vals || !touched) return QASG_ERR_INVALID_ARG;
  if (!aligned16(touched)) return QASG_ERR_ALIGNMENT;
  if ((st = enter(ctx)) != QASG_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  { Launch l(ctx, kTouchedClear, s); l += launch_touched_clear(g, d, ld_g, M, touched, ctx->shape, s); }
  {
    Launch l(ctx, kLogregCsrTouched, s);
    l += launch_logreg_csr(rowptr, colidx, vals, y, n_rows, d, M, shard_row0, batch_rows, B, t, x, g, ld_g,
                           ctx->ws.status, ctx->shape, s,
                           touched);
  }
  return leave(ctx);
}

qasg_status qasg_last_async_status(qasg_ctx* ctx, void* stream) {
  if (!ctx) return QASG_ERR_INVALID_ARG;
  if (enter(ctx) != QASG_OK) return QASG_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned int flags = 0;
  if (cudaMemcpyAsync(&flags, ctx->ws.status, sizeof(flags), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaMemsetAsync(ctx->ws.status, 0, sizeof(flags), s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) {
    cudaGetLastError();
    return QASG_ERR_CUDA;
  }
  if (flags & kFlagTimeout) {  // a call gave up half-way: its tickets and abort word are left set
    cudaMemsetAsync(ctx->sync, 0, sizeof(StreamSync), s);
    cudaMemsetAsync(ctx->slots.sum_a, 0xFF, 3 * static_cast<size_t>(ctx->M_max) * kMaxChunks * sizeof(unsigned long long), s);
    cudaStreamSynchronize(s);
    return QASG_ERR_TIMEOUT;
  }
  if (flags & kFlagNonFinite) return QASG_ERR_NONFINITE;
  if (flags & kFlagBadCode) return QASG_ERR_BAD_CODE;
  if (flags & kFlagBadIndex) return QASG_ERR_BAD_INDEX;
  return QASG_OK;
}

uint64_t qasg_launch_count(const qasg_ctx* ctx) { return ctx ? ctx->launches : 0; }

qasg_status qasg_profile_begin(qasg_ctx* ctx) {
  if (!ctx) return QASG_ERR_INVALID_ARG;
  ctx->event_kernel.clear();
  ctx->profiling = true;
  return QASG_OK;
}

qasg_status qasg_profile_end(qasg_ctx* ctx, double* ms, uint64_t* launches) {
  if (!ctx || !ms || !launches) return QASG_ERR_INVALID_ARG;
  ctx->profiling = false;
  for (int k = 0; k < QASG_KERNEL_COUNT; ++k) {
    ms[k] = 0.0;
    launches[k] = 0;
  }
  if (enter(ctx) != QASG_OK) return QASG_ERR_CUDA;
  for (size_t i = 0; i < ctx->event_kernel.size(); ++i) {
    float elapsed = 0.f;
    if (cudaEventSynchronize(ctx->events[2 * i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&elapsed, ctx->events[2 * i], ctx->events[2 * i + 1]) != cudaSuccess) {
      cudaGetLastError();
      return QASG_ERR_CUDA;
    }
    ms[ctx->event_kernel[i]] += elapsed;
    launches[ctx->event_kernel[i]] += 1;
  }
  ctx->event_kernel.clear();
  return QASG_OK;
}

const char* qasg_kernel_name(int id) {
  static const char* const names[kKernelIdCount] = {
      "abs_sum", "abs_max", "threshold_codes", "stochastic_codes", "decode_update_cmd", "decode_update_rda",
      "decode_average", "dense_update_cmd", "dense_update_rda", "logreg_dense", "logreg_csr", "avg_abs_sum",
      "avg_abs_max", "avg_threshold_codes", "avg_stochastic_codes", "select_stats", "indicator_or",
      "touched_clear", "logreg_csr_touched", "optimal_threshold", "mean_update_cmd", "mean_update_rda",
      "quantize_stream_threshold", "quantize_stream_stochastic", "fused_step_cmd", "fused_step_rda"};
  return (id >= 0 && id < kKernelIdCount) ? names[id] : "";
}

const char* qasg_status_string(qasg_status s) {
  switch (s) {
    case QASG_OK: return "ok";
    case QASG_ERR_INVALID_ARG: return "invalid argument";
    case QASG_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
    case QASG_ERR_WORKSPACE: return "size beyond the context's workspace";
    case QASG_ERR_CUDA: return "CUDA runtime error";
    case QASG_ERR_TIMEOUT: return "device-side wait timed out";
    case QASG_ERR_NONFINITE: return "non-finite gradient";
    case QASG_ERR_BAD_CODE: return "invalid code value in packed words";
    case QASG_ERR_BAD_INDEX: return "row or column index out of range";
  }
  return "unknown status";
}

}  // extern "C"
